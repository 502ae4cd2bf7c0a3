// Backward of one block-attention training step (Section 4.2: Eq. 4 early stage, Eq. 7 late stage;
// Appendix B: smooth-L1 regression of the draft state on the target's true state): the element-wise,
// normalisation, transpose and attention kernels around the dense products, which reuse the
// forward's GEMM as  dX = dY W  (the weight transposed once)  and  dW = dY^T X  (both operands
// transposed, so that the contraction runs along rows of length M).
//
// Under simulation the predicted states that earlier steps wrote in place are inputs of the final
// step, like the true states they replace: no gradient flows into them, W_K and W_V receive the
// gradient of projecting them.
#include "kernels.h"

namespace beagle {

namespace {

// ------------------------------------------------------------------------------------------------
// out[c][col0 + r] = in[r][c] for r < rows, c < cols; columns col0 + rows .. col0 + rows_pad - 1 of
// every output row are zero-filled (the contraction length is padded to a multiple of 8).
// 32 x 32 tiles through shared memory.
// ------------------------------------------------------------------------------------------------
// blockIdx.z = batch: the input advances by in_bs elements and the output column offset by col_bs per batch.
template <typename T>
__global__ void __launch_bounds__(256) transpose_pad_kernel(const T* __restrict__ in, int rows, int cols, int ld_in, T* __restrict__ out,
                                                           int ld_out, int col0, int rows_pad, size_t in_bs, int col_bs) {
    __shared__ T tile[32][33];
    in += (size_t)blockIdx.z * in_bs;
    col0 += (int)blockIdx.z * col_bs;
    const int r0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;     // 8 rows of 32 threads
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + ty + i * 8, c = c0 + tx;
        tile[ty + i * 8][tx] = (r < rows && c < cols) ? in[(size_t)r * ld_in + c] : from_float<T>(0.f);
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = c0 + ty + i * 8, r = r0 + tx;
        if (c < cols && r < rows_pad) out[(size_t)c * ld_out + col0 + r] = tile[tx][ty + i * 8];
    }
}

// bf16, 64 x 64 tiles, 16-byte global accesses on both sides.  The tile lives in shared memory as 64 rows of eight
// 16-byte chunks; chunk cc of row r is stored at chunk position cc ^ ((r >> 3) & 7), so that the eight rows
// r = 8 rc + j (rc = 0..7) which one output chunk gathers from lie in different banks.
// Needs ld_in, ld_out, col0, rows_pad multiples of 8 and 16-byte aligned bases.
__global__ void __launch_bounds__(256) transpose_pad_bf16_kernel(const bf16* __restrict__ in, int rows, int cols, int ld_in, bf16* __restrict__ out,
                                                                int ld_out, int col0, int rows_pad, size_t in_bs, int col_bs) {
    __shared__ __align__(16) bf16 tile[64 * 64];
    in += (size_t)blockIdx.z * in_bs;
    col0 += (int)blockIdx.z * col_bs;
    const int r0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int id = threadIdx.x + 256 * k;
        const int r = id >> 3, cc = id & 7;
        const int gr = r0 + r, gc = c0 + cc * 8;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (gr < rows) {
            if (gc + 8 <= cols) {
                v = *reinterpret_cast<const uint4*>(in + (size_t)gr * ld_in + gc);
            } else if (gc < cols) {
                bf16 e[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) e[i] = gc + i < cols ? in[(size_t)gr * ld_in + gc + i] : __float2bfloat16_rn(0.f);
                v = *reinterpret_cast<const uint4*>(e);
            }
        }
        *reinterpret_cast<uint4*>(tile + r * 64 + ((cc ^ ((r >> 3) & 7)) << 3)) = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int id = threadIdx.x + 256 * k;
        const int rc = id & 7, c = id >> 3;                 // output row c0 + c, elements r0 + 8 rc .. + 7
        if (c0 + c < cols && r0 + rc * 8 < rows_pad) {
            bf16 e[8];
            const int pc = (((c >> 3) ^ rc) << 3) + (c & 7);
#pragma unroll
            for (int j = 0; j < 8; ++j) e[j] = tile[(rc * 8 + j) * 64 + pc];
            *reinterpret_cast<uint4*>(out + (size_t)(c0 + c) * ld_out + col0 + r0 + rc * 8) = *reinterpret_cast<const uint4*>(e);
        }
    }
}

// act = SiLU(gate) * up, element-wise (the training forward keeps gate and up for the backward).  16-byte pieces; n is a
// multiple of the vector width (mlp_dim is a multiple of 8).
template <typename T>
__global__ void __launch_bounds__(256) silu_mul_kernel(const T* __restrict__ gate, const T* __restrict__ up, T* __restrict__ act, size_t n) {
    constexpr int VN = VecOf<T>::N;
    const size_t nv = n / VN;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nv; i += (size_t)gridDim.x * blockDim.x) {
        float g[VN], u[VN];
        unpack16<T>(reinterpret_cast<const uint4*>(gate)[i], g);
        unpack16<T>(reinterpret_cast<const uint4*>(up)[i], u);
        T o[VN];
#pragma unroll
        for (int k = 0; k < VN; ++k) o[k] = from_float<T>(silu_f(g[k]) * u[k]);
        reinterpret_cast<uint4*>(act)[i] = *reinterpret_cast<const uint4*>(o);
    }
}

// In place: gate <- d gate = dact * up * sigma(gate) (1 + gate (1 - sigma(gate))), up <- d up = dact * SiLU(gate).
template <typename T>
__global__ void __launch_bounds__(256) silu_mul_bwd_kernel(T* __restrict__ gate, T* __restrict__ up, const T* __restrict__ dact, size_t n) {
    constexpr int VN = VecOf<T>::N;
    const size_t nv = n / VN;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nv; i += (size_t)gridDim.x * blockDim.x) {
        float g[VN], u[VN], da[VN];
        unpack16<T>(reinterpret_cast<const uint4*>(gate)[i], g);
        unpack16<T>(reinterpret_cast<const uint4*>(up)[i], u);
        unpack16<T>(reinterpret_cast<const uint4*>(dact)[i], da);
        T og[VN], ou[VN];
#pragma unroll
        for (int k = 0; k < VN; ++k) {
            const float sg = 1.0f / (1.0f + __expf(-g[k]));
            og[k] = from_float<T>(da[k] * u[k] * sg * (1.0f + g[k] * (1.0f - sg)));
            ou[k] = from_float<T>(da[k] * g[k] * sg);
        }
        reinterpret_cast<uint4*>(gate)[i] = *reinterpret_cast<const uint4*>(og);
        reinterpret_cast<uint4*>(up)[i] = *reinterpret_cast<const uint4*>(ou);
    }
}

__device__ __forceinline__ float loss_weight(int row, int S, int block, int offset, int sim_steps, int stage) {
    const int p = row % S + 1;
    if (p <= offset) return 0.f;
    const int n = offset + block * ((p - 1 - offset) / block);
    const int slot = p - n;
    return stage == 0 ? 1.f : (slot <= sim_steps ? (float)(block - slot + 1) : 0.f);
}

// d z = coef(row) * (softmax(z) - p) for one chunk of materialised fp32 logits; p = softmax of the
// target logits or the point mass at the label.  stats[row] = merged (max z, exp-sum z, max t,
// exp-sum t) of the loss forward.  Columns V .. ldz-1 are zero-filled.
template <typename T, typename TT>
__global__ void __launch_bounds__(256) dlogits_kernel(const float* __restrict__ logits, int V, const TT* __restrict__ tgt,
                                                     const int32_t* __restrict__ labels, const float4* __restrict__ stats, int row0, int S,
                                                     int block, int offset, int sim_steps, int stage, float scale, T* __restrict__ dz, int ldz) {
    const int r = blockIdx.x, row = row0 + r;
    const float coef = loss_weight(row, S, block, offset, sim_steps, stage) * scale;
    const float4 st = stats[row];
    const float inv_q = 1.0f / st.y, inv_t = tgt != nullptr ? 1.0f / st.w : 0.f;
    const float* z = logits + (size_t)r * V;
    const int label = tgt == nullptr ? labels[row] : -1;
    T* out = dz + (size_t)row * ldz;
    for (int v = threadIdx.x; v < ldz; v += blockDim.x) {
        float g = 0.f;
        if (v < V && coef != 0.f) {
            const float q = __expf(z[v] - st.x) * inv_q;
            const float p = tgt != nullptr ? __expf((float)to_float<TT>(tgt[(size_t)row * V + v]) - st.z) * inv_t : (v == label ? 1.f : 0.f);
            g = coef * (q - p);
        }
        out[v] = from_float<T>(g);
    }
}

__global__ void __launch_bounds__(256) loss_coef_kernel(int rows, int S, int block, int offset, int sim_steps, int stage, float scale,
                                                       float* __restrict__ coef) {
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row < rows) coef[row] = loss_weight(row, S, block, offset, sim_steps, stage) * scale;
}

// Regression term: dh0[row] = coef * reg(row) * clip(h - h_true, -1, 1), and the row's sum of
// smooth_l1(h - h_true) (reg(row) = 1 where the position carries a loss term).
template <typename T>
__global__ void __launch_bounds__(256) vloss_kernel(const T* __restrict__ h, const T* __restrict__ h_true, int d, int S, int block, int offset,
                                                   int sim_steps, int stage, float coef, T* __restrict__ dh0, float* __restrict__ row_sum) {
    const int row = blockIdx.x;
    const bool reg = loss_weight(row, S, block, offset, sim_steps, stage) > 0.f;
    float acc = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float r = to_float<T>(h[(size_t)row * d + i]) - to_float<T>(h_true[(size_t)row * d + i]);
        const float a = fabsf(r);
        if (reg) acc += a < 1.f ? 0.5f * r * r : a - 0.5f;
        dh0[(size_t)row * d + i] = from_float<T>(reg ? coef * fminf(fmaxf(r, -1.f), 1.f) : 0.f);
    }
    acc = warp_sum(acc);
    __shared__ float s[8];
    if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += s[w];
        row_sum[row] = t;
    }
}

// out[0] = loss (already there), out[1] = vloss = sum(row_sum) * vscale, out[2] = loss + vcoef * vloss; fixed order.
__global__ void __launch_bounds__(1024) loss_total_kernel(const float* __restrict__ row_sum, int rows, float vscale, float vcoef, float* __restrict__ out) {
    __shared__ float s[1024];
    float t = 0.f;
    for (int i = threadIdx.x; i < rows; i += 1024) t += row_sum[i];
    s[threadIdx.x] = t;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const float v = s[0] * vscale;
        out[1] = v;
        out[2] = out[0] + vcoef * v;
    }
}

// ------------------------------------------------------------------------------------------------
// RMSNorm backward.  n = g * v * r, r = (mean(v^2) + eps)^(-1/2):
//   dv = r * (g * dn) - v * r^3 * mean(v * g * dn);   dg = sum_rows dn * v * r.
// out = add + dv (add may be NULL).  One CTA of 256 threads per row at a time (rows blockIdx.x,
// += gridDim.x); a thread owns the 16-byte pieces tid, tid + 256, ... of the row (at most kRmsVec of
// them), keeps its columns' dg sums in registers and writes them as one partial row per CTA;
// colsum_kernel adds the partials in a fixed order.  do_norm == 0: out = add + dn, no dg.
// ------------------------------------------------------------------------------------------------
constexpr int kRmsVec = 4;
template <typename T, int NV>      // NV: 16-byte pieces per thread (d <= NV * 256 * pieces' width)
__global__ void __launch_bounds__(256) rmsnorm_bwd_kernel(const T* __restrict__ v, const T* __restrict__ gain, const T* __restrict__ dn,
                                                         const T* __restrict__ add, int rows, int d, float eps, int do_norm,
                                                         T* __restrict__ out, float* __restrict__ dg_part) {
    constexpr int VN = VecOf<T>::N;
    const int nvec = d / VN;
    __shared__ float s_red[2][2][8];                // [parity][sum v^2 | sum v g dn][warp]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float dg[NV][VN];
#pragma unroll
    for (int k = 0; k < NV; ++k)
#pragma unroll
        for (int i = 0; i < VN; ++i) dg[k][i] = 0.f;
    int par = 0;
    for (int row = blockIdx.x; row < rows; row += gridDim.x, par ^= 1) {
        const size_t base = (size_t)row * d;
        float x[NV][VN], dd[NV][VN];
        float ss = 0.f, dot = 0.f;
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int ch = threadIdx.x + k * 256;
            if (ch < nvec) {
                float gg[VN];
                unpack16<T>(ld_cached16(v + base + ch * VN), x[k]);
                unpack16<T>(ld_cached16(dn + base + ch * VN), dd[k]);
                if (do_norm) unpack16<T>(ld_cached16(gain + ch * VN), gg);
#pragma unroll
                for (int i = 0; i < VN; ++i) {
                    ss = fmaf(x[k][i], x[k][i], ss);
                    dot = fmaf(x[k][i], do_norm ? gg[i] * dd[k][i] : dd[k][i], dot);
                }
            }
        }
        float r = 1.f, kfac = 0.f;
        if (do_norm) {
            ss = warp_sum(ss); dot = warp_sum(dot);
            if (lane == 0) { s_red[par][0][warp] = ss; s_red[par][1][warp] = dot; }
            __syncthreads();                        // the other parity's slots are rewritten only after the next barrier
            float tss = 0.f, tdot = 0.f;
#pragma unroll
            for (int w8 = 0; w8 < 8; ++w8) { tss += s_red[par][0][w8]; tdot += s_red[par][1][w8]; }
            r = rsqrtf(tss / (float)d + eps);
            kfac = r * r * r * tdot / (float)d;
        }
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int ch = threadIdx.x + k * 256;
            if (ch < nvec) {
                float av[VN], gg[VN];
                if (add != nullptr) unpack16<T>(ld_cached16(add + base + ch * VN), av);
                if (do_norm) unpack16<T>(ld_cached16(gain + ch * VN), gg);
                T o8[VN];
#pragma unroll
                for (int i = 0; i < VN; ++i) {
                    const float dv = do_norm ? r * gg[i] * dd[k][i] - x[k][i] * kfac : dd[k][i];
                    o8[i] = from_float<T>(dv + (add != nullptr ? av[i] : 0.f));
                    dg[k][i] = fmaf(dd[k][i] * x[k][i], r, dg[k][i]);
                }
                *reinterpret_cast<uint4*>(out + base + ch * VN) = *reinterpret_cast<const uint4*>(o8);
            }
        }
    }
    if (!do_norm || dg_part == nullptr) return;
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        const int ch = threadIdx.x + k * 256;
        if (ch < nvec) {
#pragma unroll
            for (int i = 0; i < VN; ++i) dg_part[(size_t)blockIdx.x * d + ch * VN + i] = dg[k][i];
        }
    }
}

// out[i] = sum over the partial rows, in a fixed order: a CTA owns 32 columns, its 8 warps take the partial rows
// w, w + 8, ... (lane = column), and the 8 warp sums are added in warp order.
__global__ void __launch_bounds__(256) colsum_kernel(const float* __restrict__ part, int nparts, int d, float* __restrict__ out) {
    __shared__ float s[8][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * 32 + lane;
    float t = 0.f;
    if (i < d)
        for (int p = warp; p < nparts; p += 8) t += part[(size_t)p * d + i];
    s[warp][lane] = t;
    __syncthreads();
    if (warp == 0 && i < d) {
        float r = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) r += s[w][lane];
        out[i] = r;
    }
}

// d embed[token[row]] += dx[row]   (fp32 atomics: the order of the additions is not fixed)
template <typename T>
__global__ void __launch_bounds__(256) embed_grad_kernel(const int32_t* __restrict__ tokens, const T* __restrict__ dx, int rows, int d,
                                                        float* __restrict__ dembed) {
    const int row = blockIdx.x;
    if (row >= rows) return;
    const int t = tokens[row];
    for (int i = threadIdx.x; i < d; i += blockDim.x) atomicAdd(dembed + (size_t)t * d + i, to_float<T>(dx[(size_t)row * d + i]));
}

// ------------------------------------------------------------------------------------------------
// Attention backward, CUDA cores.  With w_j = softmax_j(q.k_j / sqrt(dh)) over the visible keys,
// dP_j = do . v_j, delta = sum_j w_j dP_j, dS_j = w_j (dP_j - delta):
//   dq = sum_j dS_j k_j / sqrt(dh);   dk_j += dS_j q / sqrt(dh);   dv_j += w_j do.
// Query side: one warp per (sequence, query head, position); two passes over the visible keys (the
// first gives the row's max, exp-sum and delta; the second dq).  lse and delta go to [B*S, Hq]
// buffers for the key side.
// ------------------------------------------------------------------------------------------------
template <typename T, int DPL>
__global__ void __launch_bounds__(128) attn_block_bwd_q_kernel(const T* __restrict__ Q, const T* __restrict__ Kt, const T* __restrict__ Vt,
                                                              const T* __restrict__ Kp, const T* __restrict__ Vp, const T* __restrict__ dO,
                                                              int S, int Hq, int Hkv, int block, int offset, int step, float scale,
                                                              T* __restrict__ dQ, float* __restrict__ lse, float* __restrict__ delta) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int p0 = blockIdx.x * 4 + warp;
    const int h = blockIdx.y, b = blockIdx.z;
    if (p0 >= S) return;
    const int p = p0 + 1;
    const int n = (p <= offset) ? p - 1 : offset + block * ((p - 1 - offset) / block);
    const int extra = min(p - n, step) - 1;
    const int total = n + extra;
    const int G = Hq / Hkv, kvh = h / G;
    constexpr int DH = DPL * 32;
    const size_t qrow = ((size_t)b * S + p0) * Hq * DH + (size_t)h * DH;
    const size_t ld = (size_t)Hkv * DH;
    const size_t kbase = (size_t)b * S * ld + (size_t)kvh * DH;
    float qf[DPL], dof[DPL], acc[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) {
        qf[i] = to_float<T>(Q[qrow + lane * DPL + i]) * scale;
        dof[i] = to_float<T>(dO[qrow + lane * DPL + i]);
        acc[i] = 0.f;
    }
    float m = -INFINITY, l = 0.f, wd = 0.f;          // running max, exp-sum, sum exp * dP
    for (int j = 0; j < total; ++j) {
        const T* kr = (j < n ? Kt : Kp) + kbase + (size_t)j * ld + lane * DPL;
        const T* vr = (j < n ? Vt : Vp) + kbase + (size_t)j * ld + lane * DPL;
        float s = 0.f, dp = 0.f;
#pragma unroll
        for (int i = 0; i < DPL; ++i) { s = fmaf(qf[i], to_float<T>(kr[i]), s); dp = fmaf(dof[i], to_float<T>(vr[i]), dp); }
        s = warp_sum(s); dp = warp_sum(dp);
        const float mn = fmaxf(m, s);
        const float r = __expf(m - mn), e = __expf(s - mn);
        l = l * r + e;
        wd = wd * r + e * dp;
        m = mn;
    }
    const float inv = total > 0 ? 1.0f / l : 0.f;
    const float dl = wd * inv;
    for (int j = 0; j < total; ++j) {
        const T* kr = (j < n ? Kt : Kp) + kbase + (size_t)j * ld + lane * DPL;
        const T* vr = (j < n ? Vt : Vp) + kbase + (size_t)j * ld + lane * DPL;
        float kf[DPL];
        float s = 0.f, dp = 0.f;
#pragma unroll
        for (int i = 0; i < DPL; ++i) {
            kf[i] = to_float<T>(kr[i]);
            s = fmaf(qf[i], kf[i], s);
            dp = fmaf(dof[i], to_float<T>(vr[i]), dp);
        }
        s = warp_sum(s); dp = warp_sum(dp);
        const float ds = __expf(s - m) * inv * (dp - dl);
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[i] = fmaf(ds, kf[i], acc[i]);
    }
#pragma unroll
    for (int i = 0; i < DPL; ++i) dQ[qrow + lane * DPL + i] = from_float<T>(acc[i] * scale);
    if (lane == 0) {
        const size_t at = ((size_t)b * S + p0) * Hq + h;
        lse[at] = total > 0 ? m + __logf(l) : 0.f;
        delta[at] = dl;
    }
}

// Key side: one warp per (sequence, K/V head, key row, true | predicted); it walks the queries that
// read this key (all G query heads of the group) in ascending order, so dk and dv are summed in a
// fixed order.  A true key at 0-based row j is read by the positions p with n(p) > j; a predicted key
// at row j (window slot r = j + 1 - n(j + 1)) by the later slots of its own window when r < step.
template <typename T, int DPL>
__global__ void __launch_bounds__(128) attn_block_bwd_kv_kernel(const T* __restrict__ Q, const T* __restrict__ Kt, const T* __restrict__ Vt,
                                                               const T* __restrict__ Kp, const T* __restrict__ Vp, const T* __restrict__ dO,
                                                               const float* __restrict__ lse, const float* __restrict__ delta, int S, int Hq,
                                                               int Hkv, int block, int offset, int step, float scale, T* __restrict__ dKt,
                                                               T* __restrict__ dVt, T* __restrict__ dKp, T* __restrict__ dVp, int nz) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = blockIdx.x * 4 + warp;
    const int kvh = blockIdx.y, b = blockIdx.z / nz, pred = blockIdx.z % nz;    // nz = 2 when predicted keys exist (step > 1)
    if (j >= S) return;
    constexpr int DH = DPL * 32;
    const int G = Hq / Hkv;
    const size_t ld = (size_t)Hkv * DH;
    const size_t krow = ((size_t)b * S + j) * ld + (size_t)kvh * DH + lane * DPL;
    float kf[DPL], vf[DPL], dk[DPL], dv[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) {
        kf[i] = to_float<T>((pred ? Kp : Kt)[krow + i]);
        vf[i] = to_float<T>((pred ? Vp : Vt)[krow + i]);
        dk[i] = 0.f; dv[i] = 0.f;
    }
    int p_lo, p_hi;                                   // 1-based query positions [p_lo, p_hi] to test
    if (!pred) { p_lo = j + 2; p_hi = S; }
    else {
        const int pj = j + 1;
        const int nj = (pj <= offset) ? pj - 1 : offset + block * ((pj - 1 - offset) / block);
        const int r = pj - nj;
        if (pj <= offset || r >= step) { p_lo = 1; p_hi = 0; }
        else { p_lo = pj + 1; p_hi = min(S, nj + block); }
    }
    for (int p = p_lo; p <= p_hi; ++p) {
        const int n = (p <= offset) ? p - 1 : offset + block * ((p - 1 - offset) / block);
        if (!pred && n <= j) continue;
        for (int g = 0; g < G; ++g) {
            const int h = kvh * G + g;
            const size_t qrow = ((size_t)b * S + (p - 1)) * Hq * DH + (size_t)h * DH + lane * DPL;
            float qf[DPL], dof[DPL];
            float s = 0.f, dp = 0.f;
#pragma unroll
            for (int i = 0; i < DPL; ++i) {
                qf[i] = to_float<T>(Q[qrow + i]);
                dof[i] = to_float<T>(dO[qrow + i]);
                s = fmaf(qf[i], kf[i], s);
                dp = fmaf(dof[i], vf[i], dp);
            }
            s = warp_sum(s) * scale; dp = warp_sum(dp);
            const size_t at = ((size_t)b * S + (p - 1)) * Hq + h;
            const float w = __expf(s - lse[at]);
            const float ds = w * (dp - delta[at]) * scale;
#pragma unroll
            for (int i = 0; i < DPL; ++i) { dk[i] = fmaf(ds, qf[i], dk[i]); dv[i] = fmaf(w, dof[i], dv[i]); }
        }
    }
#pragma unroll
    for (int i = 0; i < DPL; ++i) {
        (pred ? dKp : dKt)[krow + i] = from_float<T>(dk[i]);
        (pred ? dVp : dVt)[krow + i] = from_float<T>(dv[i]);
    }
}

inline int ew_blocks(size_t n) {      // n elements, eight (four) per thread
    const size_t b = (n / 4 + 255) / 256 + 1;
    return (int)(b < 148 * 16 ? b : 148 * 16);
}

}  // namespace

int launch_transpose_pad_batched(int dtype, const void* in, int rows, int cols, int ld_in, size_t in_batch_stride, void* out, int ld_out, int col0,
                                 int col_batch_stride, int rows_pad, int nbatch, cudaStream_t stream) {
    if (rows_pad <= 0 || cols <= 0 || nbatch <= 0) return 0;
    if (dtype != 0 && !(ld_in & 7) && !(ld_out & 7) && !(col0 & 7) && !(rows_pad & 7) && !(in_batch_stride & 7) && !(col_batch_stride & 7) &&
        !(reinterpret_cast<uintptr_t>(in) & 15) && !(reinterpret_cast<uintptr_t>(out) & 15)) {
        dim3 grid64((rows_pad + 63) / 64, (cols + 63) / 64, nbatch);
        transpose_pad_bf16_kernel<<<grid64, 256, 0, stream>>>((const bf16*)in, rows, cols, ld_in, (bf16*)out, ld_out, col0, rows_pad, in_batch_stride,
                                                              col_batch_stride);
        return 1;
    }
    dim3 grid((rows_pad + 31) / 32, (cols + 31) / 32, nbatch);
    if (dtype == 0)
        transpose_pad_kernel<float><<<grid, 256, 0, stream>>>((const float*)in, rows, cols, ld_in, (float*)out, ld_out, col0, rows_pad, in_batch_stride,
                                                              col_batch_stride);
    else
        transpose_pad_kernel<bf16><<<grid, 256, 0, stream>>>((const bf16*)in, rows, cols, ld_in, (bf16*)out, ld_out, col0, rows_pad, in_batch_stride,
                                                             col_batch_stride);
    return 1;
}

int launch_transpose_pad(int dtype, const void* in, int rows, int cols, int ld_in, void* out, int ld_out, int col0, int rows_pad,
                         cudaStream_t stream) {
    return launch_transpose_pad_batched(dtype, in, rows, cols, ld_in, 0, out, ld_out, col0, 0, rows_pad, 1, stream);
}

int launch_silu_mul(int dtype, const void* gate, const void* up, void* act, size_t n, cudaStream_t stream) {
    if (n == 0) return 0;
    if (dtype == 0) silu_mul_kernel<float><<<ew_blocks(n), 256, 0, stream>>>((const float*)gate, (const float*)up, (float*)act, n);
    else silu_mul_kernel<bf16><<<ew_blocks(n), 256, 0, stream>>>((const bf16*)gate, (const bf16*)up, (bf16*)act, n);
    return 1;
}

int launch_silu_mul_bwd(int dtype, void* gate, void* up, const void* dact, size_t n, cudaStream_t stream) {
    if (n == 0) return 0;
    if (dtype == 0) silu_mul_bwd_kernel<float><<<ew_blocks(n), 256, 0, stream>>>((float*)gate, (float*)up, (const float*)dact, n);
    else silu_mul_bwd_kernel<bf16><<<ew_blocks(n), 256, 0, stream>>>((bf16*)gate, (bf16*)up, (const bf16*)dact, n);
    return 1;
}

int launch_dlogits(int dtype, const float* logits, int rows, int V, const void* tgt, int tgt_dtype, const int32_t* labels, const float* stats,
                   int row0, int S, int block, int offset, int sim_steps, int stage, float scale, void* dz, int ldz, cudaStream_t stream) {
    if (rows <= 0) return 0;
    const float4* st = reinterpret_cast<const float4*>(stats);
#define BEAGLE_DL(T, TT)                                                                                                      \
    dlogits_kernel<T, TT><<<rows, 256, 0, stream>>>(logits, V, (const TT*)tgt, labels, st, row0, S, block, offset, sim_steps, \
                                                    stage, scale, (T*)dz, ldz)
    if (dtype == 0) { if (tgt_dtype == 1) BEAGLE_DL(float, bf16); else BEAGLE_DL(float, float); }
    else { if (tgt_dtype == 1) BEAGLE_DL(bf16, bf16); else BEAGLE_DL(bf16, float); }
#undef BEAGLE_DL
    return 1;
}

int launch_loss_coef(int rows, int S, int block, int offset, int sim_steps, int stage, float scale, float* coef, cudaStream_t stream) {
    if (rows <= 0) return 0;
    loss_coef_kernel<<<(rows + 255) / 256, 256, 0, stream>>>(rows, S, block, offset, sim_steps, stage, scale, coef);
    return 1;
}

int launch_vloss(int dtype, const void* h, const void* h_true, int rows, int d, int S, int block, int offset, int sim_steps, int stage,
                 float grad_coef, float vscale, float vcoef, void* dh0, float* row_sum, float* loss3, cudaStream_t stream) {
    if (rows <= 0) return 0;
    if (dtype == 0)
        vloss_kernel<float><<<rows, 256, 0, stream>>>((const float*)h, (const float*)h_true, d, S, block, offset, sim_steps, stage, grad_coef,
                                                      (float*)dh0, row_sum);
    else
        vloss_kernel<bf16><<<rows, 256, 0, stream>>>((const bf16*)h, (const bf16*)h_true, d, S, block, offset, sim_steps, stage, grad_coef,
                                                     (bf16*)dh0, row_sum);
    loss_total_kernel<<<1, 1024, 0, stream>>>(row_sum, rows, vscale, vcoef, loss3);
    return 2;
}

int rmsnorm_bwd_parts(int rows) { return rows < 148 * 8 ? rows : 148 * 8; }

int launch_rmsnorm_bwd(int dtype, const void* v, const void* gain, const void* dn, const void* add, int rows, int d, float eps, int do_norm,
                       void* out, float* dg_part, float* dg_out, cudaStream_t stream) {
    if (rows <= 0) return 0;
    const int vn = dtype == 0 ? 4 : 8;
    if (d % vn || d / vn > kRmsVec * 256) return -1;
    const int nv = (d / vn + 255) / 256;            // 16-byte pieces per thread
    const int parts = rmsnorm_bwd_parts(rows);
    float* part = (do_norm && dg_out != nullptr) ? dg_part : nullptr;
#define BEAGLE_RMS(T, NV)                                                                                                              \
    rmsnorm_bwd_kernel<T, NV><<<parts, 256, 0, stream>>>((const T*)v, (const T*)gain, (const T*)dn, (const T*)add, rows, d, eps, do_norm, \
                                                         (T*)out, part)
    if (dtype == 0) { if (nv <= 1) BEAGLE_RMS(float, 1); else if (nv == 2) BEAGLE_RMS(float, 2); else BEAGLE_RMS(float, 4); }
    else { if (nv <= 1) BEAGLE_RMS(bf16, 1); else if (nv == 2) BEAGLE_RMS(bf16, 2); else BEAGLE_RMS(bf16, 4); }
#undef BEAGLE_RMS
    int n = 1;
    if (dg_out != nullptr) {
        if (do_norm) { colsum_kernel<<<(d + 31) / 32, 256, 0, stream>>>(dg_part, parts, d, dg_out); ++n; }
        else cudaMemsetAsync(dg_out, 0, (size_t)d * sizeof(float), stream);
    }
    return n;
}

int launch_embed_grad(int dtype, const int32_t* tokens, const void* dx, int rows, int d, float* dembed, cudaStream_t stream) {
    if (rows <= 0) return 0;
    if (dtype == 0) embed_grad_kernel<float><<<rows, 256, 0, stream>>>(tokens, (const float*)dx, rows, d, dembed);
    else embed_grad_kernel<bf16><<<rows, 256, 0, stream>>>(tokens, (const bf16*)dx, rows, d, dembed);
    return 1;
}

template <typename T>
static int attn_block_bwd_dispatch(const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp, const void* dO, int B, int S,
                                   int Hq, int Hkv, int dh, int block, int offset, int step, void* dQ, void* dKt, void* dVt, void* dKp,
                                   void* dVp, float* lse, float* delta, cudaStream_t stream) {
    const float scale = 1.0f / sqrtf((float)dh);
    dim3 gq((S + 3) / 4, Hq, B), gk((S + 3) / 4, Hkv, B * (step > 1 ? 2 : 1));
#define BEAGLE_ABW(DPL)                                                                                                                   \
    do {                                                                                                                                  \
        attn_block_bwd_q_kernel<T, DPL><<<gq, 128, 0, stream>>>((const T*)Q, (const T*)Kt, (const T*)Vt, (const T*)Kp, (const T*)Vp,      \
                                                                (const T*)dO, S, Hq, Hkv, block, offset, step, scale, (T*)dQ, lse, delta); \
        attn_block_bwd_kv_kernel<T, DPL><<<gk, 128, 0, stream>>>((const T*)Q, (const T*)Kt, (const T*)Vt, (const T*)Kp, (const T*)Vp,     \
                                                                 (const T*)dO, lse, delta, S, Hq, Hkv, block, offset, step, scale,        \
                                                                 (T*)dKt, (T*)dVt, (T*)dKp, (T*)dVp, step > 1 ? 2 : 1);                   \
    } while (0)
    switch (dh) {
        case 32: BEAGLE_ABW(1); break;
        case 64: BEAGLE_ABW(2); break;
        case 128: BEAGLE_ABW(4); break;
        case 256: BEAGLE_ABW(8); break;
        default: return -1;
    }
#undef BEAGLE_ABW
    return 2;
}

int launch_attn_block_bwd(int dtype, const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp, const void* dO, int B, int S,
                          int Hq, int Hkv, int dh, int block, int offset, int step, void* dQ, void* dKt, void* dVt, void* dKp, void* dVp,
                          float* lse, float* delta, cudaStream_t stream) {
    if (B <= 0 || S <= 0) return 0;
    return dtype == 0 ? attn_block_bwd_dispatch<float>(Q, Kt, Vt, Kp, Vp, dO, B, S, Hq, Hkv, dh, block, offset, step, dQ, dKt, dVt, dKp, dVp, lse,
                                                       delta, stream)
                      : attn_block_bwd_dispatch<bf16>(Q, Kt, Vt, Kp, Vp, dO, B, S, Hq, Hkv, dh, block, offset, step, dQ, dKt, dVt, dKp, dVp, lse,
                                                      delta, stream);
}

}  // namespace beagle
