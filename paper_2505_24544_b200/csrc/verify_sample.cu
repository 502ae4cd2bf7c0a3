// Draft/verify acceptance under sampling (Section 3): draft i is accepted with probability
// min(1, p_i(t_i) / q_i(t_i)); at the first rejection j (or j = gamma + 1) one token is drawn from the
// normalised max(0, p_j - q_j) (from p_{gamma+1} when nothing was rejected).  p = softmax(target / T),
// q = softmax(draft / T).  The uniforms are inputs, so the kernels are deterministic.
//
// Four HBM-bound passes:
//   1. log-sum-exp of every logit row, rows split 16 ways (the only pass that reads all logits);
//   2. per sequence: acceptance tests, accept_len, the accepted drafts, and the row j to resample at;
//   3. per sequence: the residual mass of row j in 64 chunks (fixed summation order);
//   4. per sequence: inverse CDF -- locate the chunk, then a warp scan inside it.
#include "kernels.h"

namespace beagle {

namespace {

constexpr int kLseSplit = 16;
constexpr int kChunks = 64;

struct VsScratch {
    float2* lse_p;        // [B*(gamma+1)][kLseSplit]  (max, sum exp) of the target rows
    float2* lse_q;        // [gamma*B][kLseSplit]       of the draft rows
    float* row_lse;       // [B][2]: log-sum-exp of p_j and q_j (q: -inf when there is no draft row)
    float* chunk_w;       // [B][kChunks] residual mass per chunk
    float* chunk_p;       // [B][kChunks] target mass per chunk (fallback when no residual mass is left)
};

// One launch covers the target rows (type T, blockIdx.y < rows_p) and the draft rows (fp32).
template <typename T, typename U>
__device__ __forceinline__ void lse_scan_row(const U* __restrict__ z, int V, int split, int nsplit, float inv_t, bool base_aligned,
                                             size_t row_elems, float& m, float& s) {
    constexpr int VEC = VecOf<U>::N;
    int per = (V + nsplit - 1) / nsplit;
    per = (per + VEC - 1) / VEC * VEC;
    const int lo = split * per, hi = min(V, lo + per);
    auto add = [&](float v) {
        v *= inv_t;
        if (v == -INFINITY) return;                               // a masked entry carries no mass
        if (v > m) { s = s * __expf(m - v) + 1.f; m = v; }      // m = -inf: s = 0 * exp(-inf) + 1
        else s += __expf(v - m);
    };
    if (base_aligned && row_elems % VEC == 0) {
        int i = lo + threadIdx.x * VEC;
        const int stride = blockDim.x * VEC;
        for (; i + 3 * stride + VEC <= hi; i += 4 * stride) {          // four independent 16-byte loads in flight per thread
            uint4 u[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) u[j] = ld_stream16(z + i + j * stride);
            float f[4][VEC];
            float vm = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                unpack16<U>(u[j], f[j]);
#pragma unroll
                for (int v = 0; v < VEC; ++v) vm = fmaxf(vm, f[j][v]);
            }
            vm *= inv_t;
            if (vm > m) { s *= __expf(m - vm); m = vm; }           // one rescale per 64 bytes; m = -inf: s stays 0
            if (m != -INFINITY) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int v = 0; v < VEC; ++v) s += __expf(f[j][v] * inv_t - m);
            }
        }
        for (; i < hi; i += stride) {
            if (i + VEC <= hi) {
                float f[VEC];
                unpack16<U>(ld_stream16(z + i), f);
                float vm = f[0];
#pragma unroll
                for (int v = 1; v < VEC; ++v) vm = fmaxf(vm, f[v]);
                vm *= inv_t;
                if (vm > m) { s *= __expf(m - vm); m = vm; }       // one rescale per 16 bytes; m = -inf: s stays 0
                if (m != -INFINITY) {
#pragma unroll
                    for (int v = 0; v < VEC; ++v) s += __expf(f[v] * inv_t - m);
                }
            } else {
                for (int v = i; v < hi; ++v) add(to_float<U>(z[v]));
            }
        }
    } else {
        for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) add(to_float<U>(z[i]));
    }
}

template <typename T>
__global__ void __launch_bounds__(256) vs_lse_partial_kernel(const T* __restrict__ zp, int rows_p, const float* __restrict__ zq, int V,
                                                            float inv_t, float2* __restrict__ part_p, float2* __restrict__ part_q) {
    // gridDim.x <= kLseSplit slices per row: the grid is sized to about one resident wave (every further CTA costs more in
    // launch, first-load latency and reduction than its shorter slice saves); the unused partial slots are filled with "no mass"
    const int split = blockIdx.x, nsplit = gridDim.x;
    int row = blockIdx.y;
    float m = -INFINITY, s = 0.f;
    float2* part;
    if (row < rows_p) {
        lse_scan_row<T, T>(zp + (size_t)row * V, V, split, nsplit, inv_t, (reinterpret_cast<uintptr_t>(zp) & 15) == 0, (size_t)row * V, m, s);
        part = part_p;
    } else {
        row -= rows_p;
        lse_scan_row<T, float>(zq + (size_t)row * V, V, split, nsplit, inv_t, (reinterpret_cast<uintptr_t>(zq) & 15) == 0, (size_t)row * V, m, s);
        part = part_q;
    }
    // merge (m, s) pairs: warp, then CTA, always in the same order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
        const float M = fmaxf(m, m2);
        s = (M == -INFINITY) ? 0.f : s * __expf(m - M) + s2 * __expf(m2 - M);
        m = M;
    }
    __shared__ float sm[8], ss[8];
    if ((threadIdx.x & 31) == 0) { sm[threadIdx.x >> 5] = m; ss[threadIdx.x >> 5] = s; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float M = sm[0], S = ss[0];
        for (int w = 1; w < 8; ++w) {
            const float M2 = fmaxf(M, sm[w]);
            S = (M2 == -INFINITY) ? 0.f : S * __expf(M - M2) + ss[w] * __expf(sm[w] - M2);
            M = M2;
        }
        part[(size_t)row * kLseSplit + split] = make_float2(M, S);
        if (split == 0)
            for (int e = nsplit; e < kLseSplit; ++e) part[(size_t)row * kLseSplit + e] = make_float2(-INFINITY, 0.f);
    }
}

__device__ __forceinline__ float lse_of(const float2* part) {
    float M = -INFINITY;
    for (int i = 0; i < kLseSplit; ++i) M = fmaxf(M, part[i].x);
    float S = 0.f;
    for (int i = 0; i < kLseSplit; ++i) S += (part[i].x == -INFINITY) ? 0.f : part[i].y * __expf(part[i].x - M);
    return M + __logf(S);
}

// One warp per sequence: lane i evaluates the acceptance test of position i (all positions at once,
// in rounds of 32), the first failing position is the accepted length.
template <typename T>
__global__ void __launch_bounds__(128) vs_accept_kernel(const int32_t* __restrict__ draft, const float* __restrict__ zq, const T* __restrict__ zp,
                                                        int B, int gamma, int V, float inv_t, const float* __restrict__ u_accept, VsScratch sc,
                                                        int32_t* __restrict__ accept_len, int32_t* __restrict__ out_tokens) {
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (b >= B) return;
    int a = gamma;
    for (int i0 = 0; i0 < gamma && a == gamma; i0 += 32) {
        const int i = i0 + lane;
        bool pass = true;
        if (i < gamma) {
            const int t = min(max(draft[(size_t)b * gamma + i], 0), V - 1);
            const float lp = to_float<T>(zp[((size_t)b * (gamma + 1) + i) * V + t]) * inv_t - lse_of(sc.lse_p + ((size_t)b * (gamma + 1) + i) * kLseSplit);
            const float lq = zq[((size_t)i * B + b) * V + t] * inv_t - lse_of(sc.lse_q + ((size_t)i * B + b) * kLseSplit);
            const float ratio = fminf(1.f, __expf(lp - lq));
            pass = u_accept[(size_t)b * gamma + i] < ratio;
        }
        const unsigned fail = ~__ballot_sync(0xffffffffu, pass);
        if (fail) a = i0 + __ffs(fail) - 1;
    }
    for (int r = lane; r <= gamma; r += 32) out_tokens[(size_t)b * (gamma + 1) + r] = r < a ? draft[(size_t)b * gamma + r] : -1;
    if (lane == 0) {
        accept_len[b] = a;
        sc.row_lse[2 * b] = lse_of(sc.lse_p + ((size_t)b * (gamma + 1) + a) * kLseSplit);
        sc.row_lse[2 * b + 1] = a < gamma ? lse_of(sc.lse_q + ((size_t)a * B + b) * kLseSplit) : INFINITY;   // unused: no draft row
    }
}

// Residual weight of vocabulary entry v of the row to resample at.
template <typename T>
__device__ __forceinline__ void residual_at(const T* zp, const float* zq, int v, float inv_t, float lse_p, float lse_q, float& w, float& p) {
    p = __expf(to_float<T>(zp[v]) * inv_t - lse_p);
    const float q = (zq != nullptr) ? __expf(zq[v] * inv_t - lse_q) : 0.f;
    w = fmaxf(0.f, p - q);
}

template <typename T>
__global__ void __launch_bounds__(256) vs_residual_kernel(const float* __restrict__ zq_all, const T* __restrict__ zp_all, int B, int gamma, int V,
                                                         float inv_t, const int32_t* __restrict__ accept_len, VsScratch sc) {
    const int c = blockIdx.x, b = blockIdx.y;
    const int a = accept_len[b];
    const T* zp = zp_all + ((size_t)b * (gamma + 1) + a) * V;
    const float* zq = a < gamma ? zq_all + ((size_t)a * B + b) * V : nullptr;
    const float lse_p = sc.row_lse[2 * b], lse_q = sc.row_lse[2 * b + 1];
    const int per = (V + kChunks - 1) / kChunks;
    const int lo = c * per, hi = min(V, lo + per);
    float sw = 0.f, sp = 0.f;
    for (int v = lo + threadIdx.x; v < hi; v += blockDim.x) {
        float w, p;
        residual_at<T>(zp, zq, v, inv_t, lse_p, lse_q, w, p);
        sw += w;
        sp += p;
    }
    sw = warp_sum(sw);
    sp = warp_sum(sp);
    __shared__ float s_w[8], s_p[8];
    if ((threadIdx.x & 31) == 0) { s_w[threadIdx.x >> 5] = sw; s_p[threadIdx.x >> 5] = sp; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float tw = 0.f, tp = 0.f;
        for (int w = 0; w < 8; ++w) { tw += s_w[w]; tp += s_p[w]; }
        sc.chunk_w[(size_t)b * kChunks + c] = tw;
        sc.chunk_p[(size_t)b * kChunks + c] = tp;
    }
}

constexpr int kPickThreads = 256;
constexpr int kPickSeg = 16;          // entries per thread and pass

template <typename T>
__global__ void __launch_bounds__(kPickThreads) vs_pick_kernel(const float* __restrict__ zq_all, const T* __restrict__ zp_all, int B, int gamma,
                                                              int V, float inv_t, const float* __restrict__ u_resample,
                                                              const int32_t* __restrict__ accept_len, VsScratch sc,
                                                              int32_t* __restrict__ out_tokens) {
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int a = accept_len[b];
    const T* zp = zp_all + ((size_t)b * (gamma + 1) + a) * V;
    const float* zq = a < gamma ? zq_all + ((size_t)a * B + b) * V : nullptr;
    const float lse_p = sc.row_lse[2 * b], lse_q = sc.row_lse[2 * b + 1];
    __shared__ float s_cw[kChunks], s_warp[kPickThreads / 32];
    __shared__ int s_chunk, s_use_p, s_pick, s_last;
    __shared__ float s_before, s_target;
    if (tid < kChunks) s_cw[tid] = sc.chunk_w[(size_t)b * kChunks + tid];
    if (tid == 0) { s_pick = 0x7fffffff; s_last = -1; }
    __syncthreads();
    if (tid == 0) {
        float total = 0.f;
        for (int c = 0; c < kChunks; ++c) total += s_cw[c];
        s_use_p = !(total > 0.f);                   // no residual mass (p == q): draw from p instead
    }
    __syncthreads();
    const bool use_p = s_use_p != 0;
    if (use_p) {
        __syncthreads();
        if (tid < kChunks) s_cw[tid] = sc.chunk_p[(size_t)b * kChunks + tid];
        __syncthreads();
    }
    if (tid == 0) {
        float total = 0.f;
        for (int c = 0; c < kChunks; ++c) total += s_cw[c];
        const float target = u_resample[b] * total;
        // chunk whose cumulative mass first exceeds the target (the last non-empty chunk if rounding leaves none)
        float before = 0.f;
        int chunk = -1, last_nonempty = 0;
        for (int c = 0; c < kChunks; ++c) {
            if (s_cw[c] > 0.f) last_nonempty = c;
            if (chunk < 0 && before + s_cw[c] > target) chunk = c;
            if (chunk < 0) before += s_cw[c];
        }
        if (chunk < 0) {
            chunk = last_nonempty;
            before = 0.f;
            for (int c = 0; c < chunk; ++c) before += s_cw[c];
        }
        s_chunk = chunk; s_before = before; s_target = target;
    }
    __syncthreads();
    const int per = (V + kChunks - 1) / kChunks;
    const int lo = s_chunk * per, hi = min(V, lo + per);
    const float target = s_target;
    float run = s_before;                           // mass before the current pass, identical in every thread
    for (int p0 = lo; p0 < hi; p0 += kPickThreads * kPickSeg) {
        // this thread's contiguous segment
        const int v0 = p0 + tid * kPickSeg;
        float w[kPickSeg], seg = 0.f;
#pragma unroll
        for (int j = 0; j < kPickSeg; ++j) {
            float wj = 0.f, pj = 0.f;
            if (v0 + j < hi) residual_at<T>(zp, zq, v0 + j, inv_t, lse_p, lse_q, wj, pj);
            w[j] = use_p ? pj : wj;
            seg += w[j];
        }
        // exclusive scan of the segment sums over the CTA
        float inc = seg;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) s_warp[warp] = inc;
        __syncthreads();
        float wbase = 0.f, pass_total = 0.f;
        for (int k = 0; k < kPickThreads / 32; ++k) { if (k < warp) wbase += s_warp[k]; pass_total += s_warp[k]; }
        float c = run + wbase + inc - seg;          // mass before this thread's segment
        int mine = 0x7fffffff, last = -1;
#pragma unroll
        for (int j = 0; j < kPickSeg; ++j) {
            if (v0 + j < hi) {
                c += w[j];
                if (w[j] > 0.f) last = v0 + j;
                if (mine == 0x7fffffff && c > target) mine = v0 + j;
            }
        }
        if (mine != 0x7fffffff) atomicMin(&s_pick, mine);
        if (last >= 0) atomicMax(&s_last, last);
        __syncthreads();
        if (s_pick != 0x7fffffff) break;
        run += pass_total;
        __syncthreads();
    }
    if (tid == 0) {
        int picked = s_pick;
        if (picked == 0x7fffffff) picked = s_last >= 0 ? s_last : lo;   // rounding: the target lies past the last entry with mass
        out_tokens[(size_t)b * (gamma + 1) + a] = picked;
    }
}

VsScratch carve(void* scratch, int B, int gamma) {
    VsScratch s;
    char* p = static_cast<char*>(scratch);
    auto take = [&](size_t bytes) { char* at = p; p += (bytes + 255) / 256 * 256; return at; };
    s.lse_p = reinterpret_cast<float2*>(take((size_t)B * (gamma + 1) * kLseSplit * sizeof(float2)));
    s.lse_q = reinterpret_cast<float2*>(take((size_t)B * (gamma > 0 ? gamma : 1) * kLseSplit * sizeof(float2)));
    s.row_lse = reinterpret_cast<float*>(take((size_t)B * 2 * sizeof(float)));
    s.chunk_w = reinterpret_cast<float*>(take((size_t)B * kChunks * sizeof(float)));
    s.chunk_p = reinterpret_cast<float*>(take((size_t)B * kChunks * sizeof(float)));
    return s;
}

template <typename T>
int run_verify_sample(const int32_t* draft, const float* zq, const T* zp, int B, int gamma, int V, float temperature, const float* u_accept,
                      const float* u_resample, void* scratch, int32_t* accept_len, int32_t* out_tokens, int sm_count, cudaStream_t stream) {
    const VsScratch sc = carve(scratch, B, gamma);
    const float inv_t = 1.0f / temperature;
    const int lse_rows = B * (gamma + 1) + gamma * B;
    static int per_sm = 0;                                        // resident CTAs of this instantiation per SM (same on every B200)
    if (per_sm == 0 && (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, vs_lse_partial_kernel<T>, 256, 0) != cudaSuccess || per_sm < 1)) {
        cudaGetLastError();
        per_sm = 4;
    }
    int nsplit = (per_sm * sm_count) / lse_rows;                  // one resident wave ...
    const int cap = (V + 4095) / 4096;                            // ... of slices no shorter than 4096 logits
    nsplit = nsplit < cap ? nsplit : cap;
    nsplit = nsplit < 1 ? 1 : (nsplit > kLseSplit ? kLseSplit : nsplit);
    vs_lse_partial_kernel<T><<<dim3(nsplit, lse_rows), 256, 0, stream>>>(zp, B * (gamma + 1), zq, V, inv_t, sc.lse_p, sc.lse_q);
    const int n = 1;
    vs_accept_kernel<T><<<(B + 3) / 4, 128, 0, stream>>>(draft, zq, zp, B, gamma, V, inv_t, u_accept, sc, accept_len, out_tokens);
    vs_residual_kernel<T><<<dim3(kChunks, B), 256, 0, stream>>>(zq, zp, B, gamma, V, inv_t, accept_len, sc);
    vs_pick_kernel<T><<<B, kPickThreads, 0, stream>>>(zq, zp, B, gamma, V, inv_t, u_resample, accept_len, sc, out_tokens);
    return n + 3;
}

}  // namespace

size_t verify_sample_scratch_bytes(int max_batch, int max_gamma) {
    const size_t rows_p = (size_t)max_batch * (max_gamma + 1), rows_q = (size_t)max_batch * (max_gamma > 0 ? max_gamma : 1);
    return (rows_p + rows_q) * kLseSplit * sizeof(float2) + (size_t)max_batch * (2 + 2 * kChunks) * sizeof(float) + 5 * 256;
}

int launch_verify_sample(int logits_dtype, const int32_t* draft, const float* draft_logits, const void* target_logits, int B, int gamma, int V,
                         float temperature, const float* u_accept, const float* u_resample, void* scratch, int32_t* accept_len,
                         int32_t* out_tokens, int sm_count, cudaStream_t stream) {
    if (B <= 0) return 0;
    return logits_dtype == 0
        ? run_verify_sample<float>(draft, draft_logits, static_cast<const float*>(target_logits), B, gamma, V, temperature, u_accept,
                                   u_resample, scratch, accept_len, out_tokens, sm_count, stream)
        : run_verify_sample<bf16>(draft, draft_logits, static_cast<const bf16*>(target_logits), B, gamma, V, temperature, u_accept,
                                  u_resample, scratch, accept_len, out_tokens, sm_count, stream);
}

}  // namespace beagle
