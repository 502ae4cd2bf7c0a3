// Block-path kernels that run on the CUDA cores: a tiled fp32-accumulate GEMM C = A W^T with fused
// epilogues (the fp32 configuration's GEMM, and the shape-agnostic fallback of the tensor-core
// path), and the block-masked cross-attention of the multi-token forward.
#include "kernels.h"

namespace beagle {

// ------------------------------------------------------------------------------------------------
// SIMT GEMM: 64x64 tile, K step 16, 256 threads, 4x4 outputs per thread.
// ------------------------------------------------------------------------------------------------
constexpr int kTM = 64, kTN = 64, kTK = 16;

template <typename T>
__device__ __forceinline__ void load4(const T* p, bool ok, float* f);
template <>
__device__ __forceinline__ void load4<float>(const float* p, bool ok, float* f) {
    if (ok) { const float4 v = *reinterpret_cast<const float4*>(p); f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
    else { f[0] = f[1] = f[2] = f[3] = 0.f; }
}
template <>
__device__ __forceinline__ void load4<bf16>(const bf16* p, bool ok, float* f) {
    if (ok) {
        const uint2 v = *reinterpret_cast<const uint2*>(p);
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    } else { f[0] = f[1] = f[2] = f[3] = 0.f; }
}

__device__ __forceinline__ int seq_of_row(const SeqRows& rows, int r) {
    int b = 0;
    while (b + 1 < rows.n && r >= rows.row_start[b + 1]) ++b;
    return b;
}

template <typename T, int EPI>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const GemmArgs a) {
    constexpr bool DUAL = (EPI == GEMM_SILU_MUL);
    __shared__ float sA[kTK][kTM + 4];
    __shared__ float sW[kTK][kTN + 4];
    __shared__ float sW2[DUAL ? kTK : 1][kTN + 4];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * kTM, n0 = blockIdx.x * kTN;
    const T* A = reinterpret_cast<const T*>(a.A);
    const T* W = reinterpret_cast<const T*>(a.W);
    const T* W2 = reinterpret_cast<const T*>(a.W2);
    const int lr = tid >> 2;            // tile row 0..63 loaded by this thread
    const int lk = (tid & 3) * 4;       // k offset 0,4,8,12
    const int ty = tid >> 4, tx = tid & 15;   // 16 x 16 threads, 4 x 4 outputs each
    float acc[4][4], acc2[DUAL ? 4 : 1][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; if (DUAL) acc2[i][j] = 0.f; }

    for (int k0 = 0; k0 < a.K; k0 += kTK) {
        float fa[4], fw[4], fw2[4];
        const bool kok = (k0 + lk) < a.K;       // K is a multiple of 4
        load4<T>(A + (size_t)(m0 + lr) * a.lda + k0 + lk, kok && (m0 + lr) < a.M, fa);
        load4<T>(W + (size_t)(n0 + lr) * a.K + k0 + lk, kok && (n0 + lr) < a.N, fw);
        if (DUAL) load4<T>(W2 + (size_t)(n0 + lr) * a.K + k0 + lk, kok && (n0 + lr) < a.N, fw2);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            sA[lk + i][lr] = fa[i];
            sW[lk + i][lr] = fw[i];
            if (DUAL) sW2[lk + i][lr] = fw2[i];
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kTK; ++kk) {
            float ra[4], rw[4], rw2[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) ra[i] = sA[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) { rw[j] = sW[kk][tx * 4 + j]; if (DUAL) rw2[j] = sW2[kk][tx * 4 + j]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc[i][j] = fmaf(ra[i], rw[j], acc[i][j]);
                    if (DUAL) acc2[i][j] = fmaf(ra[i], rw2[j], acc2[i][j]);
                }
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= a.M) continue;
        int slot = 0, pos = 0;
        if (EPI == GEMM_KV_CACHE) {
            const int b = seq_of_row(a.rows, m);
            slot = a.rows.slot[b];
            pos = a.rows.pos_start[b] + (m - a.rows.row_start[b]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= a.N) continue;
            const float v = acc[i][j];
            if (EPI == GEMM_STORE) reinterpret_cast<T*>(a.C)[(size_t)m * a.ldc + n] = from_float<T>(v);
            else if (EPI == GEMM_RESID)
                reinterpret_cast<T*>(a.C)[(size_t)m * a.ldc + n] =
                    from_float<T>(v + to_float<T>(reinterpret_cast<const T*>(a.R)[(size_t)m * a.ldr + n]));
            else if (EPI == GEMM_SILU_MUL) reinterpret_cast<T*>(a.C)[(size_t)m * a.ldc + n] = from_float<T>(silu_f(v) * acc2[i][j]);
            else if (EPI == GEMM_F32) reinterpret_cast<float*>(a.C)[(size_t)m * a.ldc + n] = v;
            else if (EPI == GEMM_KV_CACHE)
                reinterpret_cast<T*>(a.cache)[(((size_t)slot * a.Hkv + n / a.dh) * a.cap + pos) * a.dh + n % a.dh] = from_float<T>(v);
        }
    }
}

template <typename T>
static int gemm_simt_dispatch(int epi, const GemmArgs& a, cudaStream_t stream) {
    dim3 grid((a.N + kTN - 1) / kTN, (a.M + kTM - 1) / kTM);
    switch (epi) {
        case GEMM_STORE: gemm_simt_kernel<T, GEMM_STORE><<<grid, 256, 0, stream>>>(a); break;
        case GEMM_RESID: gemm_simt_kernel<T, GEMM_RESID><<<grid, 256, 0, stream>>>(a); break;
        case GEMM_SILU_MUL: gemm_simt_kernel<T, GEMM_SILU_MUL><<<grid, 256, 0, stream>>>(a); break;
        case GEMM_F32: gemm_simt_kernel<T, GEMM_F32><<<grid, 256, 0, stream>>>(a); break;
        case GEMM_KV_CACHE: gemm_simt_kernel<T, GEMM_KV_CACHE><<<grid, 256, 0, stream>>>(a); break;
        default: return -1;
    }
    return 1;
}
int launch_gemm_simt(int dtype, int epi, const GemmArgs& a, cudaStream_t stream) {
    if (a.M <= 0 || a.N <= 0) return 0;
    if ((a.K & 3) || (a.lda & 3)) return -1;
    return dtype == 0 ? gemm_simt_dispatch<float>(epi, a, stream) : gemm_simt_dispatch<bf16>(epi, a, stream);
}

// ------------------------------------------------------------------------------------------------
// Block-masked cross-attention (Section 4.2): one warp per (sequence, query head, position).
// The four warps of a CTA take four consecutive positions of one head, so they walk the same
// key/value rows.  Visible keys: true rows [0, n) then predicted rows [n, n + extra).
// ------------------------------------------------------------------------------------------------
template <typename T, int DPL>   // DPL = head_dim / 32 elements per lane
__global__ void __launch_bounds__(128) attn_block_kernel(const T* __restrict__ Q, const T* __restrict__ Kt,
                                                         const T* __restrict__ Vt, const T* __restrict__ Kp,
                                                         const T* __restrict__ Vp, int S, int Hq, int Hkv, int block,
                                                         int offset, int step, float scale, T* __restrict__ O) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int p0 = blockIdx.x * 4 + warp;     // 0-based position
    const int h = blockIdx.y, b = blockIdx.z;
    if (p0 >= S) return;
    const int p = p0 + 1;                     // 1-based, as in the paper
    const int n = (p <= offset) ? p - 1 : offset + block * ((p - 1 - offset) / block);
    const int slot = p - n;
    const int extra = min(slot, step) - 1;    // predicted states n+1 .. n+extra
    const int G = Hq / Hkv, kvh = h / G;
    const int DH = DPL * 32;
    const size_t qrow = ((size_t)b * S + p0) * Hq * DH + (size_t)h * DH;
    const size_t ld = (size_t)Hkv * DH;
    const size_t kbase = (size_t)b * S * ld + (size_t)kvh * DH;

    float qf[DPL], acc[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) { qf[i] = to_float<T>(Q[qrow + lane * DPL + i]) * scale; acc[i] = 0.f; }
    float m = -INFINITY, l = 0.f;
    const int total = n + extra;
    for (int j0 = 0; j0 < total; j0 += 4) {
        float s[4], vf[4][DPL];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int j = j0 + u;
            float dot = 0.f;
            if (j < total) {
                const T* kr = (j < n ? Kt : Kp) + kbase + (size_t)j * ld + lane * DPL;
                const T* vr = (j < n ? Vt : Vp) + kbase + (size_t)j * ld + lane * DPL;
#pragma unroll
                for (int i = 0; i < DPL; ++i) { dot = fmaf(qf[i], to_float<T>(kr[i]), dot); vf[u][i] = to_float<T>(vr[i]); }
            } else {
#pragma unroll
                for (int i = 0; i < DPL; ++i) vf[u][i] = 0.f;
            }
            s[u] = dot;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) { s[u] = warp_sum(s[u]); if (j0 + u >= total) s[u] = -INFINITY; }
        const float mn = fmaxf(fmaxf(fmaxf(s[0], s[1]), fmaxf(s[2], s[3])), m);
        const float r = __expf(m - mn);       // m = -inf on the first group: r = 0
        l *= r;
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[i] *= r;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float pw = __expf(s[u] - mn);
            l += pw;
#pragma unroll
            for (int i = 0; i < DPL; ++i) acc[i] = fmaf(pw, vf[u][i], acc[i]);
        }
        m = mn;
    }
    const float inv = total > 0 ? 1.0f / l : 0.f;
#pragma unroll
    for (int i = 0; i < DPL; ++i) O[qrow + lane * DPL + i] = from_float<T>(acc[i] * inv);
}

template <typename T>
static int attn_block_dispatch(const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp, int B, int S,
                               int Hq, int Hkv, int dh, int block, int offset, int step, void* O, cudaStream_t stream) {
    dim3 grid((S + 3) / 4, Hq, B);
    const float scale = 1.0f / sqrtf((float)dh);
#define BEAGLE_AB(DPL)                                                                                             \
    attn_block_kernel<T, DPL><<<grid, 128, 0, stream>>>((const T*)Q, (const T*)Kt, (const T*)Vt, (const T*)Kp,   \
                                                        (const T*)Vp, S, Hq, Hkv, block, offset, step, scale, (T*)O)
    switch (dh) {
        case 32: BEAGLE_AB(1); break;
        case 64: BEAGLE_AB(2); break;
        case 128: BEAGLE_AB(4); break;
        case 256: BEAGLE_AB(8); break;
        default: return -1;
    }
#undef BEAGLE_AB
    return 1;
}
int launch_attn_block(int dtype, const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp,
                      int B, int S, int Hq, int Hkv, int dh, int block, int offset, int step, void* O,
                      cudaStream_t stream) {
    if (B <= 0 || S <= 0) return 0;
    return dtype == 0 ? attn_block_dispatch<float>(Q, Kt, Vt, Kp, Vp, B, S, Hq, Hkv, dh, block, offset, step, O, stream)
                      : attn_block_dispatch<bf16>(Q, Kt, Vt, Kp, Vp, B, S, Hq, Hkv, dh, block, offset, step, O, stream);
}

}  // namespace beagle
