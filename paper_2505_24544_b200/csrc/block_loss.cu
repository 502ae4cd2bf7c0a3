// Forward of the block-attention training losses (Eq. 4 early stage, Eq. 7 late stage with l = i and
// beta*_{i,i} = k - i + 1): per position the cross-entropy -E_{t ~ p}[log q(t)] between the target
// distribution p (softmax of target logits, or a label) and the draft distribution q = softmax(z)
// of the block forward, then the weighted mean over window positions.
//
// The LM-head GEMM emits cross-entropy partials per (row, column tile) from its epilogue, so the
// [positions, V] logits are never written; this file merges the partials, applies the weights and
// reduces in a fixed order.  For configurations without the tensor-core GEMM the partials come
// from materialised fp32 logits (row_ce_kernel).
#include "kernels.h"

namespace beagle {

namespace {

struct CePart { float mq, sq, mt, st, dot; };

__device__ __forceinline__ CePart ce_merge(const CePart& a, const CePart& b) {
    CePart r;
    r.mq = fmaxf(a.mq, b.mq);
    r.sq = (r.mq == -INFINITY) ? 0.f : a.sq * __expf(a.mq - r.mq) + b.sq * __expf(b.mq - r.mq);
    r.mt = fmaxf(a.mt, b.mt);
    const float fa = (a.mt == -INFINITY) ? 0.f : __expf(a.mt - r.mt), fb = (b.mt == -INFINITY) ? 0.f : __expf(b.mt - r.mt);
    r.st = a.st * fa + b.st * fb;
    r.dot = a.dot * fa + b.dot * fb;
    return r;
}
__device__ __forceinline__ CePart ce_shfl_xor(const CePart& v, int o) {
    CePart r;
    r.mq = __shfl_xor_sync(0xffffffffu, v.mq, o); r.sq = __shfl_xor_sync(0xffffffffu, v.sq, o);
    r.mt = __shfl_xor_sync(0xffffffffu, v.mt, o); r.st = __shfl_xor_sync(0xffffffffu, v.st, o);
    r.dot = __shfl_xor_sync(0xffffffffu, v.dot, o);
    return r;
}

// One CTA per row of materialised logits: the partial of the whole row.
template <typename T>
__global__ void __launch_bounds__(256) row_ce_kernel(const float* __restrict__ logits, int V, const T* __restrict__ tgt,
                                                    const int32_t* __restrict__ labels, float* __restrict__ ce_part) {
    const int row = blockIdx.x;
    const float* z = logits + (size_t)row * V;
    CePart acc = {-INFINITY, 0.f, tgt != nullptr ? -INFINITY : 0.f, 0.f, 0.f};
    const int label = tgt == nullptr ? labels[row] : -1;
    for (int v = threadIdx.x; v < V; v += blockDim.x) {
        CePart one;
        one.mq = z[v]; one.sq = 1.f;
        if (tgt != nullptr) { one.mt = to_float<T>(tgt[(size_t)row * V + v]); one.st = 1.f; one.dot = z[v]; }
        else { one.mt = 0.f; one.st = v == label ? 1.f : 0.f; one.dot = v == label ? z[v] : 0.f; }
        acc = ce_merge(acc, one);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc = ce_merge(acc, ce_shfl_xor(acc, o));
    __shared__ CePart s_p[8];
    if ((threadIdx.x & 31) == 0) s_p[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        CePart r = s_p[0];
        for (int w = 1; w < 8; ++w) r = ce_merge(r, s_p[w]);
        float* dst = ce_part + (size_t)row * kCeFields;
        dst[0] = r.mq; dst[1] = r.sq; dst[2] = r.mt; dst[3] = r.st; dst[4] = r.dot;
    }
}

// One warp per row: merge the column tiles' partials, ce = lse(z) - E_p[z], weight by the position.
__global__ void __launch_bounds__(256) ce_finalize_kernel(const float* __restrict__ ce_part, int ntiles, int rows, int S, int block, int offset,
                                                         int sim_steps, int stage, float* __restrict__ ce_rows, float* __restrict__ wce,
                                                         float* __restrict__ ce_out, float4* __restrict__ row_stats) {
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (row >= rows) return;
    CePart acc = {-INFINITY, 0.f, -INFINITY, 0.f, 0.f};
    for (int t = lane; t < ntiles; t += 32) {
        const float* p = ce_part + ((size_t)row * ntiles + t) * kCeFields;
        const CePart one = {p[0], p[1], p[2], p[3], p[4]};
        acc = ce_merge(acc, one);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc = ce_merge(acc, ce_shfl_xor(acc, o));
    if (lane == 0) {
        const float ce = acc.mq + __logf(acc.sq) - acc.dot / acc.st;
        const int p = row % S + 1;                                  // 1-based position in its sequence
        float w = 0.f;
        if (p > offset) {
            const int n = offset + block * ((p - 1 - offset) / block);
            const int slot = p - n;
            w = stage == 0 ? 1.f : (slot <= sim_steps ? (float)(block - slot + 1) : 0.f);
        }
        ce_rows[row] = ce;
        wce[row] = w * ce;
        if (ce_out != nullptr) ce_out[row] = ce;
        if (row_stats != nullptr) row_stats[row] = make_float4(acc.mq, acc.sq, acc.mt, acc.st);
    }
}

// Fixed-order sum of wce[0..rows) by one CTA, scaled by 1 / (batch * windows).
__global__ void __launch_bounds__(1024) ce_reduce_kernel(const float* __restrict__ wce, int rows, float scale, float* __restrict__ loss_out) {
    __shared__ float s[1024];
    float t = 0.f;
    for (int i = threadIdx.x; i < rows; i += 1024) t += wce[i];
    s[threadIdx.x] = t;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss_out = s[0] * scale;
}

}  // namespace

int launch_row_ce(const float* logits, int rows, int V, const void* tgt, int tgt_dtype, const int32_t* labels, float* ce_part,
                  cudaStream_t stream) {
    if (rows <= 0) return 0;
    if (tgt_dtype == 1) row_ce_kernel<bf16><<<rows, 256, 0, stream>>>(logits, V, static_cast<const bf16*>(tgt), labels, ce_part);
    else row_ce_kernel<float><<<rows, 256, 0, stream>>>(logits, V, static_cast<const float*>(tgt), labels, ce_part);
    return 1;
}

int launch_ce_finalize(const float* ce_part, int ntiles, int batch, int S, int block, int offset, int sim_steps, int stage,
                       float* ce_rows, float* wce, float* ce_out, float* loss_out, cudaStream_t stream, float* row_stats) {
    const int rows = batch * S;
    if (rows <= 0) return 0;
    ce_finalize_kernel<<<(rows * 32 + 255) / 256, 256, 0, stream>>>(ce_part, ntiles, rows, S, block, offset, sim_steps, stage, ce_rows, wce, ce_out,
                                                                     reinterpret_cast<float4*>(row_stats));
    const int windows = (S - offset + block - 1) / block;
    ce_reduce_kernel<<<1, 1024, 0, stream>>>(wce, rows, 1.0f / ((float)batch * (float)windows), loss_out);
    return 2;
}

}  // namespace beagle
