// Warp-level merge of split-KV attention partials, shared by the decode-attention kernels.
#pragma once
#include "common.cuh"

namespace beagle {

// One warp merges the `nch` chunk partials of one (sequence, query head): the lanes first share the
// chunks' running maxima and exp-sums (each lane a strided subset), then each lane owns DPL
// consecutive output dims and adds the chunks' unnormalised partials with the weights
// exp(m_i - M), handed around by shuffles.  part_o: [nch][dh], part_ml: [nch][2] of this head.
// dh = DPL * 32, or 16 with DPL = 1 (upper half-warp idle).  SAME_KERNEL: the partials were
// written by other CTAs of the running kernel, so they are read through L2 (ld.global.cg), never L1.
template <bool SAME_KERNEL, typename V>
__device__ __forceinline__ V ld_partial(const V* p) { return SAME_KERNEL ? __ldcg(p) : *p; }

// Merge of chunks [i_begin, i_end): running maximum M, exp-sum den and unnormalised acc (this
// lane's DPL dims), all relative to M.
template <int DPL, bool SAME_KERNEL>
__device__ __forceinline__ void attn_combine_range(const float* part_o, const float* part_ml, int i_begin, int i_end, int dh, int lane,
                                                   float& M, float& den, float* acc) {
    const bool act = lane * DPL < dh;
    M = -INFINITY;
    for (int i = i_begin + lane; i < i_end; i += 32) M = fmaxf(M, ld_partial<SAME_KERNEL>(part_ml + 2 * i));
    M = warp_max(M);
#pragma unroll
    for (int v = 0; v < DPL; ++v) acc[v] = 0.f;
    den = 0.f;
    for (int i0 = i_begin; i0 < i_end; i0 += 32) {
        const int i = i0 + lane;
        float w = 0.f, l = 0.f;
        if (i < i_end) {
            const float2 ml = ld_partial<SAME_KERNEL>(reinterpret_cast<const float2*>(part_ml + 2 * i));
            w = (ml.x == -INFINITY) ? 0.f : __expf(ml.x - M);
            l = ml.y;
        }
        den = fmaf(w, l, den);
        const int n_here = min(32, i_end - i0);
#pragma unroll 4
        for (int j = 0; j < n_here; ++j) {
            const float wj = __shfl_sync(0xffffffffu, w, j);
            const float* src = part_o + (size_t)(i0 + j) * dh + lane * DPL;
            if (!act) continue;
            if constexpr (DPL % 4 == 0) {
#pragma unroll
                for (int v = 0; v < DPL; v += 4) {
                    const float4 t = ld_partial<SAME_KERNEL>(reinterpret_cast<const float4*>(src + v));
                    acc[v] = fmaf(wj, t.x, acc[v]); acc[v + 1] = fmaf(wj, t.y, acc[v + 1]);
                    acc[v + 2] = fmaf(wj, t.z, acc[v + 2]); acc[v + 3] = fmaf(wj, t.w, acc[v + 3]);
                }
            } else {
#pragma unroll
                for (int v = 0; v < DPL; ++v) acc[v] = fmaf(wj, ld_partial<SAME_KERNEL>(src + v), acc[v]);
            }
        }
    }
    den = warp_sum(den);
}

template <typename T, int DPL, bool SAME_KERNEL>
__device__ __forceinline__ void attn_combine_warp(const float* part_o, const float* part_ml, int nch, int dh, int lane, T* o) {
    float M, den, acc[DPL];
    attn_combine_range<DPL, SAME_KERNEL>(part_o, part_ml, 0, nch, dh, lane, M, den, acc);
    const float inv = (nch > 0 && den > 0.f) ? 1.0f / den : 0.f;
    if (lane * DPL < dh) {
#pragma unroll
        for (int v = 0; v < DPL; ++v) o[lane * DPL + v] = from_float<T>(acc[v] * inv);
    }
}

}  // namespace beagle
