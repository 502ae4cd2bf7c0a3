// Block-masked cross-attention of the multi-token forward (Section 4.2) on the tensor cores.
//
// One CTA = 64 consecutive query positions of one (sequence, query head).  Query p (1-based) reads
// the true keys 1..n(p), n(p) = p-1 before the first window and the start of p's window after it,
// and, at simulation step `step` > 1, the predicted keys n(p)+1 .. n(p)+min(slot, step)-1 of its
// own window.  The mask is arithmetic: key tiles that lie entirely below every n(p) of the CTA are
// processed unmasked, the one or two tiles on the diagonal compare j with n(p) per element, and
// the predicted keys are a second pass over those diagonal tiles with the band mask.
//
// K and V tiles of 64 keys arrive by TMA (128-byte swizzle) in a two-stage ring (64 KB per CTA,
// three CTAs per SM); each of the four
// warps owns 16 queries: S = Q K^T (ldmatrix + mma.sync m16n8k16), online softmax in registers,
// O += P V (ldmatrix.trans).  Attention is about 2.5 % of the block path's flop; the projections
// around it run on tcgen05.
#include <cstring>

#include "gemm_tc.h"
#include "tc_plan.h"
#include "mma_tiles.cuh"
#include "tc_ptx.cuh"

namespace beagle {

namespace {

using namespace tc;
using namespace mma_tiles;

constexpr int kBQ = 64, kBKey = 64, kWarps = 4;

struct BlkArgs {
    int S, Hq, Hkv, block, offset, step;
    float scale_log2;
    bf16* O;            // [B*S, Hq*DH]
    float* lse2;        // optional [B*S, Hq]: base-2 log-sum-exp of the scaled scores of every row (0 for a row without keys)
    int* error_word;
};

template <int DH>
__global__ void __launch_bounds__(kWarps * 32, 3) attn_block_tc_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                                   const __grid_constant__ CUtensorMap tmKt,
                                                                   const __grid_constant__ CUtensorMap tmVt,
                                                                   const __grid_constant__ CUtensorMap tmKp,
                                                                   const __grid_constant__ CUtensorMap tmVp, const BlkArgs a) {
    constexpr int kTile = 64 * DH * 2;          // bytes of one Q / K / V tile
    constexpr int kHalves = DH / 64;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sKV = smem_base;             // stage s: K at sKV + s*2*kTile, V right after it
    const uint32_t sQ = sKV + 2 * kTile;        // the Q tile borrows stage 1's K slot until its fragments are in registers
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + 4 * kTile);
    const uint32_t barQ = smem_u32(bars), barF = barQ + 8;      // barF[2]: tile landed
    __shared__ int s_abort;

    const int qtile = gridDim.x - 1 - blockIdx.x;               // heaviest (latest) query tiles first
    const int h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (a.Hq / a.Hkv);
    const int q0 = qtile * kBQ;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;

    // visible ranges of this thread's two query rows
    int n_row[2], hi_row[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int p = q0 + warp * 16 + g + 8 * r + 1;           // 1-based position
        const int n = (p <= a.offset) ? p - 1 : a.offset + a.block * ((p - 1 - a.offset) / a.block);
        const int slot = p - n;
        n_row[r] = (p <= a.S) ? n : 0;
        hi_row[r] = (p <= a.S) ? n + min(slot, a.step) - 1 : 0;
    }
    // tiles of true keys the CTA must visit: up to the largest n(p) in the tile
    const int p_last = min(q0 + kBQ, a.S);
    const int n_max = (p_last <= a.offset) ? p_last - 1 : a.offset + a.block * ((p_last - 1 - a.offset) / a.block);
    const int p_first = q0 + 1;
    const int n_min = (p_first <= a.offset) ? p_first - 1 : a.offset + a.block * ((p_first - 1 - a.offset) / a.block);
    const int n_true_tiles = (n_max + kBKey - 1) / kBKey;
    // predicted keys live in [n_min, n_max + block - 1): at most two tiles on the diagonal
    const int band_lo_tile = n_min / kBKey;
    const int band_hi = min(n_max + a.block - 1, a.S);
    const int n_pred_tiles = (a.step > 1 && band_hi > n_min) ? (band_hi + kBKey - 1) / kBKey - band_lo_tile : 0;
    const int n_iter = n_true_tiles + n_pred_tiles;
    const int row_base = b * a.S;

    auto issue = [&](int it) {                                  // thread 0 only
        const int st = it & 1;
        const bool pred = it >= n_true_tiles;
        const int kt = pred ? band_lo_tile + (it - n_true_tiles) : it;
        const uint32_t dK = sKV + st * 2 * kTile, dV = dK + kTile;
        const uint32_t bar = barF + 8 * st;
        mbar_expect_tx(bar, 2 * kTile);
#pragma unroll
        for (int hf = 0; hf < kHalves; ++hf) {
            tma_load_2d(dK + hf * (64 * 128), pred ? &tmKp : &tmKt, bar, kvh * DH + hf * 64, row_base + kt * kBKey);
            tma_load_2d(dV + hf * (64 * 128), pred ? &tmVp : &tmVt, bar, kvh * DH + hf * 64, row_base + kt * kBKey);
        }
    };

    if (threadIdx.x == 0) {
        mbar_init(barQ, 1);
        mbar_init(barF, 1);
        mbar_init(barF + 8, 1);
        s_abort = 0;
        fence_barrier_init();
        mbar_expect_tx(barQ, kTile);
#pragma unroll
        for (int hf = 0; hf < kHalves; ++hf) tma_load_2d(sQ + hf * (64 * 128), &tmQ, barQ, h * DH + hf * 64, row_base + q0);
        if (n_iter > 0) issue(0);
    }
    __syncthreads();

    bool ok = mbar_wait(barQ, 0, &s_abort);
    ok = __all_sync(0xffffffffu, ok);
    uint32_t qa[DH / 16][4];
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks)
        ldsm_x4(sQ + toff(warp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1), 2 * ks + (lane >> 4)), qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3]);
    __syncthreads();                                                // stage 1 may now receive K/V tiles

    float o[DH / 8][4];
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

    for (int it = 0; it < n_iter; ++it) {
        const int st = it & 1;
        if (threadIdx.x == 0 && it + 1 < n_iter) issue(it + 1);     // the other stage was released by the barrier below
        if (ok) ok = mbar_wait(barF + 8 * st, (it >> 1) & 1, &s_abort);
        ok = __all_sync(0xffffffffu, ok);
        const bool pred = it >= n_true_tiles;
        const int kt0 = (pred ? band_lo_tile + (it - n_true_tiles) : it) * kBKey;
        const uint32_t sK = sKV + st * 2 * kTile, sV = sK + kTile;

        if (ok) {
            float s[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
            for (int dg = 0; dg < DH / 32; ++dg)
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) {
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4(sK + toff(nt * 8 + (lane & 7), 4 * dg + (lane >> 3)), b0, b1, b2, b3);
                    mma16816(s[nt], qa[2 * dg], b0, b1);
                    mma16816(s[nt], qa[2 * dg + 1], b2, b3);
                }
            // mask + scale (base-2 exponent)
            const bool full = !pred && (kt0 + kBKey <= n_min);     // every key of the tile is visible to every row
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int r = e >> 1;
                    const int j = kt0 + nt * 8 + 2 * c + (e & 1);
                    const bool vis = full || (pred ? (j >= n_row[r] && j < hi_row[r]) : (j < n_row[r]));
                    const float v = vis ? s[nt][e] * a.scale_log2 : -INFINITY;
                    s[nt][e] = v;
                    mx[r] = fmaxf(mx[r], v);
                }
            float corr[2];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
                const float m_new = fmaxf(m_run[r], mx[r]);
                corr[r] = (m_new == -INFINITY) ? 1.f : exp2f(m_run[r] - m_new);    // m_run = -inf: exp2(-inf) = 0
                m_run[r] = m_new;
            }
            uint32_t pa[4][4];
            float ls[2] = {0.f, 0.f};
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                float p[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) p[e] = (m_run[e >> 1] == -INFINITY) ? 0.f : exp2f(s[nt][e] - m_run[e >> 1]);
                const __nv_bfloat162 lo = __floats2bfloat162_rn(p[0], p[1]), hi = __floats2bfloat162_rn(p[2], p[3]);
                ls[0] += __low2float(lo) + __high2float(lo);
                ls[1] += __low2float(hi) + __high2float(hi);
                pa[nt >> 1][(nt & 1) * 2] = *reinterpret_cast<const uint32_t*>(&lo);        // a0 / a2: row g
                pa[nt >> 1][(nt & 1) * 2 + 1] = *reinterpret_cast<const uint32_t*>(&hi);    // a1 / a3: row g + 8
            }
#pragma unroll
            for (int r = 0; r < 2; ++r) l_run[r] = l_run[r] * corr[r] + ls[r];
#pragma unroll
            for (int nt = 0; nt < DH / 8; ++nt) { o[nt][0] *= corr[0]; o[nt][1] *= corr[0]; o[nt][2] *= corr[1]; o[nt][3] *= corr[1]; }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
#pragma unroll
                for (int jp = 0; jp < DH / 16; ++jp) {
                    uint32_t b0, b1, b2, b3;
                    const int mi = lane >> 3;
                    ldsm_x4_t(sV + toff(kk * 16 + 8 * (mi & 1) + (lane & 7), 2 * jp + (mi >> 1)), b0, b1, b2, b3);
                    mma16816(o[2 * jp], pa[kk], b0, b1);
                    mma16816(o[2 * jp + 1], pa[kk], b2, b3);
                }
        }
        __syncthreads();                                            // everyone is done with stage st
    }

    // ---- normalise (the row sums were reduced over the 4 lanes of a row only now) and store through stage 0's memory
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
    if (a.lse2 != nullptr && c == 0) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = q0 + warp * 16 + g + 8 * r;
            if (row < a.S) a.lse2[((size_t)(row_base + row)) * a.Hq + h] = l_run[r] > 0.f ? m_run[r] + log2f(l_run[r]) : 0.f;
        }
    }
    const float inv0 = (ok && l_run[0] > 0.f) ? 1.f / l_run[0] : 0.f;
    const float inv1 = (ok && l_run[1] > 0.f) ? 1.f / l_run[1] : 0.f;
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt) {
        const int r0 = warp * 16 + g;
        *reinterpret_cast<uint32_t*>(smem_gen + toff(r0, nt) + 4 * c) = pack2(o[nt][0] * inv0, o[nt][1] * inv0);
        *reinterpret_cast<uint32_t*>(smem_gen + toff(r0 + 8, nt) + 4 * c) = pack2(o[nt][2] * inv1, o[nt][3] * inv1);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kBQ * (DH / 8); i += kWarps * 32) {
        const int row = i / (DH / 8), ch = i % (DH / 8);
        if (q0 + row < a.S)
            *reinterpret_cast<uint4*>(a.O + ((size_t)(row_base + q0 + row) * a.Hq + h) * DH + ch * 8) =
                *reinterpret_cast<const uint4*>(smem_gen + toff(row, ch));
    }
    if (threadIdx.x == 0 && s_abort) {
        if (a.error_word != nullptr) atomicExch(a.error_word, 1);
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(barQ, 0); ++i) {}
    }
}

template <int DH>
int launch_blk(const CUtensorMap* maps, const BlkArgs& a, dim3 grid, cudaStream_t stream) {
    constexpr int kSmem = 4 * 64 * DH * 2 + 1024 + 64;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(attn_block_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess) return -1;
        attr_done = true;
    }
    attn_block_tc_kernel<DH><<<grid, kWarps * 32, kSmem, stream>>>(maps[0], maps[1], maps[2], maps[3], maps[4], a);
    return 1;
}

}  // namespace

int tc_attn_block(TcPlan* p, const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp, int B, int S, int Hq,
                  int Hkv, int dh, int block, int offset, int step, void* O, int* error_word, cudaStream_t stream, float* lse2) {
    if (p == nullptr || (dh != 64 && dh != 128) || B <= 0 || S <= 0 || B > 65535 || Hq > 65535) return -1;
    const long long rows = (long long)B * S;
    CUtensorMap maps[5];
    if (!tc_encode_map(p, &maps[0], Q, rows, (long long)Hq * dh, (long long)Hq * dh, kBQ)) return -1;
    const void* kv[4] = {Kt, Vt, Kp, Vp};
    for (int i = 0; i < 4; ++i)
        if (!tc_encode_map(p, &maps[1 + i], kv[i], rows, (long long)Hkv * dh, (long long)Hkv * dh, kBKey)) return -1;
    BlkArgs a;
    a.S = S; a.Hq = Hq; a.Hkv = Hkv; a.block = block; a.offset = offset; a.step = step;
    a.scale_log2 = 1.4426950408889634f / sqrtf((float)dh);
    a.O = static_cast<bf16*>(O);
    a.lse2 = lse2;
    a.error_word = error_word;
    dim3 grid((S + kBQ - 1) / kBQ, Hq, B);
    return dh == 128 ? launch_blk<128>(maps, a, grid, stream) : launch_blk<64>(maps, a, grid, stream);
}

}  // namespace beagle
