// Backward of the block-masked cross-attention (Section 4.2) on the tensor cores, bf16, head_dim 64 / 128.
//
// With P = softmax over the visible keys of Q K^T / sqrt(dh) (recomputed from the forward's per-row
// log-sum-exp), dP = dO V^T, delta = rowsum(dO * O) and dS = P * (dP - delta):
//     dQ = dS K / sqrt(dh),   dK = dS^T Q / sqrt(dh),   dV = P^T dO.
// Two kernels, neither needs atomics, both sum in a fixed order:
//   * query side: one CTA = 64 queries of one (sequence, query head), walking the key tiles exactly as
//     the forward does (true tiles, then the predicted band) and accumulating dQ;
//   * key side: one CTA = 64 keys of one (sequence, K/V head, true | predicted), walking the query
//     tiles that read those keys, for every query head of the group, accumulating dK and dV.  The
//     products are formed transposed (keys as rows): S^T = K Q^T, dP^T = V dO^T.
// Tiles arrive by TMA (128-byte swizzle) in two-stage rings; every wait is bounded.
#include <cstring>

#include "gemm_tc.h"
#include "mma_tiles.cuh"
#include "tc_plan.h"
#include "tc_ptx.cuh"

namespace beagle {

namespace {

using namespace tc;
using namespace mma_tiles;

constexpr int kBQ = 64, kBKey = 64, kWarps = 4;

struct BwdArgs {
    int S, Hq, Hkv, block, offset, step;
    float scale_log2, scale;
    const float* lse2;      // [B*S, Hq] base-2 log-sum-exp of the scaled scores (forward)
    const float* delta;     // [B*S, Hq] rowsum(dO * O)
    bf16* dQ;               // [B*S, Hq*DH]
    bf16 *dKt, *dVt, *dKp, *dVp;   // [B*S, Hkv*DH]
    int* error_word;
};

__device__ __forceinline__ int visible_true(int p, int block, int offset) {     // n(p), p 1-based
    return (p <= offset) ? p - 1 : offset + block * ((p - 1 - offset) / block);
}

// delta[row, h] = sum_i dO[row, h, i] * O[row, h, i]; one warp per (row, head).
__global__ void __launch_bounds__(256) attn_delta_kernel(const bf16* __restrict__ dO, const bf16* __restrict__ O, long long pairs, int DH,
                                                        float* __restrict__ delta) {
    const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= pairs) return;
    const __nv_bfloat162* a = reinterpret_cast<const __nv_bfloat162*>(dO + w * DH);
    const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(O + w * DH);
    float t = 0.f;
    for (int i = lane; i < DH / 2; i += 32) {
        const float2 x = __bfloat1622float2(a[i]), y = __bfloat1622float2(b[i]);
        t = fmaf(x.x, y.x, fmaf(x.y, y.y, t));
    }
    t = warp_sum(t);
    if (lane == 0) delta[w] = t;
}

// ------------------------------------------------------------------------------------------------
// Query side.
// ------------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(kWarps * 32, 2) attn_bwd_q_tc_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                                   const __grid_constant__ CUtensorMap tmdO,
                                                                   const __grid_constant__ CUtensorMap tmKt,
                                                                   const __grid_constant__ CUtensorMap tmVt,
                                                                   const __grid_constant__ CUtensorMap tmKp,
                                                                   const __grid_constant__ CUtensorMap tmVp, const BwdArgs a) {
    constexpr int kTile = 64 * DH * 2;
    constexpr int kHalves = DH / 64;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sKV = smem_base;                    // stage s: K at sKV + s*2*kTile, V right after it
    const uint32_t sQ = sKV + 2 * kTile, sdO = sQ + kTile;   // Q and dO borrow stage 1 until their fragments are in registers
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + 4 * kTile);
    const uint32_t barQ = smem_u32(bars), barF = barQ + 8;
    __shared__ int s_abort;

    const int qtile = gridDim.x - 1 - blockIdx.x;
    const int h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (a.Hq / a.Hkv);
    const int q0 = qtile * kBQ;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const int row_base = b * a.S;

    int n_row[2], hi_row[2];
    float lse_r[2], dl_r[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int p = q0 + warp * 16 + g + 8 * r + 1;
        const int n = visible_true(p, a.block, a.offset);
        const bool valid = p <= a.S;
        n_row[r] = valid ? n : 0;
        hi_row[r] = valid ? n + min(p - n, a.step) - 1 : 0;
        lse_r[r] = valid ? a.lse2[(size_t)(row_base + p - 1) * a.Hq + h] : 0.f;
        dl_r[r] = valid ? a.delta[(size_t)(row_base + p - 1) * a.Hq + h] : 0.f;
    }
    const int p_last = min(q0 + kBQ, a.S);
    const int n_max = visible_true(p_last, a.block, a.offset);
    const int n_min = visible_true(q0 + 1, a.block, a.offset);
    const int n_true_tiles = (n_max + kBKey - 1) / kBKey;
    const int band_lo_tile = n_min / kBKey;
    const int band_hi = min(n_max + a.block - 1, a.S);
    const int n_pred_tiles = (a.step > 1 && band_hi > n_min) ? (band_hi + kBKey - 1) / kBKey - band_lo_tile : 0;
    const int n_iter = n_true_tiles + n_pred_tiles;

    auto issue = [&](int it) {
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
        mbar_expect_tx(barQ, 2 * kTile);
#pragma unroll
        for (int hf = 0; hf < kHalves; ++hf) {
            tma_load_2d(sQ + hf * (64 * 128), &tmQ, barQ, h * DH + hf * 64, row_base + q0);
            tma_load_2d(sdO + hf * (64 * 128), &tmdO, barQ, h * DH + hf * 64, row_base + q0);
        }
        if (n_iter > 0) issue(0);
    }
    __syncthreads();

    bool ok = mbar_wait(barQ, 0, &s_abort);
    ok = __all_sync(0xffffffffu, ok);
    uint32_t qa[DH / 16][4], doa[DH / 16][4];
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
        const uint32_t off = toff(warp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1), 2 * ks + (lane >> 4));
        ldsm_x4(sQ + off, qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3]);
        ldsm_x4(sdO + off, doa[ks][0], doa[ks][1], doa[ks][2], doa[ks][3]);
    }
    __syncthreads();                                   // stage 1 may now receive K/V tiles

    float dq[DH / 8][4];
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt) dq[nt][0] = dq[nt][1] = dq[nt][2] = dq[nt][3] = 0.f;

    for (int it = 0; it < n_iter; ++it) {
        const int st = it & 1;
        if (threadIdx.x == 0 && it + 1 < n_iter) issue(it + 1);
        if (ok) ok = mbar_wait(barF + 8 * st, (it >> 1) & 1, &s_abort);
        ok = __all_sync(0xffffffffu, ok);
        const bool pred = it >= n_true_tiles;
        const int kt0 = (pred ? band_lo_tile + (it - n_true_tiles) : it) * kBKey;
        const uint32_t sK = sKV + st * 2 * kTile, sV = sK + kTile;
        if (ok) {
            float s[8][4], dp[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
                dp[nt][0] = dp[nt][1] = dp[nt][2] = dp[nt][3] = 0.f;
            }
#pragma unroll
            for (int dg = 0; dg < DH / 32; ++dg)
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) {
                    uint32_t b0, b1, b2, b3;
                    const uint32_t off = toff(nt * 8 + (lane & 7), 4 * dg + (lane >> 3));
                    ldsm_x4(sK + off, b0, b1, b2, b3);
                    mma16816(s[nt], qa[2 * dg], b0, b1);
                    mma16816(s[nt], qa[2 * dg + 1], b2, b3);
                    ldsm_x4(sV + off, b0, b1, b2, b3);
                    mma16816(dp[nt], doa[2 * dg], b0, b1);
                    mma16816(dp[nt], doa[2 * dg + 1], b2, b3);
                }
            const bool full = !pred && (kt0 + kBKey <= n_min);
            uint32_t dsa[4][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                float ds[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int r = e >> 1;
                    const int j = kt0 + nt * 8 + 2 * c + (e & 1);
                    const bool vis = (full && hi_row[r] > 0) || (pred ? (j >= n_row[r] && j < hi_row[r]) : (j < n_row[r]));
                    const float p = vis ? exp2f(s[nt][e] * a.scale_log2 - lse_r[r]) : 0.f;
                    ds[e] = p * (dp[nt][e] - dl_r[r]);
                }
                dsa[nt >> 1][(nt & 1) * 2] = pack2(ds[0], ds[1]);
                dsa[nt >> 1][(nt & 1) * 2 + 1] = pack2(ds[2], ds[3]);
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
#pragma unroll
                for (int jp = 0; jp < DH / 16; ++jp) {
                    uint32_t b0, b1, b2, b3;
                    const int mi = lane >> 3;
                    ldsm_x4_t(sK + toff(kk * 16 + 8 * (mi & 1) + (lane & 7), 2 * jp + (mi >> 1)), b0, b1, b2, b3);
                    mma16816(dq[2 * jp], dsa[kk], b0, b1);
                    mma16816(dq[2 * jp + 1], dsa[kk], b2, b3);
                }
        }
        __syncthreads();
    }

    const float sc = ok ? a.scale : 0.f;
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt) {
        const int r0 = warp * 16 + g;
        *reinterpret_cast<uint32_t*>(smem_gen + toff(r0, nt) + 4 * c) = pack2(dq[nt][0] * sc, dq[nt][1] * sc);
        *reinterpret_cast<uint32_t*>(smem_gen + toff(r0 + 8, nt) + 4 * c) = pack2(dq[nt][2] * sc, dq[nt][3] * sc);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kBQ * (DH / 8); i += kWarps * 32) {
        const int row = i / (DH / 8), ch = i % (DH / 8);
        if (q0 + row < a.S)
            *reinterpret_cast<uint4*>(a.dQ + ((size_t)(row_base + q0 + row) * a.Hq + h) * DH + ch * 8) =
                *reinterpret_cast<const uint4*>(smem_gen + toff(row, ch));
    }
    if (threadIdx.x == 0 && s_abort) {
        if (a.error_word != nullptr) atomicExch(a.error_word, 1);
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(barQ, 0); ++i) {}
    }
}

// ------------------------------------------------------------------------------------------------
// Key side.  blockIdx.z = sequence * nz + kind, kind 0 = true keys, 1 = predicted keys (nz = 2 when
// step > 1).  Rows of the products are keys (16 per warp), columns are the 64 queries of a tile.
// ------------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(kWarps * 32, 2) attn_bwd_kv_tc_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                                    const __grid_constant__ CUtensorMap tmdO,
                                                                    const __grid_constant__ CUtensorMap tmKt,
                                                                    const __grid_constant__ CUtensorMap tmVt,
                                                                    const __grid_constant__ CUtensorMap tmKp,
                                                                    const __grid_constant__ CUtensorMap tmVp, const BwdArgs a, const int nz) {
    constexpr int kTile = 64 * DH * 2;
    constexpr int kHalves = DH / 64;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sK = smem_base, sV = sK + kTile;
    const uint32_t sQd = sV + kTile;                   // stage s: Q at sQd + s*2*kTile, dO right after it
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + 6 * kTile);
    const uint32_t barKV = smem_u32(bars), barF = barKV + 8;
    __shared__ int s_abort;
    __shared__ float s_ls[2][kBQ], s_dl[2][kBQ];     // the query tile's log-sum-exp and delta, per stage

    const int kt = blockIdx.x, kvh = blockIdx.y;
    const int b = blockIdx.z / nz, pred = blockIdx.z % nz;
    const int G = a.Hq / a.Hkv;
    const int kt0 = kt * kBKey;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const int row_base = b * a.S;
    const int n_qtiles = (a.S + kBQ - 1) / kBQ;

    // query tiles that read keys of this tile
    int qt_lo = kt, qt_hi;
    if (!pred) {
        qt_hi = n_qtiles - 1;
        while (qt_lo <= qt_hi && visible_true(min(qt_lo * kBQ + kBQ, a.S), a.block, a.offset) <= kt0) ++qt_lo;
    } else {
        qt_hi = min(n_qtiles - 1, (kt0 + kBKey - 1 + a.block) / kBQ);
    }
    const int n_qt = max(qt_hi - qt_lo + 1, 0);
    const int n_iter = n_qt * G;

    auto issue = [&](int it) {
        const int st = it & 1;
        const int qt = qt_lo + it / G, h = kvh * G + it % G;
        const uint32_t dQs = sQd + st * 2 * kTile, dOs = dQs + kTile;
        const uint32_t bar = barF + 8 * st;
        mbar_expect_tx(bar, 2 * kTile);
#pragma unroll
        for (int hf = 0; hf < kHalves; ++hf) {
            tma_load_2d(dQs + hf * (64 * 128), &tmQ, bar, h * DH + hf * 64, row_base + qt * kBQ);
            tma_load_2d(dOs + hf * (64 * 128), &tmdO, bar, h * DH + hf * 64, row_base + qt * kBQ);
        }
    };

    if (threadIdx.x == 0) {
        mbar_init(barKV, 1);
        mbar_init(barF, 1);
        mbar_init(barF + 8, 1);
        s_abort = 0;
        fence_barrier_init();
        mbar_expect_tx(barKV, 2 * kTile);
#pragma unroll
        for (int hf = 0; hf < kHalves; ++hf) {
            tma_load_2d(sK + hf * (64 * 128), pred ? &tmKp : &tmKt, barKV, kvh * DH + hf * 64, row_base + kt0);
            tma_load_2d(sV + hf * (64 * 128), pred ? &tmVp : &tmVt, barKV, kvh * DH + hf * 64, row_base + kt0);
        }
        if (n_iter > 0) issue(0);
    }
    __syncthreads();
    bool ok = mbar_wait(barKV, 0, &s_abort);
    ok = __all_sync(0xffffffffu, ok);

    float dk[DH / 8][4], dv[DH / 8][4];
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt) {
        dk[nt][0] = dk[nt][1] = dk[nt][2] = dk[nt][3] = 0.f;
        dv[nt][0] = dv[nt][1] = dv[nt][2] = dv[nt][3] = 0.f;
    }
    const int j_row[2] = {kt0 + warp * 16 + g, kt0 + warp * 16 + g + 8};      // 0-based key rows of this thread

    for (int it = 0; it < n_iter; ++it) {
        const int st = it & 1;
        if (threadIdx.x == 0 && it + 1 < n_iter) issue(it + 1);
        const int qt = qt_lo + it / G, h = kvh * G + it % G;
        const int qb = qt * kBQ;
        {   // this tile's row statistics (stage st was last read two iterations ago, before that iteration's closing barrier)
            const int qi = qb + (threadIdx.x & 63);
            const float val = qi < a.S ? (threadIdx.x < 64 ? a.lse2 : a.delta)[(size_t)(row_base + qi) * a.Hq + h] : 0.f;
            (threadIdx.x < 64 ? s_ls : s_dl)[st][threadIdx.x & 63] = val;
        }
        if (ok) ok = mbar_wait(barF + 8 * st, (it >> 1) & 1, &s_abort);
        ok = __all_sync(0xffffffffu, ok);
        __syncthreads();
        const uint32_t sQ = sQd + st * 2 * kTile, sdO = sQ + kTile;
        if (ok) {
            float s[8][4], dp[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
                dp[nt][0] = dp[nt][1] = dp[nt][2] = dp[nt][3] = 0.f;
            }
#pragma unroll
            for (int dg = 0; dg < DH / 32; ++dg) {
                uint32_t ka[2][4], va[2][4];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const uint32_t off = toff(warp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1), 2 * (2 * dg + u) + (lane >> 4));
                    ldsm_x4(sK + off, ka[u][0], ka[u][1], ka[u][2], ka[u][3]);
                    ldsm_x4(sV + off, va[u][0], va[u][1], va[u][2], va[u][3]);
                }
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) {
                    uint32_t b0, b1, b2, b3;
                    const uint32_t off = toff(nt * 8 + (lane & 7), 4 * dg + (lane >> 3));
                    ldsm_x4(sQ + off, b0, b1, b2, b3);
                    mma16816(s[nt], ka[0], b0, b1);
                    mma16816(s[nt], ka[1], b2, b3);
                    ldsm_x4(sdO + off, b0, b1, b2, b3);
                    mma16816(dp[nt], va[0], b0, b1);
                    mma16816(dp[nt], va[1], b2, b3);
                }
            }
            // every query of the tile sees every key of the tile: no mask needed
            const bool full = !pred && qb + kBQ <= a.S && visible_true(qb + 1, a.block, a.offset) >= kt0 + kBKey;
            // s <- P^T, dp <- dS^T
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int qi = qb + nt * 8 + 2 * c + u;                 // 0-based query position
                    const bool valid = qi < a.S;
                    const float ls = s_ls[st][nt * 8 + 2 * c + u], dl = s_dl[st][nt * 8 + 2 * c + u];
                    int n = 0, hi = 0;
                    if (!full && valid) {
                        n = visible_true(qi + 1, a.block, a.offset);
                        hi = n + min(qi + 1 - n, a.step) - 1;
                    }
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        const int e = 2 * r + u;
                        const int j = j_row[r];
                        const bool vis = full || (valid && (pred ? (j >= n && j < hi) : (j < n)));
                        const float p = vis ? exp2f(s[nt][e] * a.scale_log2 - ls) : 0.f;
                        s[nt][e] = p;
                        dp[nt][e] = p * (dp[nt][e] - dl);
                    }
                }
            }
            uint32_t pa[4][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                pa[nt >> 1][(nt & 1) * 2] = pack2(s[nt][0], s[nt][1]);
                pa[nt >> 1][(nt & 1) * 2 + 1] = pack2(s[nt][2], s[nt][3]);
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
#pragma unroll
                for (int jp = 0; jp < DH / 16; ++jp) {
                    uint32_t b0, b1, b2, b3;
                    const int mi = lane >> 3;
                    ldsm_x4_t(sdO + toff(kk * 16 + 8 * (mi & 1) + (lane & 7), 2 * jp + (mi >> 1)), b0, b1, b2, b3);
                    mma16816(dv[2 * jp], pa[kk], b0, b1);
                    mma16816(dv[2 * jp + 1], pa[kk], b2, b3);
                }
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                pa[nt >> 1][(nt & 1) * 2] = pack2(dp[nt][0], dp[nt][1]);
                pa[nt >> 1][(nt & 1) * 2 + 1] = pack2(dp[nt][2], dp[nt][3]);
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
#pragma unroll
                for (int jp = 0; jp < DH / 16; ++jp) {
                    uint32_t b0, b1, b2, b3;
                    const int mi = lane >> 3;
                    ldsm_x4_t(sQ + toff(kk * 16 + 8 * (mi & 1) + (lane & 7), 2 * jp + (mi >> 1)), b0, b1, b2, b3);
                    mma16816(dk[2 * jp], pa[kk], b0, b1);
                    mma16816(dk[2 * jp + 1], pa[kk], b2, b3);
                }
        }
        __syncthreads();
    }

    // store dK (scaled) and dV through the two stage-0 tiles
    const float sc = ok ? a.scale : 0.f, one = ok ? 1.f : 0.f;
    uint8_t* oK = smem_gen + 2 * kTile;
    uint8_t* oV = oK + kTile;
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt) {
        const int r0 = warp * 16 + g;
        *reinterpret_cast<uint32_t*>(oK + toff(r0, nt) + 4 * c) = pack2(dk[nt][0] * sc, dk[nt][1] * sc);
        *reinterpret_cast<uint32_t*>(oK + toff(r0 + 8, nt) + 4 * c) = pack2(dk[nt][2] * sc, dk[nt][3] * sc);
        *reinterpret_cast<uint32_t*>(oV + toff(r0, nt) + 4 * c) = pack2(dv[nt][0] * one, dv[nt][1] * one);
        *reinterpret_cast<uint32_t*>(oV + toff(r0 + 8, nt) + 4 * c) = pack2(dv[nt][2] * one, dv[nt][3] * one);
    }
    __syncthreads();
    bf16* outK = pred ? a.dKp : a.dKt;
    bf16* outV = pred ? a.dVp : a.dVt;
    for (int i = threadIdx.x; i < kBKey * (DH / 8); i += kWarps * 32) {
        const int row = i / (DH / 8), ch = i % (DH / 8);
        if (kt0 + row < a.S) {
            const size_t at = ((size_t)(row_base + kt0 + row) * a.Hkv + kvh) * DH + ch * 8;
            *reinterpret_cast<uint4*>(outK + at) = *reinterpret_cast<const uint4*>(oK + toff(row, ch));
            *reinterpret_cast<uint4*>(outV + at) = *reinterpret_cast<const uint4*>(oV + toff(row, ch));
        }
    }
    if (threadIdx.x == 0 && s_abort) {
        if (a.error_word != nullptr) atomicExch(a.error_word, 1);
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(barKV, 0); ++i) {}
    }
}

template <int DH>
int launch_bwd(const CUtensorMap* maps, const BwdArgs& a, int B, int nz, cudaStream_t stream) {
    constexpr int kSmemQ = 4 * 64 * DH * 2 + 1024 + 64, kSmemKV = 6 * 64 * DH * 2 + 1024 + 64;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(attn_bwd_q_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemQ) != cudaSuccess) return -1;
        if (cudaFuncSetAttribute(attn_bwd_kv_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemKV) != cudaSuccess) return -1;
        attr_done = true;
    }
    const int tiles = (a.S + kBQ - 1) / kBQ;
    attn_bwd_q_tc_kernel<DH><<<dim3(tiles, a.Hq, B), kWarps * 32, kSmemQ, stream>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], a);
    attn_bwd_kv_tc_kernel<DH><<<dim3(tiles, a.Hkv, B * nz), kWarps * 32, kSmemKV, stream>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], a,
                                                                                          nz);
    return 2;
}

}  // namespace

int tc_attn_block_bwd(TcPlan* p, const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp, const void* O, const void* dO,
                      const float* lse2, int B, int S, int Hq, int Hkv, int dh, int block, int offset, int step, float* delta, void* dQ,
                      void* dKt, void* dVt, void* dKp, void* dVp, int* error_word, cudaStream_t stream) {
    if (p == nullptr || (dh != 64 && dh != 128) || B <= 0 || S <= 0 || 2 * B > 65535 || Hq > 65535) return -1;
    const long long rows = (long long)B * S;
    CUtensorMap maps[6];
    if (!tc_encode_map(p, &maps[0], Q, rows, (long long)Hq * dh, (long long)Hq * dh, kBQ)) return -1;
    if (!tc_encode_map(p, &maps[1], dO, rows, (long long)Hq * dh, (long long)Hq * dh, kBQ)) return -1;
    const void* kv[4] = {Kt, Vt, Kp, Vp};
    for (int i = 0; i < 4; ++i)
        if (!tc_encode_map(p, &maps[2 + i], kv[i], rows, (long long)Hkv * dh, (long long)Hkv * dh, kBKey)) return -1;
    BwdArgs a;
    a.S = S; a.Hq = Hq; a.Hkv = Hkv; a.block = block; a.offset = offset; a.step = step;
    a.scale = 1.0f / sqrtf((float)dh);
    a.scale_log2 = 1.4426950408889634f * a.scale;
    a.lse2 = lse2; a.delta = delta;
    a.dQ = static_cast<bf16*>(dQ);
    a.dKt = static_cast<bf16*>(dKt); a.dVt = static_cast<bf16*>(dVt); a.dKp = static_cast<bf16*>(dKp); a.dVp = static_cast<bf16*>(dVp);
    a.error_word = error_word;
    const long long pairs = rows * Hq;
    attn_delta_kernel<<<(unsigned)((pairs * 32 + 255) / 256), 256, 0, stream>>>(static_cast<const bf16*>(dO), static_cast<const bf16*>(O), pairs, dh,
                                                                              delta);
    const int nz = step > 1 ? 2 : 1;
    const int rc = dh == 128 ? launch_bwd<128>(maps, a, B, nz, stream) : launch_bwd<64>(maps, a, B, nz, stream);
    return rc < 0 ? rc : rc + 1;
}

}  // namespace beagle
