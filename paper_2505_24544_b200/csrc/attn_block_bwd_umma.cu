// Backward of the block-masked cross-attention (Section 4.2) on tcgen05, bf16, head_dim 64 / 128.
//
// With P = softmax over the visible keys of Q K^T / sqrt(dh) (recomputed from the forward's per-row
// log-sum-exp), dP = dO V^T, delta = rowsum(dO * O) and dS = P * (dP - delta):
//     dQ = dS K / sqrt(dh),   dK = dS^T Q / sqrt(dh),   dV = P^T dO.
// Two kernels, no atomics, every sum in a fixed order (as in the mma.sync version):
//   * key side: one CTA = 128 keys of one (sequence, K/V head, true | predicted) = the 128 rows of the
//     MMA tiles; K and V stay in shared memory, the query tiles (64 queries) that read these keys are
//     streamed, for every query head of the group:  S^T = K Q^T and dP^T = V dO^T into tensor memory,
//     one thread per key row forms P^T and dS^T, writes them to shared memory in the operand layout,
//     and  dV += P^T dO,  dK += dS^T Q  accumulate in tensor memory over all tiles;
//   * query side: one CTA = 128 queries of one (sequence, query head); Q and dO stay in shared memory,
//     key tiles (64 keys) are streamed:  S = Q K^T, dP = dO V^T, dS -> shared memory, dQ += dS K.
// The accumulating products contract over the streamed dimension: their B operands (Q, dO, K tiles as they lie,
// [streamed index][head_dim]) are read in the MN-major form, so no transposed copy of any tensor is needed.
// Roles per CTA: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2-5 = one thread
// per tile row.  Every wait is bounded.
#include <cstring>

#include "gemm_tc.h"
#include "tc_plan.h"
#include "tc_ptx.cuh"

namespace beagle {

namespace {

using namespace tc;

constexpr int kBM = 128;          // rows of a CTA's tiles (keys on the key side, queries on the query side)
constexpr int kBS = 64;           // streamed tile (queries on the key side, keys on the query side)
constexpr int kBwdThreads = 320;   // warp 0 producer, warp 1 MMA issuer, warps 2-9: two threads per tile row (32 streamed columns each)

struct UBwdArgs {
    int S, Hq, Hkv, block, offset, step;
    float scale_log2, scale;
    const float* lse2;      // [B*S, Hq]
    const float* delta;     // [B*S, Hq]
    bf16* dQ;               // [B*S, Hq*DH]
    bf16 *dKt, *dVt, *dKp, *dVp;   // [B*S, Hkv*DH]
    int* error_word;
};

__device__ __forceinline__ int nvis(int p, int block, int offset) {      // n(p), p 1-based
    return (p <= offset) ? p - 1 : offset + block * ((p - 1 - offset) / block);
}
__device__ __forceinline__ void fence_async_smem_bwd() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void softmax_group_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// delta[row, h] = sum_i dO[row, h, i] * O[row, h, i]; one warp per (row, head).
__global__ void __launch_bounds__(256) attn_delta_umma_kernel(const bf16* __restrict__ dO, const bf16* __restrict__ O, long long pairs, int DH,
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
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (lane == 0) delta[w] = t;
}

// Half `half` (32 columns = four 16-byte chunks, from pk[16]) of row `row` of a [128 x 64] bf16 operand tile
// (128-byte rows, 128-byte swizzle).
__device__ __forceinline__ void store_operand_half_row(uint8_t* tile, int row, int half, const uint32_t* pk) {
#pragma unroll
    for (int c = 0; c < 4; ++c)
        *reinterpret_cast<uint4*>(tile + row * 128 + (((4 * half + c) ^ (row & 7)) << 4)) =
            make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
}

// One thread's half row of a TMEM accumulator (columns col0 .. col0 + DH/2), scaled, as bf16 to global memory.
template <int DH>
__device__ __forceinline__ void store_acc_row(uint32_t taddr, float scale, bf16* dst, bool write, int col0) {
#pragma unroll
    for (int cc = 0; cc < DH / 2; cc += 32) {
        const int c0 = col0 + cc;
        uint32_t ra[16], rb[16];
        tmem_ld16(taddr + c0, ra);
        tmem_ld16(taddr + c0 + 16, rb);
        tmem_ld_wait();
        if (write) {
            uint32_t o[16];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const __nv_bfloat162 t0 = __floats2bfloat162_rn(__uint_as_float(ra[2 * i]) * scale, __uint_as_float(ra[2 * i + 1]) * scale);
                const __nv_bfloat162 t1 = __floats2bfloat162_rn(__uint_as_float(rb[2 * i]) * scale, __uint_as_float(rb[2 * i + 1]) * scale);
                o[i] = *reinterpret_cast<const uint32_t*>(&t0);
                o[8 + i] = *reinterpret_cast<const uint32_t*>(&t1);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(dst + c0 + 8 * i) = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Key side.  blockIdx.z = sequence * nz + kind, kind 0 = true keys, 1 = predicted keys (nz = 2 when
// step > 1).  TMEM: two buffers of 128 columns (S^T, dP^T of 64 queries each) at 0 and 128, dV at
// 256, dK at 256 + DH.
// ------------------------------------------------------------------------------------------------
template <int DH>
struct UBwdKvSmem {
    static constexpr int kRes = kBM * DH * 2;           // K (or V) of the CTA's 128 keys
    static constexpr int kTile = kBS * DH * 2;          // a 64-query tile of Q / dO
    static constexpr int kOp = kBM * kBS * 2;           // P^T / dS^T operand tile
    static constexpr int kBytes = 2 * kRes + 4 * kTile + 2 * kTile + 2 * kOp + 1024 + 128;
};

template <int DH>
__global__ void __launch_bounds__(kBwdThreads, 1) attn_bwd_kv_umma_kernel(const __grid_constant__ CUtensorMap tmK128,
                                                                        const __grid_constant__ CUtensorMap tmV128,
                                                                        const __grid_constant__ CUtensorMap tmKp128,
                                                                        const __grid_constant__ CUtensorMap tmVp128,
                                                                        const __grid_constant__ CUtensorMap tmQ64,
                                                                        const __grid_constant__ CUtensorMap tmdO64, const UBwdArgs a,
                                                                        const int nz) {
    using SM = UBwdKvSmem<DH>;
    constexpr int kHalves = DH / 64;
    constexpr uint32_t kTmemCols = 512;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sKr = smem_base, sVr = sKr + SM::kRes;
    const uint32_t sQd = sVr + SM::kRes;                 // stage s: Q at sQd + 2 s kTile, dO right after it
    const uint32_t sQT = sQd + 4 * SM::kTile, sdOT = sQT + SM::kTile;
    const uint32_t sPT = sdOT + SM::kTile, sdST = sPT + SM::kOp;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + 2 * SM::kRes + 6 * SM::kTile + 2 * SM::kOp);
    const uint32_t bar0 = smem_u32(bars);
    const uint32_t kv_full = bar0, qdo_full = bar0 + 8, qdo_empty = bar0 + 24, t_full = bar0 + 40, t_empty = bar0 + 48;
    const uint32_t s_full = bar0 + 56, s_empty = bar0 + 72, p_full = bar0 + 88, p_empty = bar0 + 96, o_full = bar0 + 104;
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort_word;
    __shared__ __align__(16) float s_ls[2][kBS], s_dl[2][kBS];     // read four columns at a time
    __shared__ int s_n[2][kBS], s_hi[2][kBS];
    volatile int* s_abort = &s_abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kt = blockIdx.x;                            // early key tiles are read by the most queries: they start first
    const int kvh = blockIdx.y;
    const int b = blockIdx.z / nz, pred = blockIdx.z % nz;
    const int G = a.Hq / a.Hkv;
    const int kt0 = kt * kBM;
    const int row_base = b * a.S;
    const int n_qtiles = (a.S + kBS - 1) / kBS;

    // query tiles that read keys of this tile
    int qt_lo = kt0 / kBS, qt_hi;
    if (!pred) {
        qt_hi = n_qtiles - 1;
        while (qt_lo <= qt_hi && nvis(min(qt_lo * kBS + kBS, a.S), a.block, a.offset) <= kt0) ++qt_lo;
    } else {
        qt_hi = min(n_qtiles - 1, (kt0 + kBM - 1 + a.block) / kBS);
    }
    const int n_qt = max(qt_hi - qt_lo + 1, 0);
    const int J = n_qt * G;

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(qdo_full + 8 * s, 1); mbar_init(qdo_empty + 8 * s, 1);
            mbar_init(s_full + 8 * s, 1); mbar_init(s_empty + 8 * s, 8);
        }
        mbar_init(t_full, 1); mbar_init(t_empty, 1);
        mbar_init(p_full, 8); mbar_init(p_empty, 1);
        mbar_init(o_full, 1);
        s_abort_word = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc<kTmemCols>(smem_u32(&s_tmem));
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem_base = s_tmem;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0 && J > 0) {
            mbar_expect_tx(kv_full, 2 * SM::kRes);
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) {
                tma_load_2d(sKr + hf * (kBM * 128), pred ? &tmKp128 : &tmK128, kv_full, kvh * DH + hf * 64, row_base + kt0);
                tma_load_2d(sVr + hf * (kBM * 128), pred ? &tmVp128 : &tmV128, kv_full, kvh * DH + hf * 64, row_base + kt0);
            }
            bool ok = true;
            int issued = 0;
            for (int j = 0; j < J && ok; ++j) {
                const int st = j & 1;
                const int qt = qt_lo + j / G, h = kvh * G + j % G;
                ok = mbar_wait(qdo_empty + 8 * st, ((j >> 1) & 1) ^ 1, s_abort);
                if (!ok) break;
                mbar_expect_tx(qdo_full + 8 * st, 2 * SM::kTile);
                const uint32_t dQs = sQd + st * 2 * SM::kTile, dOs = dQs + SM::kTile;
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    tma_load_2d(dQs + hf * (kBS * 128), &tmQ64, qdo_full + 8 * st, h * DH + hf * 64, row_base + qt * kBS);
                    tma_load_2d(dOs + hf * (kBS * 128), &tmdO64, qdo_full + 8 * st, h * DH + hf * 64, row_base + qt * kBS);
                }
                ok = mbar_wait(t_empty, (j & 1) ^ 1, s_abort);
                if (!ok) { issued = j + 1; break; }
                mbar_expect_tx(t_full, 2 * SM::kTile);
                // the same two tiles once more for the accumulating products, which read them as MN-major operands
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    tma_load_2d(sQT + hf * (kBS * 128), &tmQ64, t_full, h * DH + hf * 64, row_base + qt * kBS);
                    tma_load_2d(sdOT + hf * (kBS * 128), &tmdO64, t_full, h * DH + hf * 64, row_base + qt * kBS);
                }
                issued = j + 1;
            }
            if (*s_abort) {      // copies already requested still land: bounded wait for the latest of each buffer
                for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(kv_full, 0); ++i) {}
                for (int n = max(0, issued - 2); n < issued; ++n)
                    for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(qdo_full + 8 * (n & 1), (n >> 1) & 1); ++i) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0 && J > 0) {
            constexpr uint32_t idesc_s = make_idesc(kBM, kBS), idesc_o = make_idesc_major(kBM, DH, false, true);
            bool ok = mbar_wait(kv_full, 0, s_abort);
            auto issue_s = [&](int j) {
                const int st = j & 1;
                if (ok) ok = mbar_wait(qdo_full + 8 * st, (j >> 1) & 1, s_abort);
                if (ok) ok = mbar_wait(s_empty + 8 * st, ((j >> 1) & 1) ^ 1, s_abort);
                if (!ok) return;
                fence_after();
                const uint32_t ts = tmem_base + st * 128;
                const uint32_t dQs = sQd + st * 2 * SM::kTile, dOs = dQs + SM::kTile;
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    const uint64_t dk = umma_desc(sKr + hf * (kBM * 128)), dq = umma_desc(dQs + hf * (kBS * 128));
                    const uint64_t dv = umma_desc(sVr + hf * (kBM * 128)), dd = umma_desc(dOs + hf * (kBS * 128));
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t koff = static_cast<uint64_t>((k * UMMA_K * 2) >> 4);
                        umma_bf16(ts, dk + koff, dq + koff, idesc_s, (hf > 0 || k > 0) ? 1u : 0u);            // S^T = K Q^T
                        umma_bf16(ts + kBS, dv + koff, dd + koff, idesc_s, (hf > 0 || k > 0) ? 1u : 0u);      // dP^T = V dO^T
                    }
                }
                umma_commit(qdo_empty + 8 * st);
                umma_commit(s_full + 8 * st);
            };
            issue_s(0);
            for (int j = 0; j < J && ok; ++j) {
                if (j + 1 < J) issue_s(j + 1);
                if (!ok) break;
                ok = mbar_wait(p_full, j & 1, s_abort);
                if (ok) ok = mbar_wait(t_full, j & 1, s_abort);
                if (!ok) break;
                fence_after();
                // dO and Q tiles as they lie ([query][head_dim]): MN-major B operands, 16 query rows of 128 bytes per step
                const uint64_t dpt = umma_desc(sPT), ddot = umma_desc_mn(sdOT, kBS * 128), dst = umma_desc(sdST), dqt = umma_desc_mn(sQT, kBS * 128);
#pragma unroll
                for (int k = 0; k < kBS / UMMA_K; ++k) {
                    const uint64_t koff = static_cast<uint64_t>((k * UMMA_K * 2) >> 4);
                    const uint64_t koff_mn = static_cast<uint64_t>((k * UMMA_K * 128) >> 4);
                    umma_bf16(tmem_base + 256, dpt + koff, ddot + koff_mn, idesc_o, (j > 0 || k > 0) ? 1u : 0u);           // dV += P^T dO
                    umma_bf16(tmem_base + 256 + DH, dst + koff, dqt + koff_mn, idesc_o, (j > 0 || k > 0) ? 1u : 0u);      // dK += dS^T Q
                }
                umma_commit(t_empty);
                umma_commit(p_empty);
            }
            umma_commit(o_full);
        }
    } else {
        // ---------------- one thread per key row
        const int q = warp & 3, half = (warp - 2) >> 2;          // TMEM lane quarter; which 32 of the 64 streamed columns
        const int row = q * 32 + lane;
        const int key = kt0 + row;                               // 0-based key position of this thread
        const int tid_s = threadIdx.x - 64;                      // 0..255 inside this role
        const uint32_t lane_off = static_cast<uint32_t>(q * 32) << 16;
        bool ok = true;
        for (int j = 0; j < J; ++j) {
            const int st = j & 1;
            const int qt = qt_lo + j / G, h = kvh * G + j % G;
            const int qb = qt * kBS;
            {   // this tile's per-query data: visible range bounds, log-sum-exp, delta (buffer st was last read two jobs ago)
                const int c = tid_s & 63, qi = qb + c;
                const bool qvalid = qi < a.S;
                if (tid_s < 64) {
                    const int n = qvalid ? nvis(qi + 1, a.block, a.offset) : 0;
                    s_n[st][c] = n;
                    s_hi[st][c] = qvalid ? n + min(qi + 1 - n, a.step) - 1 : 0;
                } else if (tid_s < 128) {
                    const size_t at = (size_t)(row_base + (qvalid ? qi : 0)) * a.Hq + h;
                    s_ls[st][c] = qvalid ? a.lse2[at] : 0.f;
                    s_dl[st][c] = qvalid ? a.delta[at] : 0.f;
                }
            }
            softmax_group_sync();                                // every warp of the role meets it in every job, also after giving up
            if (ok) ok = mbar_wait(s_full + 8 * st, (j >> 1) & 1, s_abort);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) continue;
            fence_after();
            // every query of the tile sees every key of the CTA: no mask
            const bool full = !pred && qb + kBS <= a.S && nvis(qb + 1, a.block, a.offset) >= kt0 + kBM;
            uint32_t pk_p[16], pk_ds[16];
            const uint32_t ts = tmem_base + st * 128 + lane_off + 32 * half;
            uint32_t rs[2][16], rd[2][16];
#pragma unroll
            for (int c = 0; c < 2; ++c) { tmem_ld16(ts + 16 * c, rs[c]); tmem_ld16(ts + kBS + 16 * c, rd[c]); }
            tmem_ld_wait();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty + 8 * st);        // this warp's part of the buffer is in registers
#pragma unroll
            for (int c = 0; c < 2; ++c) {
#pragma unroll
                for (int i = 0; i < 16; i += 4) {
                    // the four queries' log-sum-exp and delta with one 16-byte load each (the same words for every lane)
                    const int col0 = 32 * half + 16 * c + i;
                    const float4 ls4 = *reinterpret_cast<const float4*>(&s_ls[st][col0]);
                    const float4 dl4 = *reinterpret_cast<const float4*>(&s_dl[st][col0]);
                    const float lsv[4] = {ls4.x, ls4.y, ls4.z, ls4.w}, dlv[4] = {dl4.x, dl4.y, dl4.z, dl4.w};
                    float pv[4], dv[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        float p = exp2f(fmaf(__uint_as_float(rs[c][i + u]), a.scale_log2, -lsv[u]));
                        if (!full) {
                            const int n = s_n[st][col0 + u], hi = s_hi[st][col0 + u];
                            const bool vis = pred ? (key >= n && key < hi) : (key < n);
                            p = vis ? p : 0.f;
                        }
                        pv[u] = p;
                        dv[u] = p * (__uint_as_float(rd[c][i + u]) - dlv[u]);
                    }
#pragma unroll
                    for (int u = 0; u < 4; u += 2) {
                        const __nv_bfloat162 tp = __floats2bfloat162_rn(pv[u], pv[u + 1]), td = __floats2bfloat162_rn(dv[u], dv[u + 1]);
                        pk_p[(16 * c + i + u) >> 1] = *reinterpret_cast<const uint32_t*>(&tp);
                        pk_ds[(16 * c + i + u) >> 1] = *reinterpret_cast<const uint32_t*>(&td);
                    }
                }
            }
            if (ok) ok = mbar_wait(p_empty, (j & 1) ^ 1, s_abort);   // the previous tile's products have read the operand tiles
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) continue;
            store_operand_half_row(smem_gen + (sPT - smem_base), row, half, pk_p);
            store_operand_half_row(smem_gen + (sdST - smem_base), row, half, pk_ds);
            fence_async_smem_bwd();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full);
        }
        if (J > 0) {
            if (ok) ok = mbar_wait(o_full, 0, s_abort);
            ok = __all_sync(0xffffffffu, ok);
        }
        const bool write = key < a.S;
        const size_t at = ((size_t)(row_base + (write ? key : 0)) * a.Hkv + kvh) * DH;
        bf16* outK = (pred ? a.dKp : a.dKt) + at;
        bf16* outV = (pred ? a.dVp : a.dVt) + at;
        if (J > 0 && ok) {
            fence_after();
            store_acc_row<DH>(tmem_base + 256 + lane_off, 1.f, outV, write, half * (DH / 2));
            store_acc_row<DH>(tmem_base + 256 + DH + lane_off, a.scale, outK, write, half * (DH / 2));
        } else if (write && half == 0) {
#pragma unroll
            for (int c0 = 0; c0 < DH; c0 += 8) {
                *reinterpret_cast<uint4*>(outK + c0) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(outV + c0) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
    }

    fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *s_abort && a.error_word != nullptr) atomicExch(a.error_word, 1);
    if (warp == 1) {
        fence_after();
        tmem_dealloc<kTmemCols>(tmem_base);
    }
}

// ------------------------------------------------------------------------------------------------
// Query side.  TMEM: two buffers of 128 columns (S, dP of 64 keys each) at 0 and 128, dQ at 256.
// ------------------------------------------------------------------------------------------------
template <int DH>
struct UBwdQSmem {
    static constexpr int kRes = kBM * DH * 2;           // Q (or dO) of the CTA's 128 queries
    static constexpr int kTile = kBS * DH * 2;          // a 64-key tile of K / V
    static constexpr int kOp = kBM * kBS * 2;           // dS operand tile
    static constexpr int kBytes = 2 * kRes + 4 * kTile + kTile + kOp + 1024 + 128;
};

template <int DH>
__global__ void __launch_bounds__(kBwdThreads, 1) attn_bwd_q_umma_kernel(const __grid_constant__ CUtensorMap tmQ128,
                                                                       const __grid_constant__ CUtensorMap tmdO128,
                                                                       const __grid_constant__ CUtensorMap tmK64,
                                                                       const __grid_constant__ CUtensorMap tmV64,
                                                                       const __grid_constant__ CUtensorMap tmKp64,
                                                                       const __grid_constant__ CUtensorMap tmVp64, const UBwdArgs a) {
    using SM = UBwdQSmem<DH>;
    constexpr int kHalves = DH / 64;
    constexpr uint32_t kTmemCols = 512;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQr = smem_base, sdOr = sQr + SM::kRes;
    const uint32_t sKV = sdOr + SM::kRes;                // stage s: K at sKV + 2 s kTile, V right after it
    const uint32_t sKT = sKV + 4 * SM::kTile, sdS = sKT + SM::kTile;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + 2 * SM::kRes + 5 * SM::kTile + SM::kOp);
    const uint32_t bar0 = smem_u32(bars);
    const uint32_t q_full = bar0, kv_full = bar0 + 8, kv_empty = bar0 + 24, t_full = bar0 + 40, t_empty = bar0 + 48;
    const uint32_t s_full = bar0 + 56, s_empty = bar0 + 72, p_full = bar0 + 88, p_empty = bar0 + 96, o_full = bar0 + 104;
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort_word;
    volatile int* s_abort = &s_abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qtile = gridDim.x - 1 - blockIdx.x;               // heaviest (latest) query tiles first
    const int h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (a.Hq / a.Hkv);
    const int q0 = qtile * kBM;
    const int row_base = b * a.S;

    const int p_last = min(q0 + kBM, a.S);
    const int n_max = nvis(p_last, a.block, a.offset);
    const int n_min = nvis(q0 + 1, a.block, a.offset);
    const int n_true_tiles = (n_max + kBS - 1) / kBS;
    const int band_lo_tile = n_min / kBS;
    const int band_hi = min(n_max + a.block - 1, a.S);
    const int n_pred_tiles = (a.step > 1 && band_hi > n_min) ? (band_hi + kBS - 1) / kBS - band_lo_tile : 0;
    const int J = n_true_tiles + n_pred_tiles;
    auto tile_of = [&](int j, bool& pred, int& kt) {
        pred = j >= n_true_tiles;
        kt = pred ? band_lo_tile + (j - n_true_tiles) : j;
    };

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(kv_full + 8 * s, 1); mbar_init(kv_empty + 8 * s, 1);
            mbar_init(s_full + 8 * s, 1); mbar_init(s_empty + 8 * s, 8);
        }
        mbar_init(t_full, 1); mbar_init(t_empty, 1);
        mbar_init(p_full, 8); mbar_init(p_empty, 1);
        mbar_init(o_full, 1);
        s_abort_word = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc<kTmemCols>(smem_u32(&s_tmem));
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem_base = s_tmem;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0 && J > 0) {
            mbar_expect_tx(q_full, 2 * SM::kRes);
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) {
                tma_load_2d(sQr + hf * (kBM * 128), &tmQ128, q_full, h * DH + hf * 64, row_base + q0);
                tma_load_2d(sdOr + hf * (kBM * 128), &tmdO128, q_full, h * DH + hf * 64, row_base + q0);
            }
            bool ok = true;
            int issued = 0;
            for (int j = 0; j < J && ok; ++j) {
                bool pred; int kt;
                tile_of(j, pred, kt);
                const int st = j & 1;
                ok = mbar_wait(kv_empty + 8 * st, ((j >> 1) & 1) ^ 1, s_abort);
                if (!ok) break;
                mbar_expect_tx(kv_full + 8 * st, 2 * SM::kTile);
                const uint32_t dK = sKV + st * 2 * SM::kTile, dV = dK + SM::kTile;
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    tma_load_2d(dK + hf * (kBS * 128), pred ? &tmKp64 : &tmK64, kv_full + 8 * st, kvh * DH + hf * 64, row_base + kt * kBS);
                    tma_load_2d(dV + hf * (kBS * 128), pred ? &tmVp64 : &tmV64, kv_full + 8 * st, kvh * DH + hf * 64, row_base + kt * kBS);
                }
                issued = j + 1;
                ok = mbar_wait(t_empty, (j & 1) ^ 1, s_abort);
                if (!ok) break;
                mbar_expect_tx(t_full, SM::kTile);
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf)      // the K tile once more, read by dQ += dS K as an MN-major operand
                    tma_load_2d(sKT + hf * (kBS * 128), pred ? &tmKp64 : &tmK64, t_full, kvh * DH + hf * 64, row_base + kt * kBS);
            }
            if (*s_abort) {
                for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(q_full, 0); ++i) {}
                for (int n = max(0, issued - 2); n < issued; ++n)
                    for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(kv_full + 8 * (n & 1), (n >> 1) & 1); ++i) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0 && J > 0) {
            constexpr uint32_t idesc_s = make_idesc(kBM, kBS), idesc_o = make_idesc_major(kBM, DH, false, true);
            bool ok = mbar_wait(q_full, 0, s_abort);
            auto issue_s = [&](int j) {
                const int st = j & 1;
                if (ok) ok = mbar_wait(kv_full + 8 * st, (j >> 1) & 1, s_abort);
                if (ok) ok = mbar_wait(s_empty + 8 * st, ((j >> 1) & 1) ^ 1, s_abort);
                if (!ok) return;
                fence_after();
                const uint32_t ts = tmem_base + st * 128;
                const uint32_t dK = sKV + st * 2 * SM::kTile, dV = dK + SM::kTile;
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    const uint64_t dq = umma_desc(sQr + hf * (kBM * 128)), dk = umma_desc(dK + hf * (kBS * 128));
                    const uint64_t dd = umma_desc(sdOr + hf * (kBM * 128)), dv = umma_desc(dV + hf * (kBS * 128));
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t koff = static_cast<uint64_t>((k * UMMA_K * 2) >> 4);
                        umma_bf16(ts, dq + koff, dk + koff, idesc_s, (hf > 0 || k > 0) ? 1u : 0u);            // S = Q K^T
                        umma_bf16(ts + kBS, dd + koff, dv + koff, idesc_s, (hf > 0 || k > 0) ? 1u : 0u);      // dP = dO V^T
                    }
                }
                umma_commit(kv_empty + 8 * st);
                umma_commit(s_full + 8 * st);
            };
            issue_s(0);
            for (int j = 0; j < J && ok; ++j) {
                if (j + 1 < J) issue_s(j + 1);
                if (!ok) break;
                ok = mbar_wait(p_full, j & 1, s_abort);
                if (ok) ok = mbar_wait(t_full, j & 1, s_abort);
                if (!ok) break;
                fence_after();
                const uint64_t dds = umma_desc(sdS), dkt = umma_desc_mn(sKT, kBS * 128);
#pragma unroll
                for (int k = 0; k < kBS / UMMA_K; ++k) {
                    const uint64_t koff = static_cast<uint64_t>((k * UMMA_K * 2) >> 4);
                    const uint64_t koff_mn = static_cast<uint64_t>((k * UMMA_K * 128) >> 4);
                    umma_bf16(tmem_base + 256, dds + koff, dkt + koff_mn, idesc_o, (j > 0 || k > 0) ? 1u : 0u);   // dQ += dS K
                }
                umma_commit(t_empty);
                umma_commit(p_empty);
            }
            umma_commit(o_full);
        }
    } else {
        // ---------------- one thread per query row
        const int q = warp & 3, half = (warp - 2) >> 2;
        const int row = q * 32 + lane;
        const int p1 = q0 + row + 1;
        const bool valid = p1 <= a.S;
        const int n_row = valid ? nvis(p1, a.block, a.offset) : 0;
        const int hi_row = valid ? n_row + min(p1 - n_row, a.step) - 1 : 0;
        const size_t stat_at = (size_t)(row_base + (valid ? p1 - 1 : 0)) * a.Hq + h;
        const float ls = valid ? a.lse2[stat_at] : 0.f, dl = valid ? a.delta[stat_at] : 0.f;
        const uint32_t lane_off = static_cast<uint32_t>(q * 32) << 16;
        bool ok = true;
        for (int j = 0; j < J; ++j) {
            const int st = j & 1;
            bool pred; int kt;
            tile_of(j, pred, kt);
            const int kt0 = kt * kBS;
            if (ok) ok = mbar_wait(s_full + 8 * st, (j >> 1) & 1, s_abort);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            fence_after();
            const bool full = valid && !pred && (kt0 + kBS <= n_min);
            const int lo = pred ? n_row : 0, hi = pred ? hi_row : n_row;
            uint32_t pk[16];
            const uint32_t ts = tmem_base + st * 128 + lane_off + 32 * half;
            uint32_t rs[2][16], rd[2][16];
#pragma unroll
            for (int c = 0; c < 2; ++c) { tmem_ld16(ts + 16 * c, rs[c]); tmem_ld16(ts + kBS + 16 * c, rd[c]); }
            tmem_ld_wait();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty + 8 * st);        // this warp's part of the buffer is in registers
#pragma unroll
            for (int c = 0; c < 2; ++c) {
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    float dv[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int key = kt0 + 32 * half + 16 * c + i + u;
                        float p = exp2f(fmaf(__uint_as_float(rs[c][i + u]), a.scale_log2, -ls));
                        if (!full) p = (key >= lo && key < hi) ? p : 0.f;
                        dv[u] = p * (__uint_as_float(rd[c][i + u]) - dl);
                    }
                    const __nv_bfloat162 td = __floats2bfloat162_rn(dv[0], dv[1]);
                    pk[(16 * c + i) >> 1] = *reinterpret_cast<const uint32_t*>(&td);
                }
            }
            if (ok) ok = mbar_wait(p_empty, (j & 1) ^ 1, s_abort);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            store_operand_half_row(smem_gen + (sdS - smem_base), row, half, pk);
            fence_async_smem_bwd();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full);
        }
        if (J > 0) {
            if (ok) ok = mbar_wait(o_full, 0, s_abort);
            ok = __all_sync(0xffffffffu, ok);
        }
        bf16* out = a.dQ + ((size_t)(row_base + (valid ? p1 - 1 : 0)) * a.Hq + h) * DH;
        if (J > 0 && ok) {
            fence_after();
            store_acc_row<DH>(tmem_base + 256 + lane_off, a.scale, out, valid, half * (DH / 2));
        } else if (valid && half == 0) {
#pragma unroll
            for (int c0 = 0; c0 < DH; c0 += 8) *reinterpret_cast<uint4*>(out + c0) = make_uint4(0u, 0u, 0u, 0u);
        }
    }

    fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *s_abort && a.error_word != nullptr) atomicExch(a.error_word, 1);
    if (warp == 1) {
        fence_after();
        tmem_dealloc<kTmemCols>(tmem_base);
    }
}

template <int DH>
int launch_ubwd(const CUtensorMap* m, const UBwdArgs& a, int B, int nz, cudaStream_t stream) {
    static PerDeviceOnce smem_attr;
    if (!smem_attr.ensure([] {
            return cudaFuncSetAttribute(attn_bwd_kv_umma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, UBwdKvSmem<DH>::kBytes) == cudaSuccess &&
                   cudaFuncSetAttribute(attn_bwd_q_umma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, UBwdQSmem<DH>::kBytes) == cudaSuccess;
        }))
        return -1;
    const int tiles = (a.S + kBM - 1) / kBM;
    // maps: 0 Q128, 1 dO128, 2 Q64, 3 dO64, 4 K128, 5 V128, 6 Kp128, 7 Vp128, 8 K64, 9 V64, 10 Kp64, 11 Vp64
    attn_bwd_q_umma_kernel<DH><<<dim3(tiles, a.Hq, B), kBwdThreads, UBwdQSmem<DH>::kBytes, stream>>>(m[0], m[1], m[8], m[9], m[10], m[11], a);
    attn_bwd_kv_umma_kernel<DH><<<dim3(tiles, a.Hkv, B * nz), kBwdThreads, UBwdKvSmem<DH>::kBytes, stream>>>(m[4], m[5], m[6], m[7], m[2], m[3], a, nz);
    return 2;
}

}  // namespace

int tc_attn_block_bwd_umma(TcPlan* p, const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp, const void* O, const void* dO,
                           const float* lse2, int B, int S, int Hq,
                           int Hkv, int dh, int block, int offset, int step, float* delta, void* dQ, void* dKt, void* dVt, void* dKp, void* dVp,
                           int* error_word, cudaStream_t stream) {
    if (p == nullptr || (dh != 64 && dh != 128) || B <= 0 || S <= 0 || 2 * B > 65535 || Hq > 65535) return -1;
    const long long rows = (long long)B * S, qd = (long long)Hq * dh, kd = (long long)Hkv * dh;
    CUtensorMap m[12];
    bool okm = true;
    okm = okm && tc_encode_map(p, &m[0], Q, rows, qd, qd, kBM) && tc_encode_map(p, &m[1], dO, rows, qd, qd, kBM);
    okm = okm && tc_encode_map(p, &m[2], Q, rows, qd, qd, kBS) && tc_encode_map(p, &m[3], dO, rows, qd, qd, kBS);
    const void* kv[4] = {Kt, Vt, Kp, Vp};
    for (int i = 0; i < 4; ++i) {
        okm = okm && tc_encode_map(p, &m[4 + i], kv[i], rows, kd, kd, kBM);
        okm = okm && tc_encode_map(p, &m[8 + i], kv[i], rows, kd, kd, kBS);
    }
    if (!okm) return -1;
    UBwdArgs a;
    a.S = S; a.Hq = Hq; a.Hkv = Hkv; a.block = block; a.offset = offset; a.step = step;
    a.scale = 1.0f / sqrtf((float)dh);
    a.scale_log2 = 1.4426950408889634f * a.scale;
    a.lse2 = lse2; a.delta = delta;
    a.dQ = static_cast<bf16*>(dQ);
    a.dKt = static_cast<bf16*>(dKt); a.dVt = static_cast<bf16*>(dVt); a.dKp = static_cast<bf16*>(dKp); a.dVp = static_cast<bf16*>(dVp);
    a.error_word = error_word;
    const long long pairs = rows * Hq;
    attn_delta_umma_kernel<<<(unsigned)((pairs * 32 + 255) / 256), 256, 0, stream>>>(static_cast<const bf16*>(dO), static_cast<const bf16*>(O), pairs,
                                                                                    dh, delta);
    const int nz = step > 1 ? 2 : 1;
    const int rc = dh == 128 ? launch_ubwd<128>(m, a, B, nz, stream) : launch_ubwd<64>(m, a, B, nz, stream);
    return rc < 0 ? rc : rc + 1;
}

}  // namespace beagle
