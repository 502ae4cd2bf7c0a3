// Block-masked cross-attention of the multi-token forward (Section 4.2) on tcgen05: both products of
// Eq. 2 (S = Q K^T and O = P V) run as tcgen05.mma with accumulators in tensor memory.
//
// One CTA = 128 consecutive query positions of one (sequence, query head): the 128 rows of an MMA
// tile, one TMEM lane and one softmax thread per query, so row maxima and row sums need no
// cross-thread reduction.  Keys are walked in tiles of 64 (true tiles up to the largest n(p) of the
// CTA, then the predicted band on the diagonal, as in the mma.sync kernel), once:
//   S = Q K^T per tile -> P = exp2(S - m) rounded to bf16 (row sums in fp32 over the unrounded weights), written to shared
//   memory in the MMA's operand layout -> O += P V accumulated in TMEM over all tiles, read once at the end,
//   normalised and stored.
// m is the row's reference point, not its running maximum: it is set by the row's first visible tile and moves only when a
// later tile exceeds it by more than 8 (a factor 256: harmless in bf16 and fp32).  Only then the accumulated O row and row sum
// are scaled by 2^(m_old - m_new) -- a read-modify-write of the warp's O rows in tensor memory, which a running maximum would
// ask for in almost every tile and which happens here a few times per row at most.  (An earlier form avoided the rescale by
// walking the keys twice, maxima first: a third more MMA work and twice the softmax-side work.)  With O resident in TMEM two
// CTAs fit an SM and overlap each other's softmax with MMAs.  V is read as it lies ([key][head_dim]: the B operand of P V in
// its MN-major form), so no transposed copy of the values is made.
//
// Roles: warp 0 = TMA producer (Q once; K and V tiles in two-stage rings of their own: a K slot is free once its S is
// complete, a V slot once its P V is),
// warp 1 = MMA issuer and TMEM owner (two S buffers of 64 columns + the O accumulator), warps 2-5 =
// softmax (warp w owns TMEM lanes 32 (w % 4) ..).  Every wait is bounded; a wait that runs out
// raises the error word, the CTA drains and frees its TMEM.
#include <cstring>

#include "gemm_tc.h"
#include "tc_plan.h"
#include "tc_ptx.cuh"

namespace beagle {

namespace {

using namespace tc;

constexpr int kUQ = 128, kUKey = 64, kUThreads = 192;

struct UmmaAttnArgs {
    int S, Hq, Hkv, block, offset, step;
    float scale_log2;
    bf16* O;            // [B*S, Hq*DH]
    float* lse2;        // optional [B*S, Hq]
    int* error_word;
};

__device__ __forceinline__ int vis_true(int p, int block, int offset) {      // n(p), p 1-based
    return (p <= offset) ? p - 1 : offset + block * ((p - 1 - offset) / block);
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <int DH>
struct UmmaAttnSmem {
    static constexpr int kQ = kUQ * DH * 2;             // DH/64 tiles of [128 x 64]
    static constexpr int kK = kUKey * DH * 2;           // DH/64 tiles of [64 keys x 64]
    static constexpr int kV = DH * kUKey * 2;           // DH/64 blocks of [64 keys x 64 dims]
    static constexpr int kP = kUQ * kUKey * 2;          // [128 x 64 keys]
    // Q, two K tiles, two V tiles, P, then 256 bytes of barriers and flags: 112.25 KB at head_dim 128, so that two CTAs share an
    // SM.  No slack for alignment: the kernel checks that its dynamic shared memory starts on a 1 KB boundary (it does when the
    // kernel has no static shared memory) and otherwise raises the error word instead of running.
    static constexpr int kBytes = kQ + 2 * kK + 2 * kV + kP + 256;
};

template <int DH>
__global__ void __launch_bounds__(kUThreads, 2) attn_block_umma_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                                     const __grid_constant__ CUtensorMap tmKt,
                                                                     const __grid_constant__ CUtensorMap tmVt,
                                                                     const __grid_constant__ CUtensorMap tmKp,
                                                                     const __grid_constant__ CUtensorMap tmVp, const UmmaAttnArgs a) {
    using SM = UmmaAttnSmem<DH>;
    constexpr int kHalves = DH / 64;
    constexpr uint32_t kTmemCols = 256;                  // S buffers at columns 0 and 64, O at 128 .. 128 + DH
    constexpr float kSlack = 8.f;                        // how far a tile's maximum may exceed the row's reference point before it moves
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t smem_base = smem_u32(smem_raw);
    if (smem_base & 1023u) {                                    // the swizzled tiles need 1 KB alignment: refuse rather than compute nonsense
        if (threadIdx.x == 0 && a.error_word != nullptr) atomicExch(a.error_word, 1);
        return;
    }
    uint8_t* smem_gen = smem_raw;
    const uint32_t sQ = smem_base, sK = sQ + SM::kQ, sV = sK + 2 * SM::kK, sP = sV + 2 * SM::kV;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + SM::kQ + 2 * SM::kK + 2 * SM::kV + SM::kP);
    const uint32_t bar0 = smem_u32(bars);
    const uint32_t q_full = bar0, k_full = bar0 + 8, k_empty = bar0 + 24, v_full = bar0 + 40, v_empty = bar0 + 56;
    const uint32_t s_full = bar0 + 72, s_empty = bar0 + 88, p_full = bar0 + 104, p_empty = bar0 + 112, o_full = bar0 + 120;
    uint32_t& s_tmem = *reinterpret_cast<uint32_t*>(bars + 16);
    int& s_abort_word = *reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(bars + 16) + 4);
    volatile int* s_abort = &s_abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qtile = gridDim.x - 1 - blockIdx.x;               // heaviest (latest) query tiles first
    const int h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (a.Hq / a.Hkv);
    const int q0 = qtile * kUQ;
    const int row_base = b * a.S;                               // rows of Q / K in the packed [B*S, .] matrices

    // key tiles this CTA visits (identical in every role)
    const int p_last = min(q0 + kUQ, a.S);
    const int n_max = vis_true(p_last, a.block, a.offset);
    const int n_min = vis_true(q0 + 1, a.block, a.offset);
    const int n_true_tiles = (n_max + kUKey - 1) / kUKey;
    const int band_lo_tile = n_min / kUKey;
    const int band_hi = min(n_max + a.block - 1, a.S);
    const int n_pred_tiles = (a.step > 1 && band_hi > n_min) ? (band_hi + kUKey - 1) / kUKey - band_lo_tile : 0;
    const int n_iter = n_true_tiles + n_pred_tiles;
    const int J = n_iter;                                       // one pass over the key tiles
    auto tile_of = [&](int j, bool& pred, int& kt) {
        pred = j >= n_true_tiles;
        kt = pred ? band_lo_tile + (j - n_true_tiles) : j;
    };

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(k_full + 8 * s, 1); mbar_init(k_empty + 8 * s, 1);
            mbar_init(s_full + 8 * s, 1); mbar_init(s_empty + 8 * s, 4);
            mbar_init(v_full + 8 * s, 1); mbar_init(v_empty + 8 * s, 1);
        }
        mbar_init(p_full, 4); mbar_init(p_empty, 1);
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
        if (lane == 0 && n_iter > 0) {
            mbar_expect_tx(q_full, SM::kQ);
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) tma_load_2d(sQ + hf * (kUQ * 128), &tmQ, q_full, h * DH + hf * 64, row_base + q0);
            bool ok = true;
            int k_issued = 0, v_issued = 0;
            for (int j = 0; j < J && ok; ++j) {
                bool pred; int kt;
                tile_of(j, pred, kt);
                const int st = j & 1;
                ok = mbar_wait(k_empty + 8 * st, ((j >> 1) & 1) ^ 1, s_abort);
                if (!ok) break;
                mbar_expect_tx(k_full + 8 * st, SM::kK);
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf)
                    tma_load_2d(sK + st * SM::kK + hf * (kUKey * 128), pred ? &tmKp : &tmKt, k_full + 8 * st, kvh * DH + hf * 64,
                                row_base + kt * kUKey);
                ++k_issued;
                ok = mbar_wait(v_empty + 8 * st, ((j >> 1) & 1) ^ 1, s_abort);
                if (!ok) break;
                mbar_expect_tx(v_full + 8 * st, SM::kV);
                // values as they lie, [key][head_dim]: an MN-major B operand, one box of 64 keys x 64 dims per 64 dims
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf)
                    tma_load_2d(sV + st * SM::kV + hf * (kUKey * 128), pred ? &tmVp : &tmVt, v_full + 8 * st, kvh * DH + hf * 64,
                                row_base + kt * kUKey);
                ++v_issued;
            }
            if (*s_abort) {      // copies already requested still land: wait (bounded) for the last of each buffer
                for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(q_full, 0); ++i) {}
                for (int n = max(0, k_issued - 2); n < k_issued; ++n)
                    for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(k_full + 8 * (n & 1), (n >> 1) & 1); ++i) {}
                for (int n = max(0, v_issued - 2); n < v_issued; ++n)
                    for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(v_full + 8 * (n & 1), (n >> 1) & 1); ++i) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0 && n_iter > 0) {
            constexpr uint32_t idesc_s = make_idesc(kUQ, kUKey), idesc_o = make_idesc_major(kUQ, DH, false, true);
            bool ok = mbar_wait(q_full, 0, s_abort);
            auto issue_s = [&](int j) {
                const int st = j & 1;
                if (ok) ok = mbar_wait(k_full + 8 * st, (j >> 1) & 1, s_abort);
                if (ok) ok = mbar_wait(s_empty + 8 * st, ((j >> 1) & 1) ^ 1, s_abort);      // the softmax has read S(j - 2)
                if (!ok) return;
                fence_after();
                const uint32_t ts = tmem_base + st * kUKey;
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    const uint64_t dq = umma_desc(sQ + hf * (kUQ * 128)), dk = umma_desc(sK + st * SM::kK + hf * (kUKey * 128));
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t koff = static_cast<uint64_t>((k * UMMA_K * 2) >> 4);
                        umma_bf16(ts, dq + koff, dk + koff, idesc_s, (hf > 0 || k > 0) ? 1u : 0u);
                    }
                }
                umma_commit(k_empty + 8 * st);
                umma_commit(s_full + 8 * st);
            };
            issue_s(0);
            for (int j = 0; j < J && ok; ++j) {
                if (j + 1 < J) issue_s(j + 1);               // S of the next tile runs under this tile's softmax
                if (ok) {
                    const int t2 = j;
                    ok = mbar_wait(p_full, t2 & 1, s_abort);
                    if (ok) ok = mbar_wait(v_full + 8 * (j & 1), (j >> 1) & 1, s_abort);
                    if (!ok) break;
                    fence_after();
                    const uint64_t dp = umma_desc(sP), dv = umma_desc_mn(sV + (j & 1) * SM::kV, kUKey * 128);
#pragma unroll
                    for (int k = 0; k < kUKey / UMMA_K; ++k) {
                        const uint64_t koff_p = static_cast<uint64_t>((k * UMMA_K * 2) >> 4);      // P: K-major, 32 bytes per step
                        const uint64_t koff_v = static_cast<uint64_t>((k * UMMA_K * 128) >> 4);    // V: 16 key rows of 128 bytes per step
                        umma_bf16(tmem_base + 2 * kUKey, dp + koff_p, dv + koff_v, idesc_o, (t2 > 0 || k > 0) ? 1u : 0u);
                    }
                    umma_commit(v_empty + 8 * (j & 1));
                    umma_commit(p_empty);
                }
            }
            umma_commit(o_full);
        }
    } else {
        // ---------------- softmax: thread = query row = TMEM lane
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const int p1 = q0 + row + 1;                              // 1-based position
        const bool valid = p1 <= a.S;
        const int n_row = valid ? vis_true(p1, a.block, a.offset) : 0;
        const int hi_row = valid ? n_row + min(p1 - n_row, a.step) - 1 : 0;
        const uint32_t lane_off = static_cast<uint32_t>(q * 32) << 16;
        float m_row = -INFINITY, l_row = 0.f;
        bool ok = true;
        for (int j = 0; j < J; ++j) {
            const int st = j & 1;
            bool pred; int kt;
            tile_of(j, pred, kt);
            const int kt0 = kt * kUKey;
            if (ok) ok = mbar_wait(s_full + 8 * st, (j >> 1) & 1, s_abort);
            ok = __all_sync(0xffffffffu, ok);                     // the TMEM loads are warp-collective
            if (!ok) break;
            fence_after();
            uint32_t r[4][16];
            const uint32_t ts = tmem_base + st * kUKey + lane_off;
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld16(ts + 16 * c, r[c]);
            tmem_ld_wait();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty + 8 * st);        // this warp's quarter of S is in registers
            // visible keys of this row in this tile: [lo, hi) (true tiles: [0, n(p)); predicted band: [n(p), hi(p)))
            const bool full = valid && !pred && (kt0 + kUKey <= n_min);   // a tile below every n(p) of the CTA: no mask
            const int lo = pred ? n_row : 0, hi = pred ? hi_row : n_row;  // an invalid row has lo = hi = 0
            // the tile's maximum of the masked scores (the positive scale is applied to the maximum)
            float mx = -INFINITY;
            if (full) {
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 16; ++i) mx = fmaxf(mx, __uint_as_float(r[c][i]));
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int key = kt0 + 16 * c + i;
                        mx = fmaxf(mx, (key >= lo && key < hi) ? __uint_as_float(r[c][i]) : -INFINITY);
                    }
            }
            mx *= a.scale_log2;
            // The row's reference point m only moves when a tile exceeds it by more than kSlack (in log2 units): the weights stay
            // below 2^kSlack, well inside bf16 and fp32, and the accumulated O row and row sum are then scaled by 2^(m_old - m_new).
            // A row's first tile with a visible key sets m (nothing has been accumulated for that row: factor 1).
            const float m_old = m_row;
            const bool grow = mx > m_old + kSlack;
            m_row = grow ? mx : m_old;
            const float factor = (grow && m_old != -INFINITY) ? exp2f(m_old - m_row) : 1.f;
            // P = exp2(S - m), rounded to bf16 for the MMA; the row sum is taken over the unrounded weights (fp32)
            uint32_t pk[32];
            const float neg_m = (m_row == -INFINITY) ? 0.f : -m_row;          // a row without keys has every weight masked below
            float l0 = 0.f, l1 = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    float p0 = exp2f(fmaf(__uint_as_float(r[c][i]), a.scale_log2, neg_m));
                    float p1v = exp2f(fmaf(__uint_as_float(r[c][i + 1]), a.scale_log2, neg_m));
                    if (!full) {
                        const int key = kt0 + 16 * c + i;
                        p0 = (key >= lo && key < hi) ? p0 : 0.f;
                        p1v = (key + 1 >= lo && key + 1 < hi) ? p1v : 0.f;
                    }
                    const __nv_bfloat162 t = __floats2bfloat162_rn(p0, p1v);
                    l0 += p0;
                    l1 += p1v;
                    pk[(16 * c + i) >> 1] = *reinterpret_cast<const uint32_t*>(&t);
                }
            l_row = fmaf(l_row, factor, l0 + l1);
            if (ok) ok = mbar_wait(p_empty, (j & 1) ^ 1, s_abort);           // the previous tile's P V has completed: O and the P buffer are free
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (__any_sync(0xffffffffu, factor != 1.f)) {
                // some row of this warp moved its reference point: scale the warp's 32 O rows in tensor memory (factor 1 elsewhere)
                fence_after();
#pragma unroll
                for (int c0 = 0; c0 < DH; c0 += 16) {
                    uint32_t ro[16];
                    tmem_ld16(tmem_base + 2 * kUKey + c0 + lane_off, ro);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) ro[i] = __float_as_uint(__uint_as_float(ro[i]) * factor);
                    tmem_st16(tmem_base + 2 * kUKey + c0 + lane_off, ro);
                }
                tmem_st_wait();
                fence_before();
            }
            // row `row` of the [128 x 64] operand tile: 16-byte chunk c at position c ^ (row & 7) (128-byte swizzle)
#pragma unroll
            for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4*>(smem_gen + (sP - smem_base) + row * 128 + ((c ^ (row & 7)) << 4)) =
                    make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            fence_async_smem();                              // generic-proxy writes -> visible to the MMA's async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full);
        }
        // ---- O from tensor memory, normalised, straight to global memory (one 2*DH-byte row per thread)
        if (n_iter > 0) {
            if (ok) ok = mbar_wait(o_full, 0, s_abort);
            ok = __all_sync(0xffffffffu, ok);
        }
        const float inv = (ok && l_row > 0.f) ? 1.f / l_row : 0.f;
        bf16* orow = a.O + ((size_t)(row_base + q0 + row) * a.Hq + h) * DH;
        if (n_iter > 0 && ok) {
            fence_after();
#pragma unroll
            for (int c0 = 0; c0 < DH; c0 += 32) {
                uint32_t ra[16], rb[16];
                tmem_ld16(tmem_base + 2 * kUKey + c0 + lane_off, ra);
                tmem_ld16(tmem_base + 2 * kUKey + c0 + 16 + lane_off, rb);
                tmem_ld_wait();
                if (valid) {
                    uint32_t o[16];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const __nv_bfloat162 t0 = __floats2bfloat162_rn(__uint_as_float(ra[2 * i]) * inv, __uint_as_float(ra[2 * i + 1]) * inv);
                        const __nv_bfloat162 t1 = __floats2bfloat162_rn(__uint_as_float(rb[2 * i]) * inv, __uint_as_float(rb[2 * i + 1]) * inv);
                        o[i] = *reinterpret_cast<const uint32_t*>(&t0);
                        o[8 + i] = *reinterpret_cast<const uint32_t*>(&t1);
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        *reinterpret_cast<uint4*>(orow + c0 + 8 * i) = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                }
            }
        } else if (valid) {
            // no visible key at all (or the CTA gave up): o = 0
#pragma unroll
            for (int c0 = 0; c0 < DH; c0 += 8) *reinterpret_cast<uint4*>(orow + c0) = make_uint4(0u, 0u, 0u, 0u);
        }
        if (a.lse2 != nullptr && valid)
            a.lse2[(size_t)(row_base + q0 + row) * a.Hq + h] = l_row > 0.f ? m_row + log2f(l_row) : 0.f;
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
int launch_umma_attn(const CUtensorMap* maps, const UmmaAttnArgs& a, dim3 grid, cudaStream_t stream) {
    using SM = UmmaAttnSmem<DH>;
    static PerDeviceOnce smem_attr;
    if (!smem_attr.ensure([] { return cudaFuncSetAttribute(attn_block_umma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::kBytes) == cudaSuccess; }))
        return -1;
    attn_block_umma_kernel<DH><<<grid, kUThreads, SM::kBytes, stream>>>(maps[0], maps[1], maps[2], maps[3], maps[4], a);
    return 1;
}

}  // namespace

int tc_attn_block_umma(TcPlan* p, const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp, int B, int S, int Hq,
                       int Hkv, int dh, int block, int offset, int step, void* O, int* error_word, cudaStream_t stream, float* lse2) {
    if (p == nullptr || (dh != 64 && dh != 128) || B <= 0 || S <= 0 || B > 65535 || Hq > 65535) return -1;
    const long long rows = (long long)B * S;
    CUtensorMap maps[5];
    if (!tc_encode_map(p, &maps[0], Q, rows, (long long)Hq * dh, (long long)Hq * dh, kUQ)) return -1;
    if (!tc_encode_map(p, &maps[1], Kt, rows, (long long)Hkv * dh, (long long)Hkv * dh, kUKey)) return -1;
    if (!tc_encode_map_mn(p, &maps[2], Vt, (long long)Hkv * dh, rows, (long long)Hkv * dh)) return -1;
    if (!tc_encode_map(p, &maps[3], Kp, rows, (long long)Hkv * dh, (long long)Hkv * dh, kUKey)) return -1;
    if (!tc_encode_map_mn(p, &maps[4], Vp, (long long)Hkv * dh, rows, (long long)Hkv * dh)) return -1;
    UmmaAttnArgs a;
    a.S = S; a.Hq = Hq; a.Hkv = Hkv; a.block = block; a.offset = offset; a.step = step;
    a.scale_log2 = 1.4426950408889634f / sqrtf((float)dh);
    a.O = static_cast<bf16*>(O);
    a.lse2 = lse2;
    a.error_word = error_word;
    dim3 grid((S + kUQ - 1) / kUQ, Hq, B);
    return dh == 128 ? launch_umma_attn<128>(maps, a, grid, stream) : launch_umma_attn<64>(maps, a, grid, stream);
}

}  // namespace beagle
