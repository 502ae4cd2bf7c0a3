// bf16 tensor-core GEMM for sm_100a: D[128 x BN] += A[128 x 64] * B[BN x 64]^T per k-block, both
// operands K-major in shared memory (128-byte swizzle, written by TMA), fp32 accumulators in TMEM,
// issued with tcgen05.mma by one thread.  Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and
// TMEM owner, warps 2..5 = epilogue (each reads its own quarter of the 128 TMEM lanes).
//
// Used by the dense projections of the block / prefill path: A = activations [M, K], B = weights
// [N, K]; epilogues: store, +residual, SiLU(g)*u (two accumulators), fp32 logits, packed arg-max
// keys, scatter into the K/V cache.
//
// The kernel is persistent: one CTA per SM walks over its tiles with the TMA ring running ahead
// across tile boundaries and two accumulator buffers in TMEM (512 columns), so the epilogue of
// a tile overlaps the MMAs of the next.
//
// Every wait on an mbarrier is bounded; a wait that runs out sets a device error word and the CTA
// drains and frees its TMEM instead of hanging.
#include <cuda.h>

#include <cstdio>
#include <cstring>

#include "gemm_tc.h"
#include "tc_plan.h"
#include "tc_ptx.cuh"

namespace beagle {

namespace {

using namespace tc;
constexpr int BM = 128;
constexpr int kTcThreads = 192;

// ---------------------------------------------------------------------------------------------- kernel
enum TcEpilogue {
    TC_STORE = 0, TC_RESID = 1, TC_SILU_MUL = 2, TC_F32 = 3, TC_KV_CACHE = 4, TC_ARGMAX = 5, TC_CE = 6, TC_DLOGITS = 7, TC_KV_PAIR = 8
};

struct TcArgs {
    int a_rows, b_rows, K;        // A: [a_rows, K]; B: [b_rows, K]
    int group_m;                  // rasterisation: A tiles per group
    int tiles_a, tiles_b;
    void* C; int ldc;
    const void* R; int ldr;
    void* cache; void* cache2; int Hkv, dh, cap;
    SeqRows rows;
    unsigned long long* keys; int keys_ld;
    const void* tgt; int tgt_dtype; int ldt; const int32_t* labels; float* ce_part;   // TC_CE, TC_DLOGITS
    const float* row_stats; const float* row_coef;                                    // TC_DLOGITS
    int* error_word;
};

template <int BN, bool DUAL, int EPI = TC_STORE>
struct TcSmem {
    static constexpr int kStageBytes = (BM + BN * (DUAL ? 2 : 1)) * BK * 2;
    static constexpr int kStages = (BN >= 128) ? 4 : 5;
    // TC_KV_PAIR: every epilogue warp transposes its 32 rows x BN columns through shared memory so that whole cache rows
    // leave the SM as contiguous 16-byte pieces
    static constexpr int kStagingBytes = (EPI == TC_KV_PAIR) ? BM * BN * 2 : 0;
    static constexpr int kBytes = kStages * kStageBytes + kStagingBytes + 1024 /*align*/ + 256 /*barriers*/;
};

template <int BN, bool DUAL, int EPI, bool AMN = false, bool BMN = false>
__global__ void __launch_bounds__(kTcThreads) tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA,
                                                            const __grid_constant__ CUtensorMap tmB,
                                                            const __grid_constant__ CUtensorMap tmB2, const TcArgs args) {
    using SM = TcSmem<BN, DUAL, EPI>;
    constexpr int kStages = SM::kStages;
    constexpr int kABytes = BM * BK * 2, kBBytes = BN * BK * 2;
    constexpr uint32_t kAccCols = DUAL ? 2 * BN : BN;       // TMEM columns of one tile's accumulator(s)
    constexpr uint32_t kTmemCols = 2 * kAccCols;            // two tiles in flight: the epilogue of one overlaps the MMAs of the next
    static_assert(kTmemCols == 512 || kTmemCols == 256 || kTmemCols == 128 || kTmemCols == 64, "TMEM allocation must be a power of two");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    uint8_t* smem_staging = smem_gen + kStages * SM::kStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_staging + SM::kStagingBytes);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * kStages;
    const uint32_t bar_acc_full = bar_empty + 8 * kStages, bar_acc_empty = bar_acc_full + 16;     // two accumulator buffers
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
    volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // Persistent CTA: tiles blockIdx.x, blockIdx.x + gridDim.x, ...  Consecutive tile ids walk down a
    // group of `group_m` row tiles before moving to the next column tile (L2 reuse of both operands).
    const int ntiles = args.tiles_a * args.tiles_b;
    auto tile_coords = [&](int pid, int& ta, int& tb) {
        const int per_group = args.group_m * args.tiles_b;
        const int g = pid / per_group;
        const int first = g * args.group_m;
        const int gsize = min(args.tiles_a - first, args.group_m);
        ta = first + (pid % per_group) % gsize;
        tb = (pid % per_group) / gsize;
    };
    const int nkb = (args.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar_acc_full + 8 * b, 1); mbar_init(bar_acc_empty + 8 * b, 4); }
        *s_abort = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc<kTmemCols>(smem_u32(s_tmem));
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem_base = *s_tmem;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            int issued = 0;                           // k-blocks requested so far, over all tiles
            bool ok = true;
            for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
                int ta, tb;
                tile_coords(t, ta, tb);
                for (int kb = 0; kb < nkb; ++kb) {
                    const int s = issued % kStages;
                    const uint32_t ph = (issued / kStages) & 1;
                    ok = mbar_wait(bar_empty + 8 * s, ph ^ 1, s_abort);
                    if (!ok) break;
                    const uint32_t sa = smem_base + s * SM::kStageBytes, sb = sa + kABytes;
                    mbar_expect_tx(bar_full + 8 * s, kABytes + kBBytes * (DUAL ? 2 : 1));
                    const int kc = kb * BK;
                    if (AMN) {      // the operand is stored [k][m]: one box of 64 k-rows x 64 m per 64 rows of the tile
#pragma unroll
                        for (int i = 0; i < BM / 64; ++i) tma_load_2d(sa + i * (BK * 128), &tmA, bar_full + 8 * s, ta * BM + 64 * i, kc);
                    } else {
                        tma_load_2d(sa, &tmA, bar_full + 8 * s, kc, ta * BM);
                    }
                    if (BMN) {
#pragma unroll
                        for (int i = 0; i < BN / 64; ++i) tma_load_2d(sb + i * (BK * 128), &tmB, bar_full + 8 * s, tb * BN + 64 * i, kc);
                    } else {
                        tma_load_2d(sb, &tmB, bar_full + 8 * s, kc, tb * BN);
                    }
                    if (DUAL) tma_load_2d(sb + kBBytes, &tmB2, bar_full + 8 * s, kc, tb * BN);
                    ++issued;
                }
            }
            if (*s_abort) {
                // drain: copies already issued still land in shared memory; wait (bounded) for the last of each stage
                for (int kb = max(0, issued - kStages); kb < issued; ++kb) {
                    const int s = kb % kStages;
                    const uint32_t ph = (kb / kStages) & 1;
                    for (uint32_t i = 0; i < kSpinLimit; ++i)
                        if (mbar_try_wait(bar_full + 8 * s, ph)) break;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            // gate and up tiles sit back to back in the stage (256 rows of 128 bytes), so one MMA of N = 2*BN
            // fills both accumulators and reads the A tile once
            constexpr uint32_t idesc = make_idesc_major(BM, DUAL ? 2 * BN : BN, AMN, BMN);
            bool ok = true;
            int consumed = 0, it = 0;
            for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x, ++it) {
                const int buf = it & 1;
                // the epilogue must have drained this accumulator buffer (two tiles ago)
                ok = mbar_wait(bar_acc_empty + 8 * buf, ((it >> 1) & 1) ^ 1, s_abort);
                if (!ok) break;
                fence_after();
                const uint32_t tacc = tmem_base + buf * kAccCols;
                for (int kb = 0; kb < nkb; ++kb) {
                    const int s = consumed % kStages;
                    const uint32_t ph = (consumed / kStages) & 1;
                    ok = mbar_wait(bar_full + 8 * s, ph, s_abort);
                    if (!ok) break;
                    fence_after();
                    const uint32_t sa = smem_base + s * SM::kStageBytes, sb = sa + kABytes;
                    const uint64_t da = AMN ? umma_desc_mn(sa, BK * 128) : umma_desc(sa);
                    const uint64_t db = BMN ? umma_desc_mn(sb, BK * 128) : umma_desc(sb);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                        // K-major: advance inside the swizzle atom (32 bytes per step); MN-major: 16 rows of 128 bytes per step
                        const uint64_t koff_a = static_cast<uint64_t>((AMN ? k * UMMA_K * 128 : k * UMMA_K * 2) >> 4);
                        const uint64_t koff_b = static_cast<uint64_t>((BMN ? k * UMMA_K * 128 : k * UMMA_K * 2) >> 4);
                        umma_bf16(tacc, da + koff_a, db + koff_b, idesc, acc);
                    }
                    umma_commit(bar_empty + 8 * s);   // frees the stage once these MMAs have read it
                    ++consumed;
                }
                umma_commit(bar_acc_full + 8 * buf);  // this tile's accumulators are complete (or the tile was abandoned)
            }
        }
    } else {
        // ---------------- epilogue: warp w reads TMEM lanes [32*(w%4), +32)
        const int q = warp & 3;
        const int row_in_tile = q * 32 + lane;
        int it = 0;
        for (int t = blockIdx.x; t < ntiles; t += gridDim.x, ++it) {
            int ta, tb;
            tile_coords(t, ta, tb);
            const int buf = it & 1;
            const int arow = ta * BM + row_in_tile;  // row of A this thread owns
            bool ok = mbar_wait(bar_acc_full + 8 * buf, (it >> 1) & 1, s_abort);
            ok = __all_sync(0xffffffffu, ok);        // the TMEM loads below are warp-collective
            if (!ok) break;
            fence_after();
            const uint32_t taddr = tmem_base + buf * kAccCols + (static_cast<uint32_t>(q * 32) << 16);
            if constexpr (EPI == TC_KV_PAIR) {
                // K (columns [0, BN) of the accumulator) then V ([BN, 2 BN)): bf16 rows through this warp's staging
                // block (16-byte pieces, XOR-swizzled by row so that neither side has bank conflicts), then out with
                // 16 lanes per cache row: one row's BN columns leave as contiguous 16-byte pieces.
                static_assert(BN == 128, "staging layout: 16 pieces of 16 bytes per row");
                uint8_t* stg = smem_staging + q * (32 * BN * 2);
                long long rowoff = -1;               // element offset of (slot, head 0, pos, 0) in a cache half; -1: row out of range
                if (arow < args.a_rows) {
                    int b = 0;
                    while (b + 1 < args.rows.n && arow >= args.rows.row_start[b + 1]) ++b;
                    const int pos = args.rows.pos_start[b] + (arow - args.rows.row_start[b]);
                    if (BEAGLE_IN_BOUNDS(pos >= 0 && pos < args.cap && BEAGLE_SLOT_OK(args.rows.slot[b])))
                        rowoff = ((long long)args.rows.slot[b] * args.Hkv * args.cap + pos) * args.dh;
                }
#pragma unroll 1
                for (int mat = 0; mat < 2; ++mat) {
                    __syncwarp();                    // the previous read-out of the staging block is complete
#pragma unroll 1
                    for (int c0 = 0; c0 < BN; c0 += 32) {
                        uint32_t ra[16], rb[16];
                        tmem_ld16(taddr + mat * BN + c0, ra);
                        tmem_ld16(taddr + mat * BN + c0 + 16, rb);
                        tmem_ld_wait();
                        uint32_t p[16];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            __nv_bfloat162 t = __floats2bfloat162_rn(__uint_as_float(ra[2 * j]), __uint_as_float(ra[2 * j + 1]));
                            p[j] = *reinterpret_cast<uint32_t*>(&t);
                            t = __floats2bfloat162_rn(__uint_as_float(rb[2 * j]), __uint_as_float(rb[2 * j + 1]));
                            p[8 + j] = *reinterpret_cast<uint32_t*>(&t);
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int piece = c0 / 8 + j;
                            *reinterpret_cast<uint4*>(stg + lane * (BN * 2) + ((piece ^ (lane & 15)) << 4)) =
                                make_uint4(p[4 * j], p[4 * j + 1], p[4 * j + 2], p[4 * j + 3]);
                        }
                    }
                    __syncwarp();
                    bf16* cache = reinterpret_cast<bf16*>(mat == 0 ? args.cache : args.cache2);
                    const int piece = lane & 15;
                    const int n = tb * BN + piece * 8;                  // first of this lane's 8 columns
                    const int head = n / args.dh, within = n - head * args.dh;
#pragma unroll 4
                    for (int i = 0; i < 16; ++i) {
                        const int r = 2 * i + (lane >> 4);
                        const long long off = __shfl_sync(0xffffffffu, rowoff, r);
                        const uint4 v = *reinterpret_cast<const uint4*>(stg + r * (BN * 2) + ((piece ^ (r & 15)) << 4));
                        if (off >= 0 && n < args.b_rows)
                            *reinterpret_cast<uint4*>(cache + off + (long long)head * args.cap * args.dh + within) = v;
                    }
                }
            } else {
                int m = arow;
                int slot = 0, pos = 0;
                if (EPI == TC_KV_CACHE && m < args.a_rows) {
                    int b = 0;
                    while (b + 1 < args.rows.n && m >= args.rows.row_start[b + 1]) ++b;
                    slot = args.rows.slot[b];
                    pos = args.rows.pos_start[b] + (m - args.rows.row_start[b]);
                    if (!BEAGLE_IN_BOUNDS(pos >= 0 && pos < args.cap && BEAGLE_SLOT_OK(slot))) m = args.a_rows;     // the row's stores are skipped
                }
                unsigned long long best = 0ull;
                float ce_mq = -INFINITY, ce_sq = 0.f, ce_mt = -INFINITY, ce_st = 0.f, ce_dot = 0.f;   // TC_CE running partial
                const int label = ((EPI == TC_CE || EPI == TC_DLOGITS) && args.tgt == nullptr && m < args.a_rows) ? args.labels[m] : -1;
                if (EPI == TC_CE && args.tgt == nullptr) ce_mt = 0.f;
                // TC_DLOGITS: the row's softmax statistics (max z, 1 / exp-sum z, max t, 1 / exp-sum t) and loss coefficient
                float dl_mq = 0.f, dl_iq = 0.f, dl_mt = 0.f, dl_it = 0.f, dl_coef = 0.f;
                if (EPI == TC_DLOGITS && m < args.a_rows) {
                    const float4 st = reinterpret_cast<const float4*>(args.row_stats)[m];
                    dl_mq = st.x; dl_iq = 1.0f / st.y; dl_mt = st.z; dl_it = args.tgt != nullptr ? 1.0f / st.w : 0.f;
                    dl_coef = args.row_coef[m];
                }
                // 16 accumulator columns of this thread's row (r, and r2 = the second matrix of a gated pair)
                auto consume = [&](const int c0, const uint32_t* r, const uint32_t* r2) {
                    const int n0 = tb * BN + c0;
                    if (m >= args.a_rows || n0 >= args.b_rows) return;
                    const bool full = (n0 + 16 <= args.b_rows);
                    if (EPI == TC_ARGMAX) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (n0 + j < args.b_rows) { const unsigned long long k = argmax_key(__uint_as_float(r[j]), n0 + j); best = k > best ? k : best; }
                    } else if (EPI == TC_CE) {
                        const int nv = min(16, args.b_rows - n0);
                        float cm = -INFINITY;
#pragma unroll
                        for (int j = 0; j < 16; ++j) if (j < nv) cm = fmaxf(cm, __uint_as_float(r[j]));
                        if (cm > ce_mq) { ce_sq *= __expf(ce_mq - cm); ce_mq = cm; }
#pragma unroll
                        for (int j = 0; j < 16; ++j) if (j < nv) ce_sq += __expf(__uint_as_float(r[j]) - ce_mq);
                        if (args.tgt != nullptr) {
                            float t[16];
                            if (args.tgt_dtype == 0) {
                                const float* tp = reinterpret_cast<const float*>(args.tgt) + (size_t)m * args.ldt + n0;
#pragma unroll
                                for (int j = 0; j < 16; ++j) t[j] = j < nv ? tp[j] : -INFINITY;
                            } else {
                                const bf16* tp = reinterpret_cast<const bf16*>(args.tgt) + (size_t)m * args.ldt + n0;
                                if (full && ((reinterpret_cast<uintptr_t>(tp) & 15) == 0)) {
                                    unpack16<bf16>(*reinterpret_cast<const uint4*>(tp), t);
                                    unpack16<bf16>(*reinterpret_cast<const uint4*>(tp + 8), t + 8);
                                } else {
#pragma unroll
                                    for (int j = 0; j < 16; ++j) t[j] = j < nv ? __bfloat162float(tp[j]) : -INFINITY;
                                }
                            }
                            float tm = -INFINITY;
#pragma unroll
                            for (int j = 0; j < 16; ++j) if (j < nv) tm = fmaxf(tm, t[j]);
                            if (tm > ce_mt) { const float f = __expf(ce_mt - tm); ce_st *= f; ce_dot *= f; ce_mt = tm; }
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                if (j < nv) { const float e = __expf(t[j] - ce_mt); ce_st += e; ce_dot = fmaf(e, __uint_as_float(r[j]), ce_dot); }
                        } else if (label >= n0 && label < n0 + nv) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) if (n0 + j == label) { ce_dot = __uint_as_float(r[j]); ce_st = 1.f; }
                        }
                    } else if (EPI == TC_F32) {
                        float* dst = reinterpret_cast<float*>(args.C) + (size_t)m * args.ldc + n0;
                        if (full && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                *reinterpret_cast<uint4*>(dst + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
                        } else {
                            for (int j = 0; j < 16 && n0 + j < args.b_rows; ++j) dst[j] = __uint_as_float(r[j]);
                        }
                    } else {
                        float v[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
                        if (EPI == TC_SILU_MUL) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) v[j] = silu_f(v[j]) * __uint_as_float(r2[j]);
                        }
                        if (EPI == TC_DLOGITS) {        // d z = coef * (softmax(z) - p)
                            const int nv = min(16, args.b_rows - n0);
                            float t[16];
                            if (args.tgt != nullptr) {
                                if (args.tgt_dtype == 0) {
                                    const float* tp = reinterpret_cast<const float*>(args.tgt) + (size_t)m * args.ldt + n0;
#pragma unroll
                                    for (int j = 0; j < 16; ++j) t[j] = j < nv ? tp[j] : -INFINITY;
                                } else {
                                    const bf16* tp = reinterpret_cast<const bf16*>(args.tgt) + (size_t)m * args.ldt + n0;
                                    if (full && ((reinterpret_cast<uintptr_t>(tp) & 15) == 0)) {
                                        unpack16<bf16>(*reinterpret_cast<const uint4*>(tp), t);
                                        unpack16<bf16>(*reinterpret_cast<const uint4*>(tp + 8), t + 8);
                                    } else {
#pragma unroll
                                        for (int j = 0; j < 16; ++j) t[j] = j < nv ? __bfloat162float(tp[j]) : -INFINITY;
                                    }
                                }
                            }
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float q = __expf(v[j] - dl_mq) * dl_iq;
                                const float pt = args.tgt != nullptr ? __expf(t[j] - dl_mt) * dl_it : (n0 + j == label ? 1.f : 0.f);
                                v[j] = dl_coef != 0.f ? dl_coef * (q - pt) : 0.f;
                            }
                        }
                        if (EPI == TC_RESID) {
                            const bf16* rp = reinterpret_cast<const bf16*>(args.R) + (size_t)m * args.ldr + n0;
                            if (full && ((reinterpret_cast<uintptr_t>(rp) & 15) == 0)) {
                                float f[8];
                                unpack16<bf16>(*reinterpret_cast<const uint4*>(rp), f);
#pragma unroll
                                for (int j = 0; j < 8; ++j) v[j] += f[j];
                                unpack16<bf16>(*reinterpret_cast<const uint4*>(rp + 8), f);
#pragma unroll
                                for (int j = 0; j < 8; ++j) v[8 + j] += f[j];
                            } else {
                                for (int j = 0; j < 16 && n0 + j < args.b_rows; ++j) v[j] += __bfloat162float(rp[j]);
                            }
                        }
                        bf16* dst;
                        if (EPI == TC_KV_CACHE)
                            dst = reinterpret_cast<bf16*>(args.cache) + (((size_t)slot * args.Hkv + n0 / args.dh) * args.cap + pos) * args.dh + n0 % args.dh;
                        else
                            dst = reinterpret_cast<bf16*>(args.C) + (size_t)m * args.ldc + n0;
                        if (full && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
                            uint32_t p[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                __nv_bfloat162 t = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
                                p[j] = *reinterpret_cast<uint32_t*>(&t);
                            }
                            *reinterpret_cast<uint4*>(dst) = make_uint4(p[0], p[1], p[2], p[3]);
                            *reinterpret_cast<uint4*>(dst + 8) = make_uint4(p[4], p[5], p[6], p[7]);
                        } else {
                            for (int j = 0; j < 16 && n0 + j < args.b_rows; ++j) {
                                if (EPI == TC_KV_CACHE) {
                                    const int n = n0 + j;
                                    reinterpret_cast<bf16*>(args.cache)[(((size_t)slot * args.Hkv + n / args.dh) * args.cap + pos) * args.dh + n % args.dh] = __float2bfloat16_rn(v[j]);
                                } else {
                                    dst[j] = __float2bfloat16_rn(v[j]);
                                }
                            }
                            if (EPI == TC_DLOGITS)      // the padded columns of the row (b_rows .. ldc - 1) read as zero
                                for (int j = 0; j < 16; ++j)
                                    if (n0 + j >= args.b_rows && n0 + j < args.ldc) dst[j] = __float2bfloat16_rn(0.f);
                        }
                    }
                };
                // two TMEM loads in flight per wait
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    uint32_t ra[16], rb[16], ra2[16], rb2[16];
                    __syncwarp();
                    tmem_ld16(taddr + c0, ra);
                    tmem_ld16(taddr + c0 + 16, rb);
                    if (DUAL) { tmem_ld16(taddr + BN + c0, ra2); tmem_ld16(taddr + BN + c0 + 16, rb2); }
                    tmem_ld_wait();
                    consume(c0, ra, ra2);
                    consume(c0 + 16, rb, rb2);
                }
                if (EPI == TC_ARGMAX && m < args.a_rows) args.keys[(size_t)m * args.keys_ld + tb] = best;
                if (EPI == TC_CE && m < args.a_rows) {
                    float* dst = args.ce_part + ((size_t)m * args.tiles_b + tb) * kCeFields;
                    dst[0] = ce_mq; dst[1] = ce_sq; dst[2] = ce_mt; dst[3] = ce_st; dst[4] = ce_dot;
                }
            }
            // this warp has read its quarter of the buffer: hand it back to the MMA issuer
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty + 8 * buf);
        }
    }

    fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *s_abort && args.error_word != nullptr) atomicExch(args.error_word, 1);
    if (warp == 1) {
        fence_after();
        tmem_dealloc<kTmemCols>(tmem_base);
    }
}

// Self-test of the bounded-wait protocol: one CTA waits, with a short poll limit, on an mbarrier that nothing will ever
// complete (no copy is in flight, no other role exists), gives up, raises the device error word exactly as the real
// kernels do after their limit, and returns.  Nothing hangs and nothing faults: the wait simply runs out.
__global__ void wait_timeout_selftest_kernel(int* error_word, uint32_t limit) {
    __shared__ uint64_t bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_barrier_init();
        const bool ok = mbar_wait_limit(smem_u32(&bar), 0, &s_abort, limit);
        if (!ok && s_abort && error_word != nullptr) atomicExch(error_word, 1);
    }
}

// Reduces the dense LM head's per-tile keys [rows, ntiles] to ids.
__global__ void tc_keys_to_ids_kernel(const unsigned long long* __restrict__ keys, int rows, int ntiles, int32_t* __restrict__ ids) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= rows) return;
    unsigned long long k = 0ull;
    for (int t = lane; t < ntiles; t += 32) { const unsigned long long o = keys[(size_t)warp * ntiles + t]; k = o > k ? o : k; }
    k = warp_max_u64(k);
    if (lane == 0) ids[warp] = argmax_key_index(k);
}

}  // namespace

bool tc_encode_map(TcPlan* p, CUtensorMap* out, const void* base, long long rows, long long K, long long ld, int box_rows) {
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    const CUresult r = p->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// An MN-major operand: stored [krows, feat] row-major (row stride ld elements); box = 64 features x 64 k-rows.
bool tc_encode_map_mn(TcPlan* p, CUtensorMap* out, const void* base, long long feat, long long krows, long long ld) {
    cuuint64_t dims[2] = {(cuuint64_t)feat, (cuuint64_t)krows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)BK};
    cuuint32_t estr[2] = {1, 1};
    const CUresult r = p->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool tc_encode_map_u8(TcPlan* p, CUtensorMap* out, const void* base, long long rows, long long K, long long ld, int box_rows) {
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld};
    cuuint32_t box[2] = {128u, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    const CUresult r = p->encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

const CUtensorMap* tc_weight_map_u8(TcPlan* p, const void* W, int rows, int K, int box_rows) {
    auto key = std::make_pair(W, box_rows);
    auto it = p->weight_maps.find(key);
    if (it != p->weight_maps.end()) return &it->second;
    CUtensorMap m;
    if (!tc_encode_map_u8(p, &m, W, rows, K, K, box_rows)) return nullptr;
    return &p->weight_maps.emplace(key, m).first->second;
}

const CUtensorMap* tc_weight_map(TcPlan* p, const void* W, int rows, int K, int box_rows) {
    auto key = std::make_pair(W, box_rows);
    auto it = p->weight_maps.find(key);
    if (it != p->weight_maps.end()) return &it->second;
    CUtensorMap m;
    if (!tc_encode_map(p, &m, W, rows, K, K, box_rows)) return nullptr;
    return &p->weight_maps.emplace(key, m).first->second;
}

namespace {

template <int BN, bool DUAL, int EPI, bool AMN = false, bool BMN = false>
int launch_tc(const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& b2, const TcArgs& args, dim3 grid, cudaStream_t stream) {
    using SM = TcSmem<BN, DUAL, EPI>;
    static PerDeviceOnce smem_attr;
    if (!smem_attr.ensure([] { return cudaFuncSetAttribute(tc_gemm_kernel<BN, DUAL, EPI, AMN, BMN>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::kBytes) == cudaSuccess; }))
        return -1;
    tc_gemm_kernel<BN, DUAL, EPI, AMN, BMN><<<grid, kTcThreads, SM::kBytes, stream>>>(a, b, b2, args);
    return 1;
}

}  // namespace

TcPlan* tc_plan_create(const beagle_config& cfg, const beagle_weights& w, int* hard_error) {
    if (hard_error) *hard_error = 0;
    if (cfg.dtype != BEAGLE_BF16) return nullptr;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
        cudaGetLastError();
        return nullptr;             // no device in this process (host-only use of the library)
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || fn == nullptr ||
        qres != cudaDriverEntryPointSuccess) {
        if (hard_error) *hard_error = 1;
        return nullptr;
    }
    TcPlan* p = new TcPlan();
    p->encode = reinterpret_cast<EncodeTiledFn>(fn);
    p->cfg = cfg;
    p->w = w;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
        p->sm_count = sms;
    return p;
}

void tc_plan_destroy(TcPlan* plan) { delete plan; }

int tc_gemm(TcPlan* p, int epi, const GemmArgs& g, cudaStream_t stream) {
    if (p == nullptr) return -1;
    if (g.lda % 8 || (!g.a_mn && !g.b_mn && g.K % 8)) return -1;   // TMA: 16-byte row pitch
    if (reinterpret_cast<uintptr_t>(g.A) & 15) return -1;
    if ((g.a_mn || g.b_mn) && epi != GEMM_STORE && epi != GEMM_RESID && epi != GEMM_F32) return -1;
    if (g.a_mn && !g.b_mn) return -1;                              // the forms in use: W transposed, or both
    const bool dual = (epi == GEMM_SILU_MUL || epi == GEMM_KV_CACHE_PAIR);
    const int BN = dual ? 128 : 256;
    CUtensorMap mapA;
    if (g.a_mn ? !tc_encode_map_mn(p, &mapA, g.A, g.M, g.K, g.lda) : !tc_encode_map(p, &mapA, g.A, g.M, g.K, g.lda, BM)) return -1;
    CUtensorMap transient;
    const CUtensorMap* mapB;
    if (g.b_mn) {
        if ((reinterpret_cast<uintptr_t>(g.W) & 15) || g.ldw % 8 || !tc_encode_map_mn(p, &transient, g.W, g.N, g.K, g.ldw)) return -1;
        mapB = &transient;
    } else if (g.w_transient) {
        if (dual || (reinterpret_cast<uintptr_t>(g.W) & 15) || !tc_encode_map(p, &transient, g.W, g.N, g.K, g.K, BN)) return -1;
        mapB = &transient;
    } else {
        mapB = tc_weight_map(p, g.W, g.N, g.K, BN);
    }
    const CUtensorMap* mapB2 = dual ? tc_weight_map(p, g.W2, g.N, g.K, BN) : mapB;
    if (mapB == nullptr || mapB2 == nullptr) return -1;
    TcArgs a;
    memset(&a, 0, sizeof(a));
    a.a_rows = g.M; a.b_rows = g.N; a.K = g.K;
    a.tiles_a = (g.M + BM - 1) / BM;
    a.tiles_b = (g.N + BN - 1) / BN;
    a.group_m = 16;
    a.C = g.C; a.ldc = g.ldc; a.R = g.R; a.ldr = g.ldr;
    a.cache = g.cache; a.cache2 = g.cache2; a.Hkv = g.Hkv; a.dh = g.dh; a.cap = g.cap; a.rows = g.rows;
    a.keys = g.keys; a.keys_ld = a.tiles_b;
    a.tgt = g.tgt; a.tgt_dtype = g.tgt_dtype; a.ldt = g.ldt; a.labels = g.labels; a.ce_part = g.ce_part;
    a.row_stats = g.row_stats; a.row_coef = g.row_coef;
    a.error_word = g.error_word;
    if (epi == GEMM_KV_CACHE && (g.dh % 16)) return -1;
    if (epi == GEMM_KV_CACHE_PAIR && ((g.dh % 8) || (g.N % 8) || g.cache == nullptr || g.cache2 == nullptr ||
                                      ((reinterpret_cast<uintptr_t>(g.cache) | reinterpret_cast<uintptr_t>(g.cache2)) & 15)))
        return -1;
    const int ntiles = a.tiles_a * a.tiles_b;
    dim3 grid(ntiles < p->sm_count ? ntiles : p->sm_count, 1, 1);        // persistent: one CTA per SM
    if (g.b_mn) {
        if (g.a_mn) return epi == GEMM_F32 ? launch_tc<256, false, TC_F32, true, true>(mapA, *mapB, *mapB, a, grid, stream) : -1;
        if (epi == GEMM_STORE) return launch_tc<256, false, TC_STORE, false, true>(mapA, *mapB, *mapB, a, grid, stream);
        if (epi == GEMM_RESID) return launch_tc<256, false, TC_RESID, false, true>(mapA, *mapB, *mapB, a, grid, stream);
        return -1;
    }
    switch (epi) {
        case GEMM_STORE: return launch_tc<256, false, TC_STORE>(mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_RESID: return launch_tc<256, false, TC_RESID>(mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_SILU_MUL: return launch_tc<128, true, TC_SILU_MUL>(mapA, *mapB, *mapB2, a, grid, stream);
        case GEMM_F32: return launch_tc<256, false, TC_F32>(mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_KV_CACHE: return launch_tc<256, false, TC_KV_CACHE>(mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_ARGMAX_KEYS: return launch_tc<256, false, TC_ARGMAX>(mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_CE: return launch_tc<256, false, TC_CE>(mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_DLOGITS: return launch_tc<256, false, TC_DLOGITS>(mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_KV_CACHE_PAIR: return launch_tc<128, true, TC_KV_PAIR>(mapA, *mapB, *mapB2, a, grid, stream);
        default: return -1;
    }
}

int launch_wait_timeout_selftest(int* error_word, cudaStream_t stream) {
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(error_word, 4096u);
    return 1;
}

int tc_argmax_tiles(int N) { return (N + 255) / 256; }

int tc_keys_to_ids(const unsigned long long* keys, int rows, int ntiles, int32_t* ids, cudaStream_t stream) {
    if (rows <= 0) return 0;
    tc_keys_to_ids_kernel<<<(rows * 32 + 255) / 256, 256, 0, stream>>>(keys, rows, ntiles, ids);
    return 1;
}

}  // namespace beagle
