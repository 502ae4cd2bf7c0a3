// bf16 tensor-core GEMM for sm_100a: D[128 x BN] += A[128 x 64] * B[BN x 64]^T per k-block, both
// operands K-major in shared memory (128-byte swizzle, written by TMA), fp32 accumulators in TMEM,
// issued with tcgen05.mma by one thread.  Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer and
// TMEM owner, warps 2..5 = epilogue (each reads its own quarter of the 128 TMEM lanes).
//
// Two uses of the same main loop:
//   * dense projections of the block / prefill path: A = activations [M, K], B = weights [N, K];
//     epilogues: store, +residual, SiLU(g)*u (two accumulators), fp32 logits, packed arg-max keys,
//     scatter into the K/V cache;
//   * serve-time projections for 9..64 rows ("swap-AB"): A = weights [N_out, K] so that the long
//     dimension fills the 128 MMA rows, B = the batch's activations [<=64, K]; K may be split over
//     blockIdx.z, each split writing fp32 partial sums that a finishing kernel reduces in a fixed
//     order (deterministic), or, for the LM head, logits and arg-max keys directly.
//
// Every wait on an mbarrier is bounded; a wait that runs out sets a device error word and the CTA
// drains and frees its TMEM instead of hanging.
#include <cuda.h>

#include <cstdio>
#include <cstring>
#include <map>

#include "gemm_tc.h"

namespace beagle {

namespace {

constexpr int BM = 128, BK = 64, UMMA_K = 16;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int kTcThreads = 192;

// ---------------------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait.  Returns false when it gave up (and raises the CTA's abort flag).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, uint64_t hint) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "l"(hint)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64 elements),
// 128-byte swizzled, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);   // start address, 16-byte units
    d |= static_cast<uint64_t>(1024u >> 4) << 32;              // stride between 8-row groups
    d |= static_cast<uint64_t>(1) << 46;                       // descriptor version of this architecture
    d |= static_cast<uint64_t>(2) << 61;                       // 128-byte swizzle
    return d;
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__host__ __device__ constexpr uint32_t make_idesc(int bn) {
    return (1u << 4)            // D: fp32
           | (1u << 7)          // A: bf16
           | (1u << 10)         // B: bf16
           | (static_cast<uint32_t>(bn >> 3) << 17) | (static_cast<uint32_t>(BM >> 4) << 24);   // K-major A and B
}

// ---------------------------------------------------------------------------------------------- kernel
enum TcEpilogue {
    TC_STORE = 0, TC_RESID = 1, TC_SILU_MUL = 2, TC_F32 = 3, TC_KV_CACHE = 4, TC_ARGMAX = 5,   // dense: rows = tile of A
    TC_SKINNY_PARTIAL = 6,   // swap-AB: fp32 partial sums [z][col][a_rows]
    TC_SKINNY_LOGITS = 7     // swap-AB LM head: logits[col][a_row] (optional) + arg-max keys [col][tile]
};

struct TcArgs {
    int a_rows, b_rows, K;        // A: [a_rows, K]; B: [b_rows, K]
    int kb_per_split;             // k-blocks of 64 per blockIdx.z slice
    int group_m;                  // rasterisation: A tiles per group (dense path)
    int tiles_a, tiles_b;
    void* C; int ldc;
    const void* R; int ldr;
    void* cache; int Hkv, dh, cap;
    SeqRows rows;
    unsigned long long* keys; int keys_ld;
    float* partial; int partial_cols;     // skinny: [z][partial_cols][a_rows]
    float* logits;
    int valid_cols;                        // skinny: batch rows actually used
    int a_rows_second;                     // skinny with two weight matrices: rows of each
    int* error_word;
};

template <int BN, bool DUAL>
struct TcSmem {
    static constexpr int kStageBytes = (BM + BN * (DUAL ? 2 : 1)) * BK * 2;
    static constexpr int kStages = (BN >= 128) ? 4 : 5;
    static constexpr int kBytes = kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;
};

template <int BN, bool DUAL, int EPI>
__global__ void __launch_bounds__(kTcThreads) tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA,
                                                            const __grid_constant__ CUtensorMap tmA2,
                                                            const __grid_constant__ CUtensorMap tmB,
                                                            const __grid_constant__ CUtensorMap tmB2, const TcArgs args) {
    using SM = TcSmem<BN, DUAL>;
    constexpr int kStages = SM::kStages;
    constexpr int kABytes = BM * BK * 2, kBBytes = BN * BK * 2;
    constexpr uint32_t kTmemCols = (DUAL ? 2 * BN : BN) < 32 ? 32 : (DUAL ? 2 * BN : BN);
    constexpr bool SKINNY = (EPI == TC_SKINNY_PARTIAL || EPI == TC_SKINNY_LOGITS);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + kStages * SM::kStageBytes);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * kStages, bar_acc = bar_empty + 8 * kStages;
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 1);
    volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // tile coordinates
    int ta, tb;
    if (SKINNY) {
        ta = blockIdx.x;
        tb = 0;
    } else {
        const int pid = blockIdx.x;
        const int per_group = args.group_m * args.tiles_b;
        const int g = pid / per_group;
        const int first = g * args.group_m;
        const int gsize = min(args.tiles_a - first, args.group_m);
        ta = first + (pid % per_group) % gsize;
        tb = (pid % per_group) / gsize;
    }
    const int second = (SKINNY && args.a_rows_second > 0 && blockIdx.y == 1) ? 1 : 0;   // second weight matrix
    const int kb0 = blockIdx.z * args.kb_per_split;
    const int kb_total = (args.K + BK - 1) / BK;
    const int nkb = max(0, min(args.kb_per_split, kb_total - kb0));

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            const CUtensorMap* mapA = second ? &tmA2 : &tmA;
            int issued = 0;
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % kStages;
                const uint32_t ph = (kb / kStages) & 1;
                if (!mbar_wait(bar_empty + 8 * s, ph ^ 1, s_abort)) break;
                const uint32_t sa = smem_base + s * SM::kStageBytes, sb = sa + kABytes;
                mbar_expect_tx(bar_full + 8 * s, kABytes + kBBytes * (DUAL ? 2 : 1));
                const int kc = (kb0 + kb) * BK;
                tma_load_2d(sa, mapA, bar_full + 8 * s, kc, ta * BM);
                tma_load_2d(sb, &tmB, bar_full + 8 * s, kc, tb * BN);
                if (DUAL) tma_load_2d(sb + kBBytes, &tmB2, bar_full + 8 * s, kc, tb * BN);
                ++issued;
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
            constexpr uint32_t idesc = make_idesc(BN);
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const int s = kb % kStages;
                const uint32_t ph = (kb / kStages) & 1;
                ok = mbar_wait(bar_full + 8 * s, ph, s_abort);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sa = smem_base + s * SM::kStageBytes, sb = sa + kABytes;
                const uint64_t da = umma_desc(sa), db = umma_desc(sb), db2 = umma_desc(sb + kBBytes);
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k) {
                    const uint32_t acc = (kb > 0 || k > 0) ? 1u : 0u;
                    const uint64_t koff = static_cast<uint64_t>((k * UMMA_K * 2) >> 4);   // advance inside the swizzle atom
                    umma_bf16(tmem_base, da + koff, db + koff, idesc, acc);
                    if (DUAL) umma_bf16(tmem_base + BN, da + koff, db2 + koff, idesc, acc);
                }
                umma_commit(bar_empty + 8 * s);       // frees the stage once these MMAs have read it
            }
            umma_commit(bar_acc);                     // accumulators complete (or nothing was issued)
        }
    } else {
        // ---------------- epilogue: warp w reads TMEM lanes [32*(w%4), +32)
        const int q = warp & 3;
        const int row_in_tile = q * 32 + lane;
        const int arow = ta * BM + row_in_tile;      // row of A this thread owns
        bool ok = true;
        if (nkb > 0) ok = mbar_wait(bar_acc, 0, s_abort);
        tc_fence_after();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        if (ok && nkb > 0) {
            if (SKINNY) {
                unsigned long long best = 0ull;
                const int feat = arow;                                  // output feature
                const int nrows_a = second ? args.a_rows_second : args.a_rows;
#pragma unroll
                for (int c0 = 0; c0 < BN; c0 += 16) {
                    uint32_t r[16];
                    __syncwarp();
                    tmem_ld16(taddr + c0, r);
                    tmem_ld_wait();
                    if (EPI == TC_SKINNY_PARTIAL) {
                        if (feat < nrows_a) {
                            float* dst = args.partial + ((size_t)(blockIdx.z * 2 + second) * args.partial_cols) * args.a_rows;
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                if (c0 + j < args.valid_cols) dst[(size_t)(c0 + j) * args.a_rows + feat] = __uint_as_float(r[j]);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int col = c0 + j;
                            if (col >= args.valid_cols) continue;           // uniform across the warp
                            const float v = __uint_as_float(r[j]);
                            unsigned long long key = feat < args.a_rows ? argmax_key(v, feat) : 0ull;
                            if (args.logits != nullptr && feat < args.a_rows) args.logits[(size_t)col * args.a_rows + feat] = v;
                            key = warp_max_u64(key);
                            if (lane == 0) atomicMax(&args.keys[(size_t)col * args.keys_ld + ta], key);   // 4 warps share one slot
                        }
                    }
                }
                (void)best;
            } else {
                const int m = arow;
                int slot = 0, pos = 0;
                if (EPI == TC_KV_CACHE && m < args.a_rows) {
                    int b = 0;
                    while (b + 1 < args.rows.n && m >= args.rows.row_start[b + 1]) ++b;
                    slot = args.rows.slot[b];
                    pos = args.rows.pos_start[b] + (m - args.rows.row_start[b]);
                }
                unsigned long long best = 0ull;
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 16) {
                    uint32_t r[16], r2[16];
                    __syncwarp();
                    tmem_ld16(taddr + c0, r);
                    if (DUAL) tmem_ld16(taddr + BN + c0, r2);
                    tmem_ld_wait();
                    const int n0 = tb * BN + c0;
                    if (m >= args.a_rows || n0 >= args.b_rows) continue;
                    const bool full = (n0 + 16 <= args.b_rows);
                    if (EPI == TC_ARGMAX) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (n0 + j < args.b_rows) { const unsigned long long k = argmax_key(__uint_as_float(r[j]), n0 + j); best = k > best ? k : best; }
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
                        }
                    }
                }
                if (EPI == TC_ARGMAX && m < args.a_rows) args.keys[(size_t)m * args.keys_ld + tb] = best;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *s_abort && args.error_word != nullptr) atomicExch(args.error_word, 1);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------- finishing kernels (serve path)
// Sums the fp32 split-K partials of one projection in a fixed order and applies its epilogue.
enum FinishMode { FIN_STORE = 0, FIN_RESID = 1, FIN_SILU_MUL = 2, FIN_KV = 3 };

struct FinishArgs {
    const float* partial;   // [z][2][cols][N]
    int splits, cols, N;
    int B;
    bf16* out; int ldo;
    const bf16* resid; int ldr;
    bf16* out2; int ld2; RowMap orow2;     // second copy (per-slot state)
    // fused RMSNorm of the result (optional): norm_out = out * rsqrt(mean(out^2)+eps) * gain
    bf16* norm_out; const bf16* gain; float eps; int do_norm;
    bf16* kcache; bf16* vcache; int Hkv, dh, cap; RowMap slot; RowMap pos;
};

template <int MODE>
__global__ void __launch_bounds__(256) tc_finish_kernel(const FinishArgs a) {
    const int b = blockIdx.x;
    const size_t zstride = (size_t)2 * a.cols * a.N;
    const float* p0 = a.partial + (size_t)b * a.N;                       // matrix 0
    const float* p1 = a.partial + ((size_t)a.cols + b) * a.N;            // matrix 1 (gate/up, K/V)
    float ss = 0.f;
    for (int n = threadIdx.x * 4; n < a.N; n += blockDim.x * 4) {
        float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
        for (int z = 0; z < a.splits; ++z) {
            const float4 t = *reinterpret_cast<const float4*>(p0 + z * zstride + n);
            s0.x += t.x; s0.y += t.y; s0.z += t.z; s0.w += t.w;
            if (MODE == FIN_SILU_MUL || MODE == FIN_KV) {
                const float4 u = *reinterpret_cast<const float4*>(p1 + z * zstride + n);
                s1.x += u.x; s1.y += u.y; s1.z += u.z; s1.w += u.w;
            }
        }
        float v[4] = {s0.x, s0.y, s0.z, s0.w};
        if (MODE == FIN_SILU_MUL) {
            v[0] = silu_f(s0.x) * s1.x; v[1] = silu_f(s0.y) * s1.y; v[2] = silu_f(s0.z) * s1.z; v[3] = silu_f(s0.w) * s1.w;
        }
        if (MODE == FIN_RESID) {
            const bf16* r = a.resid + (size_t)b * a.ldr + n;
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] += __bfloat162float(r[j]);
        }
        if (MODE == FIN_KV) {
            const int slot = a.slot.idx[b], pos = a.pos.idx[b];
            if (pos >= 0) {
                const float v1[4] = {s1.x, s1.y, s1.z, s1.w};
                const size_t at = (((size_t)slot * a.Hkv + n / a.dh) * a.cap + pos) * a.dh + n % a.dh;   // dh % 4 == 0
#pragma unroll
                for (int j = 0; j < 4; ++j) { a.kcache[at + j] = __float2bfloat16_rn(v[j]); a.vcache[at + j] = __float2bfloat16_rn(v1[j]); }
            }
        } else {
            bf16 o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) { o[j] = __float2bfloat16_rn(v[j]); const float f = __bfloat162float(o[j]); ss += f * f; }
            bf16* dst = a.out + (size_t)b * a.ldo + n;
#pragma unroll
            for (int j = 0; j < 4; ++j) dst[j] = o[j];
            if (a.out2 != nullptr) {
                bf16* d2 = a.out2 + (size_t)a.orow2.idx[b] * a.ld2 + n;
#pragma unroll
                for (int j = 0; j < 4; ++j) d2[j] = o[j];
            }
        }
    }
    if (MODE == FIN_RESID && a.norm_out != nullptr) {
        __shared__ float s_part[8];
        __shared__ float s_scale;
        ss = warp_sum(ss);
        if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
        __syncthreads();
        if (threadIdx.x == 0) {
            float t = 0.f;
            for (int w = 0; w < 8; ++w) t += s_part[w];
            s_scale = a.do_norm ? rsqrtf(t / (float)a.N + a.eps) : 1.0f;
        }
        __syncthreads();
        const float sc = s_scale;
        // each thread re-reads the values it wrote itself
        for (int n = threadIdx.x * 4; n < a.N; n += blockDim.x * 4) {
            const bf16* src = a.out + (size_t)b * a.ldo + n;
            bf16* dst = a.norm_out + (size_t)b * a.ldo + n;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float g = a.do_norm ? __bfloat162float(a.gain[n + j]) : 1.0f;
                dst[j] = __float2bfloat16_rn(__bfloat162float(src[j]) * sc * g);
            }
        }
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct TcPlan {
    EncodeTiledFn encode = nullptr;
    beagle_config cfg;
    beagle_weights w;
    std::map<std::pair<const void*, int>, CUtensorMap> weight_maps;   // (pointer, box rows) -> map
    bool attr_set = false;
};

namespace {

// K-major bf16 matrix [rows, K] (row stride ld elements), box = 64 columns x box_rows rows, 128-byte swizzle.
bool encode_map(TcPlan* p, CUtensorMap* out, const void* base, long long rows, long long K, long long ld, int box_rows) {
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    const CUresult r = p->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

const CUtensorMap* weight_map(TcPlan* p, const void* W, int rows, int K, int box_rows) {
    auto key = std::make_pair(W, box_rows);
    auto it = p->weight_maps.find(key);
    if (it != p->weight_maps.end()) return &it->second;
    CUtensorMap m;
    if (!encode_map(p, &m, W, rows, K, K, box_rows)) return nullptr;
    return &p->weight_maps.emplace(key, m).first->second;
}

template <int BN, bool DUAL, int EPI>
int launch_tc(const CUtensorMap& a, const CUtensorMap& a2, const CUtensorMap& b, const CUtensorMap& b2, const TcArgs& args, dim3 grid,
              cudaStream_t stream) {
    using SM = TcSmem<BN, DUAL>;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(tc_gemm_kernel<BN, DUAL, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::kBytes) != cudaSuccess) return -1;
        attr_done = true;
    }
    tc_gemm_kernel<BN, DUAL, EPI><<<grid, kTcThreads, SM::kBytes, stream>>>(a, a2, b, b2, args);
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
    return p;
}

void tc_plan_destroy(TcPlan* plan) { delete plan; }

int tc_gemm(TcPlan* p, int epi, const GemmArgs& g, cudaStream_t stream) {
    if (p == nullptr) return -1;
    if (g.K % 8 || g.lda % 8) return -1;                       // TMA: 16-byte row pitch
    if (reinterpret_cast<uintptr_t>(g.A) & 15) return -1;
    const bool dual = (epi == GEMM_SILU_MUL);
    const int BN = dual ? 128 : 256;
    CUtensorMap mapA;
    if (!encode_map(p, &mapA, g.A, g.M, g.K, g.lda, BM)) return -1;
    const CUtensorMap* mapB = weight_map(p, g.W, g.N, g.K, BN);
    const CUtensorMap* mapB2 = dual ? weight_map(p, g.W2, g.N, g.K, BN) : mapB;
    if (mapB == nullptr || mapB2 == nullptr) return -1;
    TcArgs a;
    memset(&a, 0, sizeof(a));
    a.a_rows = g.M; a.b_rows = g.N; a.K = g.K;
    a.kb_per_split = (g.K + BK - 1) / BK;
    a.tiles_a = (g.M + BM - 1) / BM;
    a.tiles_b = (g.N + BN - 1) / BN;
    a.group_m = 16;
    a.C = g.C; a.ldc = g.ldc; a.R = g.R; a.ldr = g.ldr;
    a.cache = g.cache; a.Hkv = g.Hkv; a.dh = g.dh; a.cap = g.cap; a.rows = g.rows;
    a.keys = g.keys; a.keys_ld = a.tiles_b;
    a.error_word = g.error_word;
    if (epi == GEMM_KV_CACHE && (g.dh % 16)) return -1;
    dim3 grid(a.tiles_a * a.tiles_b, 1, 1);
    switch (epi) {
        case GEMM_STORE: return launch_tc<256, false, TC_STORE>(mapA, mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_RESID: return launch_tc<256, false, TC_RESID>(mapA, mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_SILU_MUL: return launch_tc<128, true, TC_SILU_MUL>(mapA, mapA, *mapB, *mapB2, a, grid, stream);
        case GEMM_F32: return launch_tc<256, false, TC_F32>(mapA, mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_KV_CACHE: return launch_tc<256, false, TC_KV_CACHE>(mapA, mapA, *mapB, *mapB, a, grid, stream);
        case GEMM_ARGMAX_KEYS: return launch_tc<256, false, TC_ARGMAX>(mapA, mapA, *mapB, *mapB, a, grid, stream);
        default: return -1;
    }
}

int tc_argmax_tiles(int N) { return (N + 255) / 256; }

int tc_keys_to_ids(const unsigned long long* keys, int rows, int ntiles, int32_t* ids, cudaStream_t stream) {
    if (rows <= 0) return 0;
    tc_keys_to_ids_kernel<<<(rows * 32 + 255) / 256, 256, 0, stream>>>(keys, rows, ntiles, ids);
    return 1;
}

}  // namespace beagle
