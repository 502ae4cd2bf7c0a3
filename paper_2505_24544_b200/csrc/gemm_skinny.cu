// Serve-time projections for 9..64 batch rows on the tensor cores ("swap-AB"): the weight matrix
// [N, K] supplies the 128 rows of each tcgen05.mma, the batch's activations [B, K] its BN <= 64
// columns, so every weight byte crosses HBM exactly once per projection whatever the batch.
//
// One CTA = one 128-row weight tile x one slice of K.  Warp 0 streams the tile with TMA
// (128-byte swizzle, a ring of stages), warp 1 issues the MMAs into a TMEM accumulator of BN
// columns, warps 2..5 read the accumulator (thread = output feature, register j = batch row j)
// and either write fp32 partial sums [split][matrix][b][n] for the finishing kernel below or, for
// the LM head, logits and one packed arg-max key per (b, tile).  Shared memory is sized so that
// three CTAs share an SM: one CTA's prologue and epilogue hide behind the others' streams.
//
// Every wait on an mbarrier is bounded; a wait that runs out raises a device error word and the
// CTA drains its copies and frees its TMEM instead of hanging.
#include <cstring>

#include "gemm_tc.h"
#include "tc_plan.h"
#include "tc_ptx.cuh"

namespace beagle {

namespace {

using namespace tc;
constexpr int BM = 128;
constexpr int kSkThreads = 192;
constexpr int kCtaSlots = 296;          // CTAs the split policy aims at (two per SM on 148 SMs)
constexpr int kQkvCtaSlots = 444;       // the merged Q + K/V launch: three CTAs per SM fit, its clusters must all be resident at once
constexpr int kABytes = BM * BK * 2;

template <int BN>
struct SkSmem {
    static constexpr int kStageBytes = kABytes + BN * BK * 2;
    static constexpr int kStages = 3;            // 54-72 KB per CTA: three CTAs per SM, so a dependent launch finds a free slot to prefetch in
    static constexpr int kBytes = kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;   // 64 columns: 75 KB, still three CTAs per SM
};

struct SkArgs {
    int N, K, B;              // weight rows, reduction length, valid batch rows
    int nmat;                 // weight matrices (blockIdx.y)
    int kb_per_split;         // k-blocks of 64 per blockIdx.z slice
    float* partial;           // [split][nmat][B][N]
    float* logits;            // [B][N] or null
    unsigned long long* keys; // [B][gridDim.x]
    const float* w_scale;     // FP8 LM head: per weight row
    const float* x_scale;     // FP8 LM head: per batch row
    int packed;               // the weight maps describe tile-major copies: tile (ta, kb) is rows [(ta * kb_total + kb) * 128, +128)
    int* error_word;
};

// Arguments of a projection's epilogue: adds the fp32 split partials in a fixed order, then store /
// +residual / SiLU*mul / K,V cache scatter (and, in the finishing kernel, RMSNorm of the result).
struct FinishArgs {
    const float* partial;   // [splits][nmat][B][N]
    int splits, nmat, B, N;
    bf16* out; int ldo;
    const bf16* resid; int ldr;
    bf16* out2; int ld2; RowMap orow2;     // second copy (per-slot state)
    bf16* norm_out; const bf16* gain; float eps; int do_norm;   // RMSNorm of the stored result (optional)
    bf16* kcache; bf16* vcache; int Hkv, dh, cap; RowMap slot; RowMap pos;
};

// Cluster helpers (the fused variant runs the K splits of one tile as one thread-block cluster).
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t ra;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
    return v;
}

// VAR 0: fp32 split partials to global memory (a finishing kernel follows).  VAR 1: LM head (logits + keys).
// VAR 2: the CTAs that share a tile form a cluster (its K splits, or gate and up); each leaves its accumulator
// in its own shared memory and, after a cluster barrier, reduces one slice of the tile's rows over all CTAs'
// shared memory (distributed shared memory, fixed order) and applies the epilogue: no partials, no second kernel.
// FP8 (LM head only): both operands are FP8 E4M3 bytes with a scale per row; a 128-byte swizzle row then holds 128
// elements and one MMA reads 32 of them, the same bytes as in the bf16 case, so only the element coordinates of the
// copies, the MMA kind and the epilogue's scaling differ.
// The body takes this CTA's weight map, activation map, tile index `ta` and matrix index `mat` from its entry point.
template <int BN, int VAR, bool FP8>
__device__ __forceinline__ void sk_body(const CUtensorMap* mapW, const CUtensorMap* mapX, const SkArgs& args, const FinishArgs& fin,
                                        const int mode, const int ta, const int mat) {
    constexpr bool LOGITS = (VAR == 1), FUSED = (VAR == 2);
    using SM = SkSmem<BN>;
    constexpr int kStages = SM::kStages;
    constexpr uint32_t kTmemCols = BN < 32 ? 32 : BN;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + kStages * SM::kStageBytes);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * kStages, bar_acc = bar_empty + 8 * kStages;
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 1);
    volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
    unsigned long long* s_keys = reinterpret_cast<unsigned long long*>(smem_gen);     // [4][BN], over the ring: it is idle once the accumulator is complete

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int BKE = FP8 ? 2 * BK : BK;        // elements per 128-byte row of a tile
    const int kb_total = (args.K + BKE - 1) / BKE;
    const int kb0 = blockIdx.z * args.kb_per_split;
    const int nkb = max(0, min(args.kb_per_split, kb_total - kb0));

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc, 1);
        *s_abort = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc<kTmemCols>(smem_u32(s_tmem));
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem_base = *s_tmem;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            const uint64_t stream_once = policy_evict_first(), keep = policy_evict_last();
            // The weights do not depend on the previous kernel: fill the ring with weight tiles
            // while that kernel drains, then wait for it and add the activation tiles.
            const int npre = min(nkb, kStages);
            // row-major weights: the tile's 128 rows, 128 bytes at column kb of each; packed: one contiguous tile of 16 KB
            const int wx = args.packed ? 0 : BKE, wy0 = args.packed ? (ta * kb_total + kb0) * BM : ta * BM, wy = args.packed ? BM : 0;
            for (int kb = 0; kb < npre; ++kb) {
                mbar_expect_tx(bar_full + 8 * kb, SM::kStageBytes);
                tma_load_2d_hint(smem_base + kb * SM::kStageBytes, mapW, bar_full + 8 * kb, (kb0 + kb) * wx, wy0 + kb * wy, stream_once);
            }
            pdl_wait();
            for (int kb = 0; kb < npre; ++kb)
                tma_load_2d_hint(smem_base + kb * SM::kStageBytes + kABytes, mapX, bar_full + 8 * kb, (kb0 + kb) * BKE, 0, keep);
            int issued = npre;
            for (int kb = npre; kb < nkb; ++kb) {
                const int s = kb % kStages;
                const uint32_t ph = (kb / kStages) & 1;
                if (!mbar_wait(bar_empty + 8 * s, ph ^ 1, s_abort)) break;
                const uint32_t sa = smem_base + s * SM::kStageBytes, sb = sa + kABytes;
                mbar_expect_tx(bar_full + 8 * s, SM::kStageBytes);
                const int kc = (kb0 + kb) * BKE;
                tma_load_2d_hint(sa, mapW, bar_full + 8 * s, (kb0 + kb) * wx, wy0 + kb * wy, stream_once);
                tma_load_2d_hint(sb, mapX, bar_full + 8 * s, kc, 0, keep);
                ++issued;
            }
            if (*s_abort) {
                // copies already issued still land in shared memory: wait (bounded) for the last of each stage
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
            constexpr uint32_t idesc = FP8 ? make_idesc_e4m3(BM, BN) : make_idesc(BM, BN);
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % kStages;
                const uint32_t ph = (kb / kStages) & 1;
                if (!mbar_wait(bar_full + 8 * s, ph, s_abort)) break;
                fence_after();
                const uint32_t sa = smem_base + s * SM::kStageBytes, sb = sa + kABytes;
                const uint64_t da = umma_desc(sa), db = umma_desc(sb);
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k) {
                    const uint64_t koff = static_cast<uint64_t>((k * UMMA_K * 2) >> 4);   // advance inside the swizzle atom
                    if (FP8) umma_e4m3(tmem_base, da + koff, db + koff, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                    else umma_bf16(tmem_base, da + koff, db + koff, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                }
                umma_commit(bar_empty + 8 * s);       // frees the stage once these MMAs have read it
            }
            umma_commit(bar_acc);                     // accumulator complete (or nothing was issued)
        }
    } else {
        // ---------------- epilogue: warp w reads TMEM lanes [32*(w%4), +32)
        const int q = warp & 3;
        const int feat = ta * BM + q * 32 + lane;    // output feature owned by this thread
        pdl_wait();                                  // the buffers written below may still be read by the previous kernel
        bool ok = nkb > 0;
        if (ok) ok = mbar_wait(bar_acc, 0, s_abort);
        ok = __all_sync(0xffffffffu, ok);            // the TMEM loads below are warp-collective
        fence_after();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        if (ok) {
#pragma unroll
            for (int c0 = 0; c0 < BN; c0 += 16) {
                uint32_t r[16];
                __syncwarp();
                tmem_ld16(taddr + c0, r);
                tmem_ld_wait();
                if (FUSED) {
                    float* red = reinterpret_cast<float*>(smem_gen);     // [BN][128]: the ring is idle once the accumulator is complete
#pragma unroll
                    for (int j = 0; j < 16; ++j) red[(c0 + j) * BM + q * 32 + lane] = __uint_as_float(r[j]);
                } else if (!LOGITS) {
                    if (feat < args.N) {
                        float* dst = args.partial + ((size_t)(blockIdx.z * args.nmat + mat) * args.B) * args.N + feat;
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (c0 + j < args.B) dst[(size_t)(c0 + j) * args.N] = __uint_as_float(r[j]);
                    }
                } else if (c0 < args.B) {
                    // the 16 columns' keys first, then the five shuffle rounds over all of them at once: sixteen independent
                    // chains per round instead of sixteen reductions one after the other (each a chain of five shuffle latencies)
                    unsigned long long key[16];
                    const float ws = FP8 ? (feat < args.N ? args.w_scale[feat] : 0.f) : 1.f;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int col = c0 + j;
                        const bool live = col < args.B && feat < args.N;
                        float v = __uint_as_float(r[j]);
                        if (FP8) v *= ws * (col < args.B ? args.x_scale[col] : 0.f);
                        if (live && args.logits != nullptr) args.logits[(size_t)col * args.N + feat] = v;
                        key[j] = live ? argmax_key(v, feat) : 0ull;
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const unsigned long long other = __shfl_xor_sync(0xffffffffu, key[j], o);
                            key[j] = other > key[j] ? other : key[j];
                        }
                    }
                    if (lane == 0) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (c0 + j < args.B) s_keys[q * BN + c0 + j] = key[j];
                    }
                }
            }
        }
        if (FUSED && !ok) {                                               // an empty K slice (or an abandoned wait) adds nothing
            float* red = reinterpret_cast<float*>(smem_gen);
            for (int c = 0; c < BN; ++c) red[c * BM + q * 32 + lane] = 0.f;
        }
        if (LOGITS) {
            asm volatile("bar.sync 1, 128;" ::: "memory");                // the four epilogue warps only
            const int col = threadIdx.x - 64;
            if (ok && col < args.B) {
                unsigned long long key = s_keys[col];
#pragma unroll
                for (int w = 1; w < 4; ++w) { const unsigned long long o = s_keys[w * BN + col]; key = o > key ? o : key; }
                args.keys[(size_t)col * gridDim.x + ta] = key;
            }
        }
    }

    if (FUSED) {
        // every CTA of the cluster has its [BN][128] accumulator in shared memory; CTA r reduces rows [r*rows, +rows)
        __syncthreads();
        pdl_wait();
        cluster_sync_all();
        const bool pair = (mode == SK_SILU_MUL);                     // cluster = (gate, up); otherwise = the K splits
        const int csize = pair ? 2 : (int)gridDim.z;
        const int rank = (int)cluster_rank();
        const int rows = BM / csize;
        const uint32_t red0 = smem_base;
        const int me = pair ? 0 : mat;                               // K/V: this cluster's matrix
        for (int idx = threadIdx.x; idx < rows * args.B; idx += kSkThreads) {
            const int rl = idx % rows, col = idx / rows;
            const int row = rank * rows + rl, n = ta * BM + row;
            if (n >= args.N) continue;
            const uint32_t la = red0 + (uint32_t)(col * BM + row) * 4u;
            float v = 0.f, v1 = 0.f;
            if (pair) { v = ld_cluster_f32(la, 0); v1 = ld_cluster_f32(la, 1); }
            else { for (int z = 0; z < csize; ++z) v += ld_cluster_f32(la, (uint32_t)z); }
            if (mode == SK_SILU_MUL) {
                fin.out[(size_t)col * fin.ldo + n] = __float2bfloat16_rn(silu_f(v) * v1);
            } else if (mode == SK_KV) {
                const int pos = fin.pos.idx[col];
                if (pos >= 0 && BEAGLE_IN_BOUNDS(pos < fin.cap && BEAGLE_SLOT_OK(fin.slot.idx[col]))) {
                    bf16* cache = me ? fin.vcache : fin.kcache;
                    cache[(((size_t)fin.slot.idx[col] * fin.Hkv + n / fin.dh) * fin.cap + pos) * fin.dh + n % fin.dh] = __float2bfloat16_rn(v);
                }
            } else {
                if (mode == SK_RESID) v += __bfloat162float(fin.resid[(size_t)col * fin.ldr + n]);
                const bf16 o = __float2bfloat16_rn(v);
                fin.out[(size_t)col * fin.ldo + n] = o;
                if (fin.out2 != nullptr) fin.out2[(size_t)fin.orow2.idx[col] * fin.ld2 + n] = o;
            }
        }
        cluster_sync_all();                                          // nobody leaves while its shared memory is being read
    }
    fence_before();
    __syncthreads();
    pdl_wait();                                      // every thread, so that this grid's completion implies its predecessors'
    if (threadIdx.x == 0 && *s_abort && args.error_word != nullptr) atomicExch(args.error_word, 1);
    if (warp == 1) {
        fence_after();
        tmem_dealloc<kTmemCols>(tmem_base);
    }
}

template <int BN, int VAR, bool FP8>
__global__ void __launch_bounds__(kSkThreads, 3) tc_skinny_kernel(const __grid_constant__ CUtensorMap tmW,
                                                               const __grid_constant__ CUtensorMap tmW2,
                                                               const __grid_constant__ CUtensorMap tmX, const SkArgs args,
                                                               const FinishArgs fin, const int mode) {
    sk_body<BN, VAR, FP8>(blockIdx.y ? &tmW2 : &tmW, &tmX, args, fin, mode, blockIdx.x, blockIdx.y);
}

// Two projections of one draft step in ONE launch (cluster variant): tiles [0, q_tiles) of blockIdx.x are the query projection
// (W_q on the normalised embeddings, stored), the next kv_tiles the key and the last kv_tiles the value projection of the
// previous step's states (written to the cache).  Same reduction length, same K slices, one kernel boundary fewer.
template <int BN>
__global__ void __launch_bounds__(kSkThreads) tc_skinny_qkv_kernel(const __grid_constant__ CUtensorMap tmWq,
                                                                   const __grid_constant__ CUtensorMap tmWk,
                                                                   const __grid_constant__ CUtensorMap tmWv,
                                                                   const __grid_constant__ CUtensorMap tmXq,
                                                                   const __grid_constant__ CUtensorMap tmXkv, const SkArgs args,
                                                                   const FinishArgs fin, const int q_tiles, const int kv_tiles,
                                                                   const int kv_N) {
    const int x = blockIdx.x;
    const bool kv = x >= q_tiles;
    const int mat = kv ? (x - q_tiles) / kv_tiles : 0;
    const int ta = kv ? (x - q_tiles) % kv_tiles : x;
    SkArgs a = args;
    if (kv) a.N = kv_N;
    sk_body<BN, 2, false>(kv ? (mat ? &tmWv : &tmWk) : &tmWq, kv ? &tmXkv : &tmXq, a, fin, kv ? (int)SK_KV : (int)SK_STORE, ta, mat);
}

// ---------------------------------------------------------------------------------------------- finishing kernel
// Adds the fp32 split partials of one projection in a fixed order and applies its epilogue.

constexpr int kFinThreads = 256;             // whole-row mode (fused RMSNorm)
constexpr int kFinColThreads = 64;           // column mode: many small CTAs, one float4 per thread
constexpr int kFinCols = kFinColThreads * 4; // features per CTA in column mode

template <int MODE>
__global__ void __launch_bounds__(kFinThreads) tc_finish_kernel(const FinishArgs a) {
    const int b = blockIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    const size_t mstride = (size_t)a.B * a.N;
    const size_t zstride = mstride * a.nmat;
    const float* p0 = a.partial + (size_t)b * a.N;
    const float* p1 = p0 + mstride;                 // second matrix (gate/up, K/V)
    const bool whole_row = (MODE == SK_RESID && a.norm_out != nullptr);
    const int n_begin = whole_row ? 0 : blockIdx.y * kFinCols;
    const int n_end = whole_row ? a.N : min(a.N, n_begin + kFinCols);
    float ss = 0.f;
    for (int n = n_begin + threadIdx.x * 4; n < n_end; n += kFinThreads * 4) {     // N is a multiple of 4
        float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
        constexpr bool kTwo = (MODE == SK_SILU_MUL || MODE == SK_KV);
        for (int z0 = 0; z0 < a.splits; z0 += 8) {                 // all loads of a group first, then the adds in split order
            float4 t[8], u[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const bool in = z0 + j < a.splits;
                t[j] = in ? *reinterpret_cast<const float4*>(p0 + (size_t)(z0 + j) * zstride + n) : make_float4(0.f, 0.f, 0.f, 0.f);
                if (kTwo) u[j] = in ? *reinterpret_cast<const float4*>(p1 + (size_t)(z0 + j) * zstride + n) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                s0.x += t[j].x; s0.y += t[j].y; s0.z += t[j].z; s0.w += t[j].w;
                if (kTwo) { s1.x += u[j].x; s1.y += u[j].y; s1.z += u[j].z; s1.w += u[j].w; }
            }
        }
        float v[4] = {s0.x, s0.y, s0.z, s0.w};
        if (MODE == SK_SILU_MUL) {
            v[0] = silu_f(s0.x) * s1.x; v[1] = silu_f(s0.y) * s1.y; v[2] = silu_f(s0.z) * s1.z; v[3] = silu_f(s0.w) * s1.w;
        }
        if (MODE == SK_RESID) {
            const bf16* r = a.resid + (size_t)b * a.ldr + n;
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] += __bfloat162float(r[j]);
        }
        if (MODE == SK_KV) {
            const int slot = a.slot.idx[b], pos = a.pos.idx[b];
            if (pos >= 0 && BEAGLE_IN_BOUNDS(pos < a.cap && BEAGLE_SLOT_OK(slot))) {
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
    if (whole_row) {
        __shared__ float s_part[kFinThreads / 32];
        __shared__ float s_scale;
        ss = warp_sum(ss);
        if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
        __syncthreads();
        if (threadIdx.x == 0) {
            float t = 0.f;
            for (int w = 0; w < kFinThreads / 32; ++w) t += s_part[w];
            s_scale = a.do_norm ? rsqrtf(t / (float)a.N + a.eps) : 1.0f;
        }
        __syncthreads();
        const float sc = s_scale;
        // each thread re-reads the values it wrote itself
        for (int n = threadIdx.x * 4; n < a.N; n += kFinThreads * 4) {
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

// ---------------------------------------------------------------------------------------------- tile-major weight copies
// One thread per 16-byte piece of the destination: tile t = ta * kb_total + kb holds rows [128 ta, +128) x bytes [128 kb, +128)
// of the source, row r of the tile at 128 r inside it; pieces outside the matrix are zero.
__global__ void __launch_bounds__(256) pack_tiles_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, const int N,
                                                         const long long row_bytes, const int kb_total, const long long pieces) {
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    if (idx >= pieces) return;
    const int c = (int)(idx & 7), r = (int)((idx >> 3) & 127);
    const long long t = idx >> 10;
    const int kb = (int)(t % kb_total);
    const long long row = (t / kb_total) * BM + r, byte = (long long)kb * 128 + c * 16;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row < N && byte < row_bytes) v = src[(row * row_bytes + byte) >> 4];
    dst[idx] = v;
}

struct SplitPlan { int tiles, kb_total, kb_per_split, splits; };
SplitPlan split_plan(int N, int K, int nmat, bool allow_split) {
    SplitPlan s;
    s.tiles = (N + BM - 1) / BM;
    s.kb_total = (K + BK - 1) / BK;
    int want = allow_split ? kCtaSlots / (s.tiles * nmat) : 1;
    if (want < 1) want = 1;
    s.kb_per_split = (s.kb_total + want - 1) / want;
    if (s.kb_per_split < 4) s.kb_per_split = s.kb_total < 4 ? s.kb_total : 4;
    s.splits = (s.kb_total + s.kb_per_split - 1) / s.kb_per_split;
    return s;
}

template <int BN, int VAR, bool FP8 = false>
int launch_sk(const CUtensorMap& w, const CUtensorMap& w2, const CUtensorMap& x, const SkArgs& args, const FinishArgs& fin, int mode,
              dim3 grid, dim3 cluster, cudaStream_t stream) {
    using SM = SkSmem<BN>;
    static PerDeviceOnce smem_attr;
    if (!smem_attr.ensure([] { return cudaFuncSetAttribute(tc_skinny_kernel<BN, VAR, FP8>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::kBytes) == cudaSuccess; }))
        return -1;
    if (VAR != 2) {
        launch_pdl(tc_skinny_kernel<BN, VAR, FP8>, grid, dim3(kSkThreads), SM::kBytes, stream, w, w2, x, args, fin, mode);
        return 1;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(kSkThreads); cfg.dynamicSmemBytes = SM::kBytes; cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster.x; attr[0].val.clusterDim.y = cluster.y; attr[0].val.clusterDim.z = cluster.z;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, tc_skinny_kernel<BN, VAR, FP8>, w, w2, x, args, fin, mode) != cudaSuccess) {
        cudaGetLastError();
        return -1;                                   // the caller falls back to partials + finishing kernel
    }
    return 1;
}

template <int VAR>
int launch_sk_bn(int bn, const CUtensorMap& w, const CUtensorMap& w2, const CUtensorMap& x, const SkArgs& args, const FinishArgs& fin, int mode,
                 dim3 grid, dim3 cluster, cudaStream_t stream) {
    switch (bn) {
        case 16: return launch_sk<16, VAR>(w, w2, x, args, fin, mode, grid, cluster, stream);
        case 32: return launch_sk<32, VAR>(w, w2, x, args, fin, mode, grid, cluster, stream);
        default: return launch_sk<64, VAR>(w, w2, x, args, fin, mode, grid, cluster, stream);
    }
}

template <int BN>
int launch_sk_qkv(const CUtensorMap& wq, const CUtensorMap& wk, const CUtensorMap& wv, const CUtensorMap& xq, const CUtensorMap& xkv,
                  const SkArgs& args, const FinishArgs& fin, int q_tiles, int kv_tiles, int kv_N, int cs, cudaStream_t stream) {
    using SM = SkSmem<BN>;
    static PerDeviceOnce smem_attr;
    if (!smem_attr.ensure([] { return cudaFuncSetAttribute(tc_skinny_qkv_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::kBytes) == cudaSuccess; }))
        return -1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(q_tiles + 2 * kv_tiles, 1, cs); cfg.blockDim = dim3(kSkThreads); cfg.dynamicSmemBytes = SM::kBytes; cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = cs;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, tc_skinny_qkv_kernel<BN>, wq, wk, wv, xq, xkv, args, fin, q_tiles, kv_tiles, kv_N) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    return 1;
}

}  // namespace

size_t tc_skinny_packed_bytes(int N, int K, int elt_bytes) {
    const size_t tiles = (N + BM - 1) / BM, kb_total = ((size_t)K * elt_bytes + 127) / 128;
    return tiles * kb_total * (size_t)(BM * 128);
}

int tc_skinny_pack(TcPlan* p, const void* W, int N, int K, int elt_bytes, void* dst, cudaStream_t stream) {
    if (p == nullptr || W == nullptr) return -1;
    p->packed.erase(W);
    if (dst == nullptr) return 0;
    const long long row_bytes = (long long)K * elt_bytes;
    if ((elt_bytes != 1 && elt_bytes != 2) || N <= 0 || K <= 0 || row_bytes % 16 || (reinterpret_cast<uintptr_t>(W) & 15) ||
        (reinterpret_cast<uintptr_t>(dst) & 127))
        return -1;
    const int kb_total = (int)((row_bytes + 127) / 128);
    const long long rows = (long long)((N + BM - 1) / BM) * kb_total * BM, pieces = rows * 8;
    if (rows > 0x7fffffffLL) return -1;                    // the tile's first row is a 32-bit TMA coordinate
    TcPlan::Packed e;
    e.tiles = dst; e.N = N; e.K = K; e.elt_bytes = elt_bytes;
    // the copy as a matrix of `rows` rows of 128 bytes: a box of 128 rows is one tile
    const bool ok = elt_bytes == 2 ? tc_encode_map(p, &e.map, dst, rows, BK, BK, BM) : tc_encode_map_u8(p, &e.map, dst, rows, 128, 128, BM);
    if (!ok) return -1;
    pack_tiles_kernel<<<(unsigned)((pieces + 255) / 256), 256, 0, stream>>>(static_cast<const uint4*>(W), static_cast<uint4*>(dst), N, row_bytes,
                                                                            kb_total, pieces);
    if (cudaGetLastError() != cudaSuccess) return -1;
    p->packed.emplace(W, e);
    return 1;
}

void tc_skinny_forget_packed(TcPlan* p) {
    if (p != nullptr) p->packed.clear();
}

namespace {
// The tile-major copy's map when W [N, K] has one, else nullptr.
const CUtensorMap* packed_map(TcPlan* p, const void* W, int N, int K, int elt_bytes) {
    auto it = p->packed.find(W);
    if (it == p->packed.end() || it->second.N != N || it->second.K != K || it->second.elt_bytes != elt_bytes) return nullptr;
    return &it->second.map;
}
}  // namespace

int tc_skinny_qkv(TcPlan* p, const SkinnyArgs& q, const SkinnyArgs& kv, cudaStream_t stream) {
    if (p == nullptr || q.B <= 0 || q.B > kMaxCallBatch || kv.B != q.B || kv.K != q.K) return -1;
    if (q.K % 8 || q.ldx % 8 || kv.ldx % 8 || (q.N % 4) || (kv.N % 4) || (kv.dh % 4)) return -1;
    if ((reinterpret_cast<uintptr_t>(q.X) & 15) || (reinterpret_cast<uintptr_t>(kv.X) & 15)) return -1;
    const int bn = q.B <= 16 ? 16 : (q.B <= 32 ? 32 : 64);
    const CUtensorMap* mapWq = packed_map(p, q.W, q.N, q.K, 2);
    const CUtensorMap* mapWk = packed_map(p, kv.W, kv.N, kv.K, 2);
    const CUtensorMap* mapWv = packed_map(p, kv.W2, kv.N, kv.K, 2);
    const bool packed = mapWq != nullptr && mapWk != nullptr && mapWv != nullptr;       // one flag for the launch: all three or none
    if (!packed) {
        mapWq = tc_weight_map(p, q.W, q.N, q.K, BM);
        mapWk = tc_weight_map(p, kv.W, kv.N, kv.K, BM);
        mapWv = tc_weight_map(p, kv.W2, kv.N, kv.K, BM);
    }
    CUtensorMap mapXq, mapXkv;
    if (mapWq == nullptr || mapWk == nullptr || mapWv == nullptr || !tc_encode_map(p, &mapXq, q.X, q.B, q.K, q.ldx, bn) ||
        !tc_encode_map(p, &mapXkv, kv.X, kv.B, kv.K, kv.ldx, bn))
        return -1;
    const int q_tiles = (q.N + BM - 1) / BM, kv_tiles = (kv.N + BM - 1) / BM;
    const int kb_total = (q.K + BK - 1) / BK;
    int cs = 1;                                       // K splits = cluster size: a power of two, at most 8, slices of at least 4 k-blocks
    while (cs * 2 <= 8 && (q_tiles + 2 * kv_tiles) * cs * 2 <= kQkvCtaSlots && kb_total / (cs * 2) >= 4) cs *= 2;
    SkArgs a;
    memset(&a, 0, sizeof(a));
    a.N = q.N; a.K = q.K; a.B = q.B; a.nmat = 1; a.kb_per_split = (kb_total + cs - 1) / cs; a.error_word = q.error_word;
    a.packed = packed ? 1 : 0;
    FinishArgs f;
    memset(&f, 0, sizeof(f));
    f.splits = cs; f.nmat = 1; f.B = q.B; f.N = q.N;
    f.out = static_cast<bf16*>(q.out); f.ldo = q.ldo;
    f.kcache = static_cast<bf16*>(kv.kcache); f.vcache = static_cast<bf16*>(kv.vcache); f.Hkv = kv.Hkv; f.dh = kv.dh; f.cap = kv.cap;
    f.slot = kv.slot; f.pos = kv.pos;
    switch (bn) {
        case 16: return launch_sk_qkv<16>(*mapWq, *mapWk, *mapWv, mapXq, mapXkv, a, f, q_tiles, kv_tiles, kv.N, cs, stream);
        case 32: return launch_sk_qkv<32>(*mapWq, *mapWk, *mapWv, mapXq, mapXkv, a, f, q_tiles, kv_tiles, kv.N, cs, stream);
        default: return launch_sk_qkv<64>(*mapWq, *mapWk, *mapWv, mapXq, mapXkv, a, f, q_tiles, kv_tiles, kv.N, cs, stream);
    }
}

size_t tc_skinny_partial_bytes(int N, int K, int nmat) {
    const SplitPlan s = split_plan(N, K, nmat, true);
    return (size_t)s.splits * nmat * kMaxCallBatch * N * sizeof(float);
}

int tc_skinny_key_tiles(int N) { return (N + BM - 1) / BM; }

int tc_skinny(TcPlan* p, int mode, const SkinnyArgs& g, cudaStream_t stream) {
    if (p == nullptr || g.B <= 0 || g.B > kMaxCallBatch) return -1;
    if (g.K % 8 || g.ldx % 8) return -1;                        // TMA: 16-byte row pitch
    if (mode != SK_LOGITS && (g.N % 4)) return -1;              // finishing kernel: float4
    if (reinterpret_cast<uintptr_t>(g.X) & 15) return -1;
    if (mode == SK_KV && (g.dh % 4)) return -1;
    const int nmat = (mode == SK_SILU_MUL || mode == SK_KV) ? 2 : 1;
    const int bn = g.B <= 16 ? 16 : (g.B <= 32 ? 32 : 64);
    const CUtensorMap* mapW = packed_map(p, g.W, g.N, g.K, 2);
    const CUtensorMap* mapW2 = nmat == 2 ? packed_map(p, g.W2, g.N, g.K, 2) : mapW;
    const bool packed = mapW != nullptr && mapW2 != nullptr;
    if (!packed) {
        mapW = tc_weight_map(p, g.W, g.N, g.K, BM);
        mapW2 = nmat == 2 ? tc_weight_map(p, g.W2, g.N, g.K, BM) : mapW;
    }
    CUtensorMap mapX;
    if (mapW == nullptr || mapW2 == nullptr || !tc_encode_map(p, &mapX, g.X, g.B, g.K, g.ldx, bn)) return -1;
    const bool logits = (mode == SK_LOGITS);
    if (logits && g.W8 != nullptr) {
        // FP8 LM head: byte tensor maps (128 elements per swizzle row), scales applied in the epilogue
        if (g.K % 16 || g.X8 == nullptr || g.w_scale == nullptr || g.x_scale == nullptr || (reinterpret_cast<uintptr_t>(g.X8) & 15)) return -1;
        const CUtensorMap* mapW8 = packed_map(p, g.W8, g.N, g.K, 1);
        const bool packed8 = mapW8 != nullptr;
        if (!packed8) mapW8 = tc_weight_map_u8(p, g.W8, g.N, g.K, BM);
        CUtensorMap mapX8;
        if (mapW8 == nullptr || !tc_encode_map_u8(p, &mapX8, g.X8, g.B, g.K, g.K, bn)) return -1;
        SkArgs a8;
        memset(&a8, 0, sizeof(a8));
        a8.N = g.N; a8.K = g.K; a8.B = g.B; a8.nmat = 1; a8.kb_per_split = (g.K + 2 * BK - 1) / (2 * BK);
        a8.logits = g.logits; a8.keys = g.keys; a8.w_scale = g.w_scale; a8.x_scale = g.x_scale; a8.error_word = g.error_word;
        a8.packed = packed8 ? 1 : 0;
        FinishArgs f8;
        memset(&f8, 0, sizeof(f8));
        const dim3 grid8((g.N + BM - 1) / BM, 1, 1);
        switch (bn) {
            case 16: return launch_sk<16, 1, true>(*mapW8, *mapW8, mapX8, a8, f8, mode, grid8, dim3(1, 1, 1), stream);
            case 32: return launch_sk<32, 1, true>(*mapW8, *mapW8, mapX8, a8, f8, mode, grid8, dim3(1, 1, 1), stream);
            default: return launch_sk<64, 1, true>(*mapW8, *mapW8, mapX8, a8, f8, mode, grid8, dim3(1, 1, 1), stream);
        }
    }
    const SplitPlan sp = split_plan(g.N, g.K, nmat, !logits);
    SkArgs a;
    memset(&a, 0, sizeof(a));
    a.N = g.N; a.K = g.K; a.B = g.B; a.nmat = nmat; a.kb_per_split = sp.kb_per_split;
    a.partial = g.partial; a.logits = g.logits; a.keys = g.keys; a.error_word = g.error_word;
    a.packed = packed ? 1 : 0;
    dim3 grid(sp.tiles, nmat, sp.splits);
    FinishArgs f;
    memset(&f, 0, sizeof(f));
    if (logits) return launch_sk_bn<1>(bn, *mapW, *mapW2, mapX, a, f, mode, grid, dim3(1, 1, 1), stream);
    f.partial = g.partial; f.splits = sp.splits; f.nmat = nmat; f.B = g.B; f.N = g.N;
    f.out = static_cast<bf16*>(g.out); f.ldo = g.ldo;
    f.resid = static_cast<const bf16*>(g.resid); f.ldr = g.ldr;
    f.out2 = static_cast<bf16*>(g.out2); f.ld2 = g.ld2; f.orow2 = g.orow2;
    f.norm_out = static_cast<bf16*>(g.norm_out); f.gain = static_cast<const bf16*>(g.gain); f.eps = g.eps; f.do_norm = g.do_norm;
    f.kcache = static_cast<bf16*>(g.kcache); f.vcache = static_cast<bf16*>(g.vcache); f.Hkv = g.Hkv; f.dh = g.dh; f.cap = g.cap;
    f.slot = g.slot; f.pos = g.pos;
    const bool whole_row = (mode == SK_RESID && g.norm_out != nullptr);
    // Preferred: the CTAs of a tile reduce among themselves (cluster of the K splits, or of gate and up).  The fused
    // RMSNorm needs whole rows, so that projection keeps the finishing kernel.
    if (!whole_row) {
        int cs = 1;                                   // power-of-two number of K splits, at most 8 (portable cluster size)
        while (cs * 2 <= sp.splits && cs * 2 <= 8) cs *= 2;
        if (mode == SK_SILU_MUL) cs = 1;
        SkArgs af = a;
        af.kb_per_split = (sp.kb_total + cs - 1) / cs;
        const dim3 fgrid_c(sp.tiles, nmat, cs), cluster(1, mode == SK_SILU_MUL ? 2 : 1, cs);
        if (launch_sk_bn<2>(bn, *mapW, *mapW2, mapX, af, f, mode, fgrid_c, cluster, stream) > 0) return 1;
    }
    if (launch_sk_bn<0>(bn, *mapW, *mapW2, mapX, a, f, mode, grid, dim3(1, 1, 1), stream) < 0) return -1;
    dim3 fgrid(g.B, whole_row ? 1 : (g.N + kFinCols - 1) / kFinCols);
    const dim3 fblock(whole_row ? kFinThreads : kFinColThreads);
    switch (mode) {
        case SK_STORE: launch_pdl(tc_finish_kernel<SK_STORE>, fgrid, fblock, 0, stream, f); break;
        case SK_RESID: launch_pdl(tc_finish_kernel<SK_RESID>, fgrid, fblock, 0, stream, f); break;
        case SK_SILU_MUL: launch_pdl(tc_finish_kernel<SK_SILU_MUL>, fgrid, fblock, 0, stream, f); break;
        case SK_KV: launch_pdl(tc_finish_kernel<SK_KV>, fgrid, fblock, 0, stream, f); break;
        default: return -1;
    }
    return 2;
}

}  // namespace beagle
