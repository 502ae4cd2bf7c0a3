// Cross-attention decode over the bf16 K/V cache (Eq. 2, lines 2-3), TMA-staged.
//
// One CTA = one (sequence, K/V head, chunk of 128 cached states).  A chunk of the cache is a
// contiguous run of 128 rows of 2*dh bytes, so one thread issues the whole K tile and the whole V
// tile as TMA tile copies (128-byte swizzle) the moment the CTA starts; three CTAs share an SM, so
// about 190 KB per SM are in flight with no registers tied up and the kernel stays HBM-bound.
//
// The G = Hq/Hkv query heads that share the K/V head are rows of a 16-row mma.sync tile: with
// grouped queries the path does G*4 flop per cache byte, which the CUDA cores cannot sustain next
// to the unpacking at HBM speed, while the tensor pipe does it in passing.  Each of the four warps
// owns 32 keys: S = Q K^T (ldmatrix + m16n8k16), a warp-local softmax in registers, O = P V
// (ldmatrix.trans), then the four partial (m, l, O) triples are merged in shared memory and the
// chunk's unnormalised partial goes to the split-KV scratch.  The CTA that finishes last for its
// (sequence, K/V head) -- a counter in global memory, reset by that CTA -- merges the chunks of
// its G heads and writes o, so no second kernel is needed.
//
// Rows past the sequence's length inside the last chunk hold whatever the cache held before:
// their scores are replaced by -inf and their V rows are zeroed in shared memory, so they
// contribute exactly nothing.  The wait for the tiles is bounded; a wait that runs out raises the
// device error word and the CTA writes an empty partial instead of hanging.
#include <cstring>

#include "attn_combine.cuh"
#include "gemm_tc.h"
#include "tc_plan.h"
#include "tc_ptx.cuh"

namespace beagle {

namespace {

using namespace tc;

constexpr int kChunk = 128;             // cached states per CTA
constexpr int kWarps = 4;
constexpr int kKeysPerWarp = kChunk / kWarps;

struct AttnWork {                       // by value in the kernel parameters
    int32_t slot[kMaxCallBatch];
    int32_t kv_len[kMaxCallBatch];
    int32_t item_start[kMaxCallBatch + 1];   // prefix sum of chunks per batch row
    int32_t stable_len[kMaxCallBatch];       // leading rows written before this chain of kernels began (the true states)
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float* d, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}
// Byte offset of the 16-byte chunk `chunk` (8 elements) of row `row` inside a tile of 128-byte
// rows written by TMA with the 128-byte swizzle; a tile holds 64 columns, wider rows use
// consecutive tiles of kChunk rows.
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
    return static_cast<uint32_t>((chunk >> 3) * (kChunk * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

template <int DH, int G>
__global__ void __launch_bounds__(kWarps * 32) attn_decode_tma_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                     const __grid_constant__ CUtensorMap tmV,
                                                                     const bf16* q, const AttnWork work, int nbatch,
                                                                     int Hq, int Hkv, int cap, int nch_stride, float scale_log2,
                                                                     float* part_o, float* part_ml, int* done_count,
                                                                     bf16* __restrict__ o_out, int* error_word) {
    constexpr int kTileBytes = kChunk * DH * 2;         // one of K / V
    constexpr int kHalves = DH / 64;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sK = smem_base, sV = smem_base + kTileBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_gen + 2 * kTileBytes);
    const uint32_t barK = smem_u32(bars), barV = barK + 8;
    __shared__ float s_m[kWarps][8], s_l[kWarps][8];
    __shared__ int s_abort, s_last;

    // which (sequence, chunk) this CTA owns
    int b = 0;
    while (b + 1 < nbatch && (int)blockIdx.x >= work.item_start[b + 1]) ++b;
    const int chunk = blockIdx.x - work.item_start[b];
    const int kvh = blockIdx.y;
    const int kv_len = work.kv_len[b];
    const int start = chunk * kChunk;
    const int cnt = min(kChunk, kv_len - start);       // >= 1 by construction of item_start
    const int row0 = (work.slot[b] * Hkv + kvh) * cap + start;
    (void)BEAGLE_IN_BOUNDS(cnt >= 1 && kv_len <= cap && BEAGLE_SLOT_OK(work.slot[b]));     // (a TMA tile past the tensor's end reads zeros: nothing to skip)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;

    // When to let the next kernel's CTAs in (measured): with the batched tensor-core projections after it, right away (their
    // weight tiles are requested while this kernel runs, +1 % at batch 32); with the batch <= 8 projections, only at the end
    // (their early CTAs slow this kernel's stream down, -1.5 % at batch 1).
    const bool release_early = nbatch > 8;
    if (release_early) pdl_launch_dependents();
    // A chunk that lies entirely inside the true states cannot be touched by the kernels this one
    // may overlap with (they only append draft states), so its tiles are requested right away;
    // the last chunks wait for the previous kernels first.
    const bool stable = start + kChunk <= work.stable_len[b];
    if (threadIdx.x == 0) {
        mbar_init(barK, 1);
        mbar_init(barV, 1);
        s_abort = 0;
        fence_barrier_init();
        if (!stable) pdl_wait();
        const uint64_t once = policy_evict_first();
        mbar_expect_tx(barK, kTileBytes);
#pragma unroll
        for (int h = 0; h < kHalves; ++h) tma_load_2d_hint(sK + h * (kChunk * 128), &tmK, barK, h * 64, row0, once);
        mbar_expect_tx(barV, kTileBytes);
#pragma unroll
        for (int h = 0; h < kHalves; ++h) tma_load_2d_hint(sV + h * (kChunk * 128), &tmV, barV, h * 64, row0, once);
    }

    pdl_wait();                                                          // Q comes from the previous kernel
    // Q fragments: rows of the A operand are the G query heads of this K/V head (rows >= G are zero)
    uint32_t qa[DH / 16][2];
    {
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(q + ((size_t)b * Hq + kvh * G + (g < G ? g : 0)) * DH);
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
            qa[ks][0] = g < G ? ld_act32(qrow + ks * 8 + c) : 0u;         // dims 16ks + 2c, +1
            qa[ks][1] = g < G ? ld_act32(qrow + ks * 8 + 4 + c) : 0u;     // dims 16ks + 8 + 2c, +1
        }
    }
    __syncthreads();                                                     // barriers initialised

    bool ok = mbar_wait(barK, 0, &s_abort);
    ok = __all_sync(0xffffffffu, ok);

    // ---- S = Q K^T for this warp's 32 keys
    float s[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
    const int krow = warp * kKeysPerWarp;
    if (ok) {
#pragma unroll
        for (int dg = 0; dg < DH / 32; ++dg) {
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(sK + tile_off(krow + nt * 8 + (lane & 7), 4 * dg + (lane >> 3)), b0, b1, b2, b3);
                mma_bf16(s[nt], qa[2 * dg][0], 0u, qa[2 * dg][1], 0u, b0, b1);
                mma_bf16(s[nt], qa[2 * dg + 1][0], 0u, qa[2 * dg + 1][1], 0u, b2, b3);
            }
        }
    }

    // ---- warp-local softmax of head g (lanes g*4 .. g*4+3 hold its 32 scores); base-2 exponent
    float m = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int j = krow + nt * 8 + 2 * c + e;
            s[nt][e] = (j < cnt) ? s[nt][e] * scale_log2 : -INFINITY;
            m = fmaxf(m, s[nt][e]);
        }
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
    uint32_t pa[2][2];
    float l = 0.f;
#pragma unroll
    for (int kk = 0; kk < 2; ++kk)
#pragma unroll
        for (int hlf = 0; hlf < 2; ++hlf) {
            const int nt = 2 * kk + hlf;
            const float p0 = (m == -INFINITY) ? 0.f : exp2f(s[nt][0] - m);
            const float p1 = (m == -INFINITY) ? 0.f : exp2f(s[nt][1] - m);
            const __nv_bfloat162 pr = __floats2bfloat162_rn(p0, p1);     // the weights the tensor cores will use
            l += __low2float(pr) + __high2float(pr);
            pa[kk][hlf] = *reinterpret_cast<const uint32_t*>(&pr);
        }
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);

    // ---- V tile: wait, blank the rows past the sequence's end, then O = P V
    bool okv = mbar_wait(barV, 0, &s_abort);
    okv = __all_sync(0xffffffffu, okv);
    if (okv && cnt < kChunk) {
        const int nz = (kChunk - cnt) * (DH / 8);                        // 16-byte pieces to clear
        for (int i = threadIdx.x; i < nz; i += kWarps * 32) {
            const int row = cnt + i / (DH / 8), ch = i % (DH / 8);
            *reinterpret_cast<uint4*>(smem_gen + kTileBytes + tile_off(row, ch)) = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    __syncthreads();                                                     // zeroes visible; K tile no longer read

    float o[DH / 8][4];
#pragma unroll
    for (int nt = 0; nt < DH / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    if (ok && okv) {
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
#pragma unroll
            for (int jp = 0; jp < DH / 16; ++jp) {
                uint32_t b0, b1, b2, b3;
                const int mi = lane >> 3;
                ldmatrix_x4_trans(sV + tile_off(krow + kk * 16 + 8 * (mi & 1) + (lane & 7), 2 * jp + (mi >> 1)), b0, b1, b2, b3);
                mma_bf16(o[2 * jp], pa[kk][0], 0u, pa[kk][1], 0u, b0, b1);
                mma_bf16(o[2 * jp + 1], pa[kk][0], 0u, pa[kk][1], 0u, b2, b3);
            }
        }
    }

    // ---- merge the four warps' partials (the K tile's memory is free now)
    float* comb = reinterpret_cast<float*>(smem_gen);                    // [warp][G][DH]
    if (g < G) {
#pragma unroll
        for (int nt = 0; nt < DH / 8; ++nt)
            *reinterpret_cast<float2*>(comb + ((size_t)(warp * G + g) * DH + nt * 8 + 2 * c)) = make_float2(o[nt][0], o[nt][1]);
        if (c == 0) { s_m[warp][g] = m; s_l[warp][g] = l; }
    }
    __syncthreads();
    const bool good = ok && okv;
    for (int i = threadIdx.x; i < G * DH; i += kWarps * 32) {
        const int hg = i / DH, d = i % DH;
        float M = s_m[0][hg];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) M = fmaxf(M, s_m[w][hg]);
        float acc = 0.f, L = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float wgt = (s_m[w][hg] == -INFINITY) ? 0.f : exp2f(s_m[w][hg] - M);
            acc = fmaf(wgt, comb[(size_t)(w * G + hg) * DH + d], acc);
            L = fmaf(wgt, s_l[w][hg], L);
        }
        const size_t pi = ((size_t)b * Hq + kvh * G + hg) * nch_stride + chunk;
        part_o[pi * DH + d] = good ? acc : 0.f;
        if (d == 0) {
            part_ml[2 * pi] = good ? M * 0.6931471805599453f : -INFINITY;      // back to the natural-log scale of attn_combine
            part_ml[2 * pi + 1] = good ? L : 0.f;
        }
    }
    // ---- the last CTA of this (sequence, K/V head) merges all chunks of its G heads
    // (done_count == NULL: a separate kernel merges, which is faster for large batches)
    const int nchunks = (kv_len + kChunk - 1) / kChunk;
    if (done_count != nullptr) {
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) {
            const int prev = atomicAdd(&done_count[b * Hkv + kvh], 1);
            s_last = (prev == nchunks - 1);
            if (s_last) done_count[b * Hkv + kvh] = 0;                  // ready for the next launch
        }
        __syncthreads();
    }
    if (done_count != nullptr && s_last) {
        __threadfence();
        for (int hg = warp; hg < G; hg += kWarps) {
            const size_t head = (size_t)b * Hq + kvh * G + hg;
            attn_combine_warp<bf16, DH / 32, true>(part_o + head * nch_stride * DH, part_ml + 2 * head * nch_stride, nchunks, DH, lane,
                                             o_out + head * DH);
        }
    }
    if (threadIdx.x == 0 && s_abort) {
        if (error_word != nullptr) atomicExch(error_word, 1);
        // the copies may still be in flight: give them a second bounded chance to land before the CTA ends
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(barK, 0); ++i) {}
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(barV, 0); ++i) {}
    }
    if (!release_early) pdl_launch_dependents();
}

template <int DH, int G>
int launch_attn(const CUtensorMap& mk, const CUtensorMap& mv, const bf16* q, const AttnWork& work, int nbatch, int items, int Hq,
                int Hkv, int cap, int nch_stride, float scale_log2, float* po, float* pml, int* done_count, bf16* o, int* error_word,
                cudaStream_t stream) {
    constexpr int kSmem = 2 * kChunk * DH * 2 + 1024 + 64;
    static PerDeviceOnce smem_attr;
    if (!smem_attr.ensure([] { return cudaFuncSetAttribute(attn_decode_tma_kernel<DH, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) == cudaSuccess; }))
        return -1;
    launch_pdl(attn_decode_tma_kernel<DH, G>, dim3(items, Hkv), dim3(kWarps * 32), (size_t)kSmem, stream, mk, mv, q, work, nbatch, Hq, Hkv,
               cap, nch_stride, scale_log2, po, pml, done_count, o, error_word);
    return 1;
}

template <int DH>
int launch_attn_g(int G, const CUtensorMap& mk, const CUtensorMap& mv, const bf16* q, const AttnWork& work, int nbatch, int items,
                  int Hq, int Hkv, int cap, int nch_stride, float scale_log2, float* po, float* pml, int* done_count, bf16* o,
                  int* error_word, cudaStream_t stream) {
    switch (G) {
        case 1: return launch_attn<DH, 1>(mk, mv, q, work, nbatch, items, Hq, Hkv, cap, nch_stride, scale_log2, po, pml, done_count, o, error_word, stream);
        case 2: return launch_attn<DH, 2>(mk, mv, q, work, nbatch, items, Hq, Hkv, cap, nch_stride, scale_log2, po, pml, done_count, o, error_word, stream);
        case 4: return launch_attn<DH, 4>(mk, mv, q, work, nbatch, items, Hq, Hkv, cap, nch_stride, scale_log2, po, pml, done_count, o, error_word, stream);
        case 8: return launch_attn<DH, 8>(mk, mv, q, work, nbatch, items, Hq, Hkv, cap, nch_stride, scale_log2, po, pml, done_count, o, error_word, stream);
        default: return -1;
    }
}

}  // namespace

int tc_attn_chunk(void) { return kChunk; }

bool tc_attn_bind_cache(TcPlan* p, const void* kcache, const void* vcache, long long rows, int dh) {
    if (p == nullptr) return false;
    p->cache_maps_ok = false;
    if (dh != 64 && dh != 128) return false;
    if (rows <= 0 || rows > 0x7fffffffll) return false;
    if (!tc_encode_map(p, &p->cache_k, kcache, rows, dh, dh, kChunk)) return false;
    if (!tc_encode_map(p, &p->cache_v, vcache, rows, dh, dh, kChunk)) return false;
    p->cache_maps_ok = true;
    return true;
}

int tc_attn_decode(TcPlan* p, const void* q, const BatchMeta& meta, const int32_t* stable_len, int B, int Hq, int Hkv, int dh, int cap,
                   int max_kv_len, void* scratch, int* done_count, void* o, int* error_word, cudaStream_t stream, int defer_merge,
                   float** part_o_out, float** part_ml_out, int* nch_stride_out) {
    if (p == nullptr || !p->cache_maps_ok || B <= 0 || B > kMaxCallBatch || Hkv > 65535) return -1;
    if (dh != 64 && dh != 128) return -1;
    const int G = Hq / Hkv;
    AttnWork work;
    memset(&work, 0, sizeof(work));
    int items = 0;
    for (int b = 0; b < B; ++b) {
        work.slot[b] = meta.slot[b];
        work.kv_len[b] = meta.kv_len[b];
        work.stable_len[b] = stable_len != nullptr ? stable_len[b] : 0;
        work.item_start[b] = items;
        items += (meta.kv_len[b] + kChunk - 1) / kChunk;
    }
    for (int b = B; b <= kMaxCallBatch; ++b) work.item_start[b] = items;
    const int nch = (max_kv_len + kChunk - 1) / kChunk + 1;              // row stride of the partial buffers
    float* po = reinterpret_cast<float*>(scratch);
    float* pml = po + (size_t)B * Hq * nch * dh;
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)dh);
    // Few sequences: the last CTA of each head group merges its chunks (one launch less on a
    // latency-bound step).  Many sequences: a separate, wider merge kernel is faster than the tails.
    const bool fuse_merge = B <= 8 && !defer_merge;
    if (part_o_out != nullptr) { *part_o_out = po; *part_ml_out = pml; *nch_stride_out = nch; }
    if (!fuse_merge) done_count = nullptr;
    int launched = 0;
    if (items > 0) {
        const int rc = dh == 128
            ? launch_attn_g<128>(G, p->cache_k, p->cache_v, static_cast<const bf16*>(q), work, B, items, Hq, Hkv, cap, nch, scale_log2, po, pml,
                                 done_count, static_cast<bf16*>(o), error_word, stream)
            : launch_attn_g<64>(G, p->cache_k, p->cache_v, static_cast<const bf16*>(q), work, B, items, Hq, Hkv, cap, nch, scale_log2, po, pml,
                                done_count, static_cast<bf16*>(o), error_word, stream);
        if (rc < 0) return rc;
        launched += rc;
    }
    // rows without any cached state got no CTA: their attention output is zero
    bool any_empty = !fuse_merge;
    for (int b = 0; b < B; ++b) any_empty |= (meta.kv_len[b] == 0);
    if (any_empty && !defer_merge) launched += launch_attn_combine(1, po, pml, meta, B, Hq, dh, nch, kChunk, o, stream);
    return launched;
}

}  // namespace beagle
