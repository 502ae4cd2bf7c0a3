// Serve-time kernels of the Beagle draft head: embedding + RMSNorm, weight-streaming skinny
// projections with fused epilogues, split-KV cross-attention decode over the cache, arg-max and
// greedy acceptance.  All HBM-bound: 16-byte coalesced loads, fp32 accumulation.
#include "kernels.h"
#include "attn_combine.cuh"

namespace beagle {

// ------------------------------------------------------------------------------------------------
// Embedding gather + RMSNorm (Eq. 1: e(t_p); normalisation as configured)
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) embed_norm_kernel(const int32_t* tokens, const int32_t* last_token,     // (no __restrict__ on
                                                         const BatchMeta meta,                                   //  what earlier kernels of the
                                                         const T* __restrict__ embed, int vocab,                //  launch chain write)
                                                         const T* src, const T* __restrict__ gain,
                                                         int d, float eps, int do_norm, T* __restrict__ x_out,
                                                         T* __restrict__ xn_out, const T* gather_src,
                                                         T* __restrict__ gather_dst) {
    constexpr int VEC = VecOf<T>::N;
    constexpr int kMaxVec = 4;                  // 16-byte pieces a thread keeps in registers (d <= 256 * 4 * VEC)
    const int r = blockIdx.x;
    const int nvec = d / VEC;                   // d is a multiple of 8
    // First kernel of a draft step: it waits BEFORE it lets its dependents start, so every kernel
    // of this step begins after all earlier work in the stream (cache prefill, the previous step)
    // has completed.  The later kernels' early reads of weights and true-state cache rows rely on it.
    pdl_wait();
    const bool release_early = gridDim.x > 8;      // small batches: at the end (measured, as in the projection kernel below)
    if (release_early) pdl_launch_dependents();
    if (gather_src != nullptr) {
        const uint4* g = reinterpret_cast<const uint4*>(gather_src + (size_t)meta.slot[r] * d);
        uint4* dst = reinterpret_cast<uint4*>(gather_dst + (size_t)r * d);
        for (int i = threadIdx.x; i < nvec; i += blockDim.x) dst[i] = ld_act16(g + i);
    }
    const T* row;
    if (src != nullptr) {
        row = src + (size_t)r * d;
    } else {
        int tok = tokens != nullptr ? tokens[r] : last_token[meta.slot[r]];
        (void)BEAGLE_IN_BOUNDS(tok >= 0 && tok < vocab && (tokens != nullptr || BEAGLE_SLOT_OK(meta.slot[r])));
        tok = min(max(tok, 0), vocab - 1);      // ids are validated by contract; never read out of range
        row = embed + (size_t)tok * d;
    }
    const uint4* row4 = reinterpret_cast<const uint4*>(row);
    const bool in_regs = nvec <= kMaxVec * (int)blockDim.x && (d % VEC) == 0;
    uint4 keep[kMaxVec];
    float ss = 0.f;
    if (in_regs) {
#pragma unroll
        for (int j = 0; j < kMaxVec; ++j) {
            const int i = threadIdx.x + j * blockDim.x;
            keep[j] = i < nvec ? ld_act16(row4 + i) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int j = 0; j < kMaxVec; ++j) {
            float f[VEC];
            unpack16<T>(keep[j], f);
#pragma unroll
            for (int v = 0; v < VEC; ++v) ss = fmaf(f[v], f[v], ss);
        }
    } else {
        for (int i = threadIdx.x; i < d; i += blockDim.x) {
            float v = to_float<T>(row[i]);
            ss += v * v;
        }
    }
    __shared__ float s_part[8];
    __shared__ float s_scale;
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += s_part[w];
        s_scale = do_norm ? rsqrtf(t / (float)d + eps) : 1.0f;
    }
    __syncthreads();
    const float sc = s_scale;
    if (in_regs) {
#pragma unroll
        for (int j = 0; j < kMaxVec; ++j) {
            const int i = threadIdx.x + j * blockDim.x;
            if (i >= nvec) break;
            if (x_out != nullptr) reinterpret_cast<uint4*>(x_out + (size_t)r * d)[i] = keep[j];
            float f[VEC], g[VEC];
            unpack16<T>(keep[j], f);
            if (do_norm) unpack16<T>(__ldg(reinterpret_cast<const uint4*>(gain) + i), g);
            T o[VEC];
#pragma unroll
            for (int v = 0; v < VEC; ++v) o[v] = from_float<T>(f[v] * sc * (do_norm ? g[v] : 1.0f));
            reinterpret_cast<uint4*>(xn_out + (size_t)r * d)[i] = *reinterpret_cast<const uint4*>(o);
        }
    } else {
        for (int i = threadIdx.x; i < d; i += blockDim.x) {
            float v = to_float<T>(row[i]);
            if (x_out != nullptr) x_out[(size_t)r * d + i] = from_float<T>(v);
            float g = do_norm ? to_float<T>(gain[i]) : 1.0f;
            xn_out[(size_t)r * d + i] = from_float<T>(v * sc * g);
        }
    }
    if (!release_early) pdl_launch_dependents();
}

int launch_embed_norm(int dtype, const int32_t* tokens, const int32_t* last_token, const BatchMeta* meta,
                      const void* embed, int vocab, const void* src, const void* gain, int d, float eps, int do_norm,
                      void* x_out, void* xn_out, int rows, const void* gather_src, void* gather_dst, cudaStream_t stream) {
    if (rows <= 0) return 0;
    BatchMeta m;
    if (meta != nullptr) m = *meta; else memset(&m, 0, sizeof(m));
    if (dtype == 0)
        launch_pdl(embed_norm_kernel<float>, dim3(rows), dim3(256), 0, stream, tokens, last_token, m, (const float*)embed, vocab,
                   (const float*)src, (const float*)gain, d, eps, do_norm, (float*)x_out, (float*)xn_out,
                   (const float*)gather_src, (float*)gather_dst);
    else
        launch_pdl(embed_norm_kernel<bf16>, dim3(rows), dim3(256), 0, stream, tokens, last_token, m, (const bf16*)embed, vocab,
                   (const bf16*)src, (const bf16*)gain, d, eps, do_norm, (bf16*)x_out, (bf16*)xn_out,
                   (const bf16*)gather_src, (bf16*)gather_dst);
    return 1;
}

// ------------------------------------------------------------------------------------------------
// Skinny projection: out[b][n] = W[n,:] . x_b for B <= 64 rows.  One warp owns two weight rows
// (or one row of each of W / W2 in the gated mode) and streams them once per group of NB batch
// rows with 16-byte loads; the activations are re-read through L1.
// ------------------------------------------------------------------------------------------------
// HALVES (K/V append of a narrow projection, e.g. 8 K/V heads): the warp owns ONE weight row and its two streams are the
// row's halves, which doubles the CTAs of a grid that would otherwise leave most SMs without work.
template <typename T, int NB, int MODE, bool HALVES = false>
__global__ void __launch_bounds__(256) stream_proj_kernel(const GemvArgs a) {
    constexpr int VEC = VecOf<T>::N;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int unit = blockIdx.x * 8 + warp;
    const T* W = reinterpret_cast<const T*>(a.W);
    const T* W2 = reinterpret_cast<const T*>(a.W2);
    const T* Wsel = (MODE == GEMV_KV && blockIdx.y == 1) ? W2 : W;
    const int klen = HALVES ? a.K / 2 : a.K;     // elements each of the warp's two streams covers
    int n0, n1;
    bool v0, v1;
    const T *w0, *w1;
    if (HALVES) {
        n0 = n1 = unit;
        v0 = unit < a.N;
        v1 = false;                              // (the second accumulator is folded into the first below)
        w0 = Wsel + (size_t)(v0 ? unit : 0) * a.K;
        w1 = w0 + klen;
    } else if (MODE == GEMV_SILU_MUL) {
        n0 = n1 = unit;
        v0 = v1 = unit < a.N;
        const int nn = v0 ? unit : 0;
        w0 = W + (size_t)nn * a.K;
        w1 = W2 + (size_t)nn * a.K;
    } else {
        n0 = 2 * unit;
        n1 = n0 + 1;
        v0 = n0 < a.N;
        v1 = n1 < a.N;
        w0 = Wsel + (size_t)(v0 ? n0 : 0) * a.K;
        w1 = Wsel + (size_t)(v1 ? n1 : 0) * a.K;
    }
    const T* X = reinterpret_cast<const T*>(a.X);
    __shared__ unsigned long long s_keys[8][NB];

    // The weights do not depend on the previous kernel: pull the head of this warp's rows towards
    // L2 while that kernel drains, then wait for the activations.  The dependents are released only at
    // the END of this kernel: measured at batch 1, CTAs of the next kernel that become resident while
    // this one still streams slow the chain down (releasing before the wait: -3.7 % drafted tokens/s).
    if (lane < 16) {                            // the first 2 KB of each row (bf16; 4 KB in fp32, every other line)
        const int k = lane * 64;
        if (k < klen) { prefetch_l2(w0 + k); prefetch_l2(w1 + k); }
    }
    pdl_wait();

    for (int b0 = 0; b0 < a.B; b0 += NB) {
        const T* xp[NB];
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            const int b = min(b0 + j, a.B - 1);
            xp[j] = X + (size_t)a.xrow.idx[b] * a.ldx;
        }
        float acc0[NB], acc1[NB];
#pragma unroll
        for (int j = 0; j < NB; ++j) { acc0[j] = 0.f; acc1[j] = 0.f; }

        // one step of both streams against the NB activation rows
        auto consume = [&](const uint4& ua, const uint4& ub, int k) {
            float wf0[VEC], wf1[VEC];
            unpack16<T>(ua, wf0);
            unpack16<T>(ub, wf1);
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                float xf[VEC];
                unpack16<T>(ld_act16(xp[j] + k), xf);      // activations: written by the previous kernel of the chain
                if (HALVES) {
                    float xg[VEC];
                    unpack16<T>(ld_act16(xp[j] + klen + k), xg);
#pragma unroll
                    for (int v = 0; v < VEC; ++v) {
                        acc0[j] = fmaf(wf0[v], xf[v], acc0[j]);
                        acc1[j] = fmaf(wf1[v], xg[v], acc1[j]);
                    }
                } else {
#pragma unroll
                    for (int v = 0; v < VEC; ++v) {
                        acc0[j] = fmaf(wf0[v], xf[v], acc0[j]);
                        acc1[j] = fmaf(wf1[v], xf[v], acc1[j]);
                    }
                }
            }
        };
        if constexpr (MODE == GEMV_LOGITS && NB == 1) {
            // The LM head at batch 1 is one long stream (0.26 - 1.05 GB): eight steps of both rows are requested before the first
            // is consumed (16 loads of 16 bytes in flight per lane; measured 164 -> 153 us at V = 128256).  The shorter
            // projections lose with this form (fewer resident CTAs, longer tails: down-projection 27 -> 33 us) and keep the loop below.
            constexpr int U = 8;
            for (int k0 = lane * VEC; k0 < klen; k0 += U * 32 * VEC) {
                uint4 wa[U], wb[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int k = k0 + u * 32 * VEC;
                    if (k < klen) { wa[u] = ld_stream16(w0 + k); wb[u] = ld_stream16(w1 + k); }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int k = k0 + u * 32 * VEC;
                    if (k >= klen) break;
                    consume(wa[u], wb[u], k);
                }
            }
        } else {
#pragma unroll 4
            for (int k = lane * VEC; k < klen; k += 32 * VEC) consume(ld_stream16(w0 + k), ld_stream16(w1 + k), k);
        }
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            if (HALVES) acc0[j] += acc1[j];
            acc0[j] = warp_sum(acc0[j]);
            if (!HALVES) acc1[j] = warp_sum(acc1[j]);
        }

        if (MODE == GEMV_LOGITS) {
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                unsigned long long key = 0ull;
                if (v0) key = argmax_key(acc0[j], n0);
                if (v1) { unsigned long long k1 = argmax_key(acc1[j], n1); key = k1 > key ? k1 : key; }
                if (lane == 0) s_keys[warp][j] = key;
                if (lane == 0 && a.logits != nullptr && b0 + j < a.B) {
                    if (v0) a.logits[(size_t)(b0 + j) * a.N + n0] = acc0[j];
                    if (v1) a.logits[(size_t)(b0 + j) * a.N + n1] = acc1[j];
                }
            }
            __syncthreads();
            if (threadIdx.x < NB && b0 + (int)threadIdx.x < a.B) {
                unsigned long long key = s_keys[0][threadIdx.x];
#pragma unroll
                for (int w = 1; w < 8; ++w) { unsigned long long o = s_keys[w][threadIdx.x]; key = o > key ? o : key; }
                a.partials[(size_t)(b0 + threadIdx.x) * gridDim.x + blockIdx.x] = key;
            }
            __syncthreads();
        } else if (lane == 0) {
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                const int b = b0 + j;
                if (b >= a.B) break;
                if (MODE == GEMV_STORE) {
                    T* out = reinterpret_cast<T*>(a.out) + (size_t)b * a.ldo;
                    if (v0) out[n0] = from_float<T>(acc0[j]);
                    if (v1) out[n1] = from_float<T>(acc1[j]);
                } else if (MODE == GEMV_RESID) {
                    const T* r = reinterpret_cast<const T*>(a.resid) + (size_t)b * a.ldr;
                    T* out = reinterpret_cast<T*>(a.out) + (size_t)b * a.ldo;
                    T* out2 = a.out2 ? reinterpret_cast<T*>(a.out2) + (size_t)a.orow2.idx[b] * a.ld2 : nullptr;
                    if (v0) { T y = from_float<T>(acc0[j] + to_float<T>(r[n0])); out[n0] = y; if (out2) out2[n0] = y; }
                    if (v1) { T y = from_float<T>(acc1[j] + to_float<T>(r[n1])); out[n1] = y; if (out2) out2[n1] = y; }
                } else if (MODE == GEMV_SILU_MUL) {
                    if (v0) reinterpret_cast<T*>(a.out)[(size_t)b * a.ldo + n0] = from_float<T>(silu_f(acc0[j]) * acc1[j]);
                } else if (MODE == GEMV_KV) {
                    T* cache = reinterpret_cast<T*>(blockIdx.y == 1 ? a.vcache : a.kcache);
                    const int slot = a.orow2.idx[b], pos = a.pos.idx[b];
                    if (pos < 0) continue;          // this row appends nothing
                    if (!BEAGLE_IN_BOUNDS(pos < a.cap && BEAGLE_SLOT_OK(slot))) continue;
                    if (v0) cache[(((size_t)slot * a.Hkv + n0 / a.dh) * a.cap + pos) * a.dh + n0 % a.dh] = from_float<T>(acc0[j]);
                    if (v1) cache[(((size_t)slot * a.Hkv + n1 / a.dh) * a.cap + pos) * a.dh + n1 % a.dh] = from_float<T>(acc1[j]);
                }
            }
        }
    }
    pdl_launch_dependents();
}

int gemv_grid_blocks(int mode, int N) {
    const int units = (mode == GEMV_SILU_MUL) ? N : (N + 1) / 2;
    return (units + 7) / 8;
}
// K/V append of a narrow projection: two-rows-per-warp CTAs would number fewer than two per SM (148 SMs)
static bool kv_use_halves(const GemvArgs& a, int vec) { return 2 * gemv_grid_blocks(GEMV_KV, a.N) < 296 && a.K % (2 * vec) == 0; }

template <typename T, int MODE>
static void gemv_dispatch_nb(const GemvArgs& a, dim3 grid, cudaStream_t stream) {
    if (MODE == GEMV_KV && kv_use_halves(a, VecOf<T>::N)) {
        grid.x = (a.N + 7) / 8;                  // one row per warp
        if (a.B <= 1) launch_pdl(stream_proj_kernel<T, 1, GEMV_KV, true>, grid, dim3(256), 0, stream, a);
        else if (a.B <= 2) launch_pdl(stream_proj_kernel<T, 2, GEMV_KV, true>, grid, dim3(256), 0, stream, a);
        else if (a.B <= 4) launch_pdl(stream_proj_kernel<T, 4, GEMV_KV, true>, grid, dim3(256), 0, stream, a);
        else launch_pdl(stream_proj_kernel<T, 8, GEMV_KV, true>, grid, dim3(256), 0, stream, a);
        return;
    }
    if (a.B <= 1) launch_pdl(stream_proj_kernel<T, 1, MODE>, grid, dim3(256), 0, stream, a);
    else if (a.B <= 2) launch_pdl(stream_proj_kernel<T, 2, MODE>, grid, dim3(256), 0, stream, a);
    else if (a.B <= 4) launch_pdl(stream_proj_kernel<T, 4, MODE>, grid, dim3(256), 0, stream, a);
    else launch_pdl(stream_proj_kernel<T, 8, MODE>, grid, dim3(256), 0, stream, a);
}
template <typename T>
static void gemv_dispatch_mode(int mode, const GemvArgs& a, dim3 grid, cudaStream_t stream) {
    switch (mode) {
        case GEMV_STORE: gemv_dispatch_nb<T, GEMV_STORE>(a, grid, stream); break;
        case GEMV_RESID: gemv_dispatch_nb<T, GEMV_RESID>(a, grid, stream); break;
        case GEMV_SILU_MUL: gemv_dispatch_nb<T, GEMV_SILU_MUL>(a, grid, stream); break;
        case GEMV_LOGITS: gemv_dispatch_nb<T, GEMV_LOGITS>(a, grid, stream); break;
        default: gemv_dispatch_nb<T, GEMV_KV>(a, grid, stream); break;
    }
}
int launch_gemv(int dtype, int mode, const GemvArgs& a, cudaStream_t stream) {
    if (a.B <= 0 || a.N <= 0) return 0;
    dim3 grid(gemv_grid_blocks(mode, a.N), mode == GEMV_KV ? 2 : 1);
    if (dtype == 0) gemv_dispatch_mode<float>(mode, a, grid, stream);
    else gemv_dispatch_mode<bf16>(mode, a, grid, stream);
    return 1;
}

// ------------------------------------------------------------------------------------------------
// Cross-attention decode (Eq. 2 lines 2-3 over the cached K/V): split-KV partials + combine.
// One CTA = one (sequence, K/V head, chunk of kAttnChunk keys); its G = Hq/Hkv query heads share
// every key/value row it streams.  LPK lanes cover one cache row with one 16-byte load each.
// ------------------------------------------------------------------------------------------------
constexpr int kAttnChunk = 256;
constexpr int kAttnMinChunk = 128;      // smallest chunk any decode kernel uses (sizes the partial buffers)
constexpr int kAttnWarps = 4;

template <typename T, int G, int LPK>
__global__ void __launch_bounds__(kAttnWarps * 32) attn_decode_kernel(
    const T* q, const T* kcache, const T* vcache, const BatchMeta meta,       // written by earlier kernels of the chain: no __restrict__
    int Hq, int Hkv, int cap, int nchunk_max, float scale, float* __restrict__ part_o, float* __restrict__ part_ml) {
    constexpr int VEC = VecOf<T>::N;
    constexpr int DH = LPK * VEC;
    constexpr int KPW = 32 / LPK;                 // keys per warp per iteration
    constexpr int KPI = KPW * kAttnWarps;         // keys per CTA per iteration
    const int chunk = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int kv_len = meta.kv_len[b];
    const int start = chunk * kAttnChunk;
    pdl_launch_dependents();
    pdl_wait();
    if (start >= kv_len) return;
    const int cnt = min(kAttnChunk, kv_len - start);
    const int slot = meta.slot[b];
    if (!BEAGLE_IN_BOUNDS(kv_len <= cap && BEAGLE_SLOT_OK(slot))) return;
    const size_t base = (((size_t)slot * Hkv + kvh) * cap + start) * DH;
    const T* kb = kcache + base;
    const T* vb = vcache + base;

    __shared__ float s_q[G][DH];
    __shared__ float s_s[G][kAttnChunk];
    __shared__ float s_acc[kAttnWarps][G][DH];
    __shared__ float s_m[G], s_l[G];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < G * DH; i += kAttnWarps * 32)
        s_q[i / DH][i % DH] = to_float<T>(q[((size_t)b * Hq + kvh * G + i / DH) * DH + i % DH]) * scale;
    __syncthreads();

    const int sub = lane % LPK, kgrp = lane / LPK;
    float qf[G][VEC];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int v = 0; v < VEC; ++v) qf[g][v] = s_q[g][sub * VEC + v];

    // phase 1: scores
#pragma unroll 4
    for (int jb = warp * KPW; jb < cnt; jb += KPI) {
        const int j = jb + kgrp;
        const bool valid = j < cnt;
        float kf[VEC];
        if (valid) unpack16<T>(ld_act_stream16(kb + (size_t)j * DH + sub * VEC), kf);    // may be a draft-tail row appended by the previous kernel
        else {
#pragma unroll
            for (int v = 0; v < VEC; ++v) kf[v] = 0.f;
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float dot = 0.f;
#pragma unroll
            for (int v = 0; v < VEC; ++v) dot = fmaf(qf[g][v], kf[v], dot);
#pragma unroll
            for (int o = LPK / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
            if (valid && sub == 0) s_s[g][j] = dot;
        }
    }
    __syncthreads();

    // phase 2: chunk-local max and exp-sum per query head
    for (int g = warp; g < G; g += kAttnWarps) {
        float m = -INFINITY;
        for (int j = lane; j < cnt; j += 32) m = fmaxf(m, s_s[g][j]);
        m = warp_max(m);
        float l = 0.f;
        for (int j = lane; j < cnt; j += 32) {
            const float p = __expf(s_s[g][j] - m);
            s_s[g][j] = p;
            l += p;
        }
        l = warp_sum(l);
        if (lane == 0) { s_m[g] = m; s_l[g] = l; }
    }
    __syncthreads();

    // phase 3: unnormalised P.V
    float acc[G][VEC];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[g][v] = 0.f;
#pragma unroll 4
    for (int jb = warp * KPW; jb < cnt; jb += KPI) {
        const int j = jb + kgrp;
        if (j < cnt) {
            float vf[VEC];
            unpack16<T>(ld_act_stream16(vb + (size_t)j * DH + sub * VEC), vf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float p = s_s[g][j];
#pragma unroll
                for (int v = 0; v < VEC; ++v) acc[g][v] = fmaf(p, vf[v], acc[g][v]);
            }
        }
    }
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            float t = acc[g][v];
#pragma unroll
            for (int o = LPK; o < 32; o <<= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if (kgrp == 0) s_acc[warp][g][sub * VEC + v] = t;
        }
    __syncthreads();
    for (int i = tid; i < G * DH; i += kAttnWarps * 32) {
        const int g = i / DH, c = i % DH;
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) t += s_acc[w][g][c];
        part_o[(((size_t)b * Hq + kvh * G + g) * nchunk_max + chunk) * DH + c] = t;
    }
    if (tid < G) {
        const size_t pi = ((size_t)b * Hq + kvh * G + tid) * nchunk_max + chunk;
        part_ml[2 * pi] = s_m[tid];
        part_ml[2 * pi + 1] = s_l[tid];
    }
}

// One CTA of four warps per (sequence, query head): each warp merges a quarter of the chunks
// (attn_combine_range), warp 0 merges the four results.
template <typename T, int DPL>
__global__ void __launch_bounds__(128) attn_combine_kernel(const float* part_o, const float* part_ml,      // the previous kernel's output
                                                          const BatchMeta meta, int Hq, int dh, int nchunk_max, int chunk,
                                                          int extra_chunks, T* __restrict__ o) {
    const int head = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    pdl_wait();
    const int kv_len = meta.kv_len[head / Hq];
    const int nch = (kv_len + chunk - 1) / chunk + extra_chunks;
    const size_t p0 = (size_t)head * nchunk_max;
    const int per = (nch + 3) / 4;
    float M, den, acc[DPL];
    attn_combine_range<DPL, false>(part_o + p0 * dh, part_ml + 2 * p0, min(nch, warp * per), min(nch, (warp + 1) * per), dh, lane, M, den, acc);
    __shared__ float s_M[4], s_den[4], s_acc[4][DPL * 32];
    if (lane == 0) { s_M[warp] = M; s_den[warp] = den; }
#pragma unroll
    for (int v = 0; v < DPL; ++v) s_acc[warp][lane * DPL + v] = acc[v];
    __syncthreads();
    if (warp == 0) {
        const float Mx = fmaxf(fmaxf(s_M[0], s_M[1]), fmaxf(s_M[2], s_M[3]));
        float d = 0.f, out[DPL];
#pragma unroll
        for (int v = 0; v < DPL; ++v) out[v] = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float wgt = (s_M[w] == -INFINITY) ? 0.f : __expf(s_M[w] - Mx);
            d = fmaf(wgt, s_den[w], d);
#pragma unroll
            for (int v = 0; v < DPL; ++v) out[v] = fmaf(wgt, s_acc[w][lane * DPL + v], out[v]);
        }
        const float inv = (nch > 0 && d > 0.f) ? 1.0f / d : 0.f;
        if (lane * DPL < dh) {
#pragma unroll
            for (int v = 0; v < DPL; ++v) o[(size_t)head * dh + lane * DPL + v] = from_float<T>(out[v] * inv);
        }
    }
}

template <typename T>
static int attn_combine_dispatch(const float* part_o, const float* part_ml, const BatchMeta& meta, int B, int Hq, int dh,
                                 int nchunk_stride, int chunk, T* o, cudaStream_t stream, int extra = 0) {
    const int grid = B * Hq;
    switch (dh) {
        case 32: launch_pdl(attn_combine_kernel<T, 1>, dim3(grid), dim3(128), 0, stream, part_o, part_ml, meta, Hq, dh, nchunk_stride, chunk, extra, o); return 1;
        case 64: launch_pdl(attn_combine_kernel<T, 2>, dim3(grid), dim3(128), 0, stream, part_o, part_ml, meta, Hq, dh, nchunk_stride, chunk, extra, o); return 1;
        case 128: launch_pdl(attn_combine_kernel<T, 4>, dim3(grid), dim3(128), 0, stream, part_o, part_ml, meta, Hq, dh, nchunk_stride, chunk, extra, o); return 1;
        case 256: launch_pdl(attn_combine_kernel<T, 8>, dim3(grid), dim3(128), 0, stream, part_o, part_ml, meta, Hq, dh, nchunk_stride, chunk, extra, o); return 1;
        case 16: launch_pdl(attn_combine_kernel<T, 1>, dim3(grid), dim3(128), 0, stream, part_o, part_ml, meta, Hq, dh, nchunk_stride, chunk, extra, o); return 1;
        default: return -1;
    }
}

int launch_attn_combine(int dtype, const float* part_o, const float* part_ml, const BatchMeta& meta, int B, int Hq, int dh,
                        int nchunk_stride, int chunk, void* o, cudaStream_t stream, int extra_chunks) {
    if (B <= 0) return 0;
    return dtype == 0 ? attn_combine_dispatch<float>(part_o, part_ml, meta, B, Hq, dh, nchunk_stride, chunk, (float*)o, stream, extra_chunks)
                      : attn_combine_dispatch<bf16>(part_o, part_ml, meta, B, Hq, dh, nchunk_stride, chunk, (bf16*)o, stream, extra_chunks);
}

size_t attn_decode_scratch_bytes(int max_batch, int Hq, int dh, int max_kv) {
    const size_t nch = (size_t)(max_kv + kAttnMinChunk - 1) / kAttnMinChunk + 1;
    const size_t rows = (size_t)max_batch * Hq * nch;
    return rows * dh * sizeof(float) + rows * 2 * sizeof(float) + 256;
}

template <typename T, int G>
static int attn_dispatch_lpk(int lpk, dim3 grid, cudaStream_t stream, const T* q, const T* kc, const T* vc,
                             const BatchMeta& meta, int Hq, int Hkv, int cap, int nch, float scale, float* po, float* pml) {
    switch (lpk) {
        case 4: launch_pdl(attn_decode_kernel<T, G, 4>, grid, dim3(kAttnWarps * 32), 0, stream, q, kc, vc, meta, Hq, Hkv, cap, nch, scale, po, pml); return 1;
        case 8: launch_pdl(attn_decode_kernel<T, G, 8>, grid, dim3(kAttnWarps * 32), 0, stream, q, kc, vc, meta, Hq, Hkv, cap, nch, scale, po, pml); return 1;
        case 16: launch_pdl(attn_decode_kernel<T, G, 16>, grid, dim3(kAttnWarps * 32), 0, stream, q, kc, vc, meta, Hq, Hkv, cap, nch, scale, po, pml); return 1;
        case 32:
            if constexpr (G * 32 * VecOf<T>::N <= 1024) {   // static shared memory stays under 48 KB
                launch_pdl(attn_decode_kernel<T, G, 32>, grid, dim3(kAttnWarps * 32), 0, stream, q, kc, vc, meta, Hq, Hkv, cap, nch, scale, po, pml);
                return 1;
            } else {
                return -1;
            }
        default: return -1;
    }
}
template <typename T>
static int attn_dispatch(const void* q, const void* kc, const void* vc, const BatchMeta& meta, int B, int Hq, int Hkv,
                         int dh, int cap, int max_kv_len, void* scratch, void* o, cudaStream_t stream) {
    const int G = Hq / Hkv;
    const int lpk = dh / VecOf<T>::N;
    if (dh % VecOf<T>::N != 0) return -1;
    const int nch = (max_kv_len + kAttnChunk - 1) / kAttnChunk + 1;   // row stride of the partial buffers
    const int nch_launch = (max_kv_len + kAttnChunk - 1) / kAttnChunk;
    float* po = reinterpret_cast<float*>(scratch);
    float* pml = po + (size_t)B * Hq * nch * dh;
    const float scale = 1.0f / sqrtf((float)dh);
    int launched = 0;
    if (nch_launch > 0) {
        dim3 grid(nch_launch, Hkv, B);
        int rc;
        switch (G) {
            case 1: rc = attn_dispatch_lpk<T, 1>(lpk, grid, stream, (const T*)q, (const T*)kc, (const T*)vc, meta, Hq, Hkv, cap, nch, scale, po, pml); break;
            case 2: rc = attn_dispatch_lpk<T, 2>(lpk, grid, stream, (const T*)q, (const T*)kc, (const T*)vc, meta, Hq, Hkv, cap, nch, scale, po, pml); break;
            case 4: rc = attn_dispatch_lpk<T, 4>(lpk, grid, stream, (const T*)q, (const T*)kc, (const T*)vc, meta, Hq, Hkv, cap, nch, scale, po, pml); break;
            case 8: rc = attn_dispatch_lpk<T, 8>(lpk, grid, stream, (const T*)q, (const T*)kc, (const T*)vc, meta, Hq, Hkv, cap, nch, scale, po, pml); break;
            default: rc = -1;
        }
        if (rc < 0) return rc;
        launched += rc;
    }
    if (attn_combine_dispatch<T>(po, pml, meta, B, Hq, dh, nch, kAttnChunk, (T*)o, stream) < 0) return -1;
    return launched + 1;
}
int launch_attn_decode(int dtype, const void* q, const void* kcache, const void* vcache, const BatchMeta& meta,
                       int B, int Hq, int Hkv, int dh, int cap, int max_kv_len, void* scratch, void* o,
                       cudaStream_t stream) {
    if (B <= 0) return 0;
    return dtype == 0 ? attn_dispatch<float>(q, kcache, vcache, meta, B, Hq, Hkv, dh, cap, max_kv_len, scratch, o, stream)
                      : attn_dispatch<bf16>(q, kcache, vcache, meta, B, Hq, Hkv, dh, cap, max_kv_len, scratch, o, stream);
}

// ------------------------------------------------------------------------------------------------
// Arg-max finalisation of the LM head's per-block keys
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) argmax_finalize_kernel(const unsigned long long* partials, int nblk,       // the LM head's output
                                                               const BatchMeta meta, int32_t* __restrict__ tokens_out,
                                                               int tokens_out_stride, int32_t* __restrict__ last_token) {
    const int b = blockIdx.x;
    const bool release_early = gridDim.x > 8;      // as in the decode attention: early for large batches, at the end for small ones (measured)
    if (release_early) pdl_launch_dependents();
    pdl_wait();
    const unsigned long long* row = partials + (size_t)b * nblk;
    unsigned long long key = 0ull;
    for (int i0 = threadIdx.x; i0 < nblk; i0 += 4 * blockDim.x) {      // four independent loads in flight per thread
        unsigned long long k[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { const int i = i0 + j * blockDim.x; k[j] = i < nblk ? row[i] : 0ull; }
#pragma unroll
        for (int j = 0; j < 4; ++j) key = k[j] > key ? k[j] : key;
    }
    key = warp_max_u64(key);
    __shared__ unsigned long long s_k[32];
    if ((threadIdx.x & 31) == 0) s_k[threadIdx.x >> 5] = key;
    __syncthreads();
    if (threadIdx.x < 32) {
        key = threadIdx.x < (blockDim.x >> 5) ? s_k[threadIdx.x] : 0ull;
        key = warp_max_u64(key);
        if (threadIdx.x == 0) {
            const int tok = argmax_key_index(key);
            if (tokens_out != nullptr) tokens_out[(size_t)b * tokens_out_stride] = tok;
            if (BEAGLE_IN_BOUNDS(BEAGLE_SLOT_OK(meta.slot[b]))) last_token[meta.slot[b]] = tok;
        }
    }
    if (!release_early) pdl_launch_dependents();
}
int launch_argmax_finalize(const unsigned long long* partials, int nblk, const BatchMeta& meta, int B,
                           int32_t* tokens_out, int tokens_out_stride, int32_t* last_token, cudaStream_t stream) {
    if (B <= 0) return 0;
    const int threads = nblk >= 2048 ? 1024 : 256;
    launch_pdl(argmax_finalize_kernel, dim3(B), dim3(threads), 0, stream, partials, nblk, meta, tokens_out, tokens_out_stride, last_token);
    return 1;
}

// ------------------------------------------------------------------------------------------------
// Row arg-max over [rows, V] logits and greedy acceptance (Section 3)
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) row_argmax_partial_kernel(const T* __restrict__ logits, int V,
                                                                 unsigned long long* __restrict__ scratch) {
    constexpr int VEC = VecOf<T>::N;
    const int split = blockIdx.x, row = blockIdx.y;
    const T* z = logits + (size_t)row * V;
    int per = (V + kRowArgmaxSplit - 1) / kRowArgmaxSplit;
    per = (per + VEC - 1) / VEC * VEC;
    const int lo = split * per, hi = min(V, lo + per);
    unsigned long long key = 0ull;
    const bool aligned = (((size_t)row * V) % VEC == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15) == 0);
    if (aligned) {
        for (int i = lo + threadIdx.x * VEC; i < hi; i += blockDim.x * VEC) {
            if (i + VEC <= hi) {
                float f[VEC];
                unpack16<T>(ld_stream16(z + i), f);
#pragma unroll
                for (int v = 0; v < VEC; ++v) { const unsigned long long k = argmax_key(f[v], i + v); key = k > key ? k : key; }
            } else {
                for (int v = i; v < hi; ++v) { const unsigned long long k = argmax_key(to_float<T>(z[v]), v); key = k > key ? k : key; }
            }
        }
    } else {
        for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) {
            const unsigned long long k = argmax_key(to_float<T>(z[i]), i);
            key = k > key ? k : key;
        }
    }
    key = warp_max_u64(key);
    __shared__ unsigned long long s_k[8];
    if ((threadIdx.x & 31) == 0) s_k[threadIdx.x >> 5] = key;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) key = s_k[w] > key ? s_k[w] : key;
        scratch[(size_t)row * kRowArgmaxSplit + split] = key;
    }
}
__global__ void row_argmax_final_kernel(const unsigned long long* __restrict__ scratch, int rows, int32_t* __restrict__ ids) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    unsigned long long key = 0ull;
    for (int s = 0; s < kRowArgmaxSplit; ++s) { const unsigned long long o = scratch[(size_t)r * kRowArgmaxSplit + s]; key = o > key ? o : key; }
    ids[r] = argmax_key_index(key);
}
int launch_row_argmax(int logits_dtype, const void* logits, int rows, int V, unsigned long long* scratch,
                      int32_t* ids_out, cudaStream_t stream) {
    if (rows <= 0) return 0;
    int done = 0;
    while (done < rows) {                       // gridDim.y is limited to 65535
        const int n = min(rows - done, 32768);
        dim3 grid(kRowArgmaxSplit, n);
        if (logits_dtype == 0)
            row_argmax_partial_kernel<float><<<grid, 256, 0, stream>>>((const float*)logits + (size_t)done * V, V, scratch + (size_t)done * kRowArgmaxSplit);
        else
            row_argmax_partial_kernel<bf16><<<grid, 256, 0, stream>>>((const bf16*)logits + (size_t)done * V, V, scratch + (size_t)done * kRowArgmaxSplit);
        done += n;
    }
    row_argmax_final_kernel<<<(rows + 255) / 256, 256, 0, stream>>>(scratch, rows, ids_out);
    return (rows + 32767) / 32768 + 1;
}

// ------------------------------------------------------------------------------------------------
// Greedy verification from target logits in ONE launch (Section 3): CTA (slice, row) scans its slice
// of one logit row with 16-byte streaming loads, leaves one packed key in `keys[row][slice]` and takes
// a ticket of its sequence; the CTA that takes the sequence's last ticket reduces the (gamma + 1) x
// nsplit keys to the target's greedy tokens and walks the acceptance rule.  Nobody waits for anybody.
// `tickets` [B] must be zero before the first launch; the finishing CTA leaves them zero.
// The grid is sized to about one resident wave (8 CTAs of 256 threads per SM: the kernel is compiled
// for that); measured at 32 x 7 x 128256 fp32 logits, more and smaller slices only add per-CTA cost.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256, 8) verify_greedy_fused_kernel(const T* logits, int V, int nsplit, int per, int gamma,
                                                                     const int32_t* draft, unsigned long long* keys, int* tickets,
                                                                     int32_t* accept_len, int32_t* out_tokens) {
    constexpr int VEC = VecOf<T>::N;
    const int split = blockIdx.x, row = blockIdx.y;
    pdl_launch_dependents();
    pdl_wait();                      // the logits and the drafted tokens may be the output of the kernels before
    const int b = row / (gamma + 1);
    const T* z = logits + (size_t)row * V;
    const int lo = split * per, hi = min(V, lo + per);
    // Per thread a running (value, index): the indices a thread visits only grow, so a strict '>' keeps the lowest index of
    // equal values; NaN never compares greater; -0 and +0 compare equal.  The packed key then orders the threads' results
    // (key 0 = "saw nothing", below every real key).
    float bv = -INFINITY;
    int bi = -1;
    auto take = [&](float v, int i) {
        if (v > bv) { bv = v; bi = i; }
    };
    if (lo < hi) {
        // scalar head up to the first 16-byte boundary of the row's slice, vector body, scalar tail
        const uintptr_t addr = reinterpret_cast<uintptr_t>(z + lo);
        int head = (int)(((16 - (addr & 15)) & 15) / sizeof(T));
        if ((addr & (sizeof(T) - 1)) != 0 || head > hi - lo) head = hi - lo;
        const int body0 = lo + head;
        const int nvec = (hi - body0) / VEC;
        for (int i = lo + threadIdx.x; i < body0; i += 256) take(to_float<T>(z[i]), i);
        const T* zb = z + body0;
        int i = threadIdx.x;
        for (; i + 3 * 256 < nvec; i += 4 * 256) {       // four independent 16-byte loads in flight per thread
            uint4 u[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) u[j] = ld_act_stream16(zb + (size_t)(i + j * 256) * VEC);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float f[VEC];
                unpack16<T>(u[j], f);
#pragma unroll
                for (int v = 0; v < VEC; ++v) take(f[v], body0 + (i + j * 256) * VEC + v);
            }
        }
        for (; i < nvec; i += 256) {
            float f[VEC];
            unpack16<T>(ld_act_stream16(zb + (size_t)i * VEC), f);
#pragma unroll
            for (int v = 0; v < VEC; ++v) take(f[v], body0 + i * VEC + v);
        }
        for (int t = body0 + nvec * VEC + threadIdx.x; t < hi; t += 256) take(to_float<T>(z[t]), t);
        // a slice that holds nothing above -inf (only -inf / NaN) answers with its first index: thread 0 always visits it
        if (threadIdx.x == 0 && bi < 0) bi = lo;
    }
    unsigned long long key = bi >= 0 ? argmax_key(bv, bi) : 0ull;
    key = warp_max_u64(key);
    __shared__ unsigned long long s_k[8];
    __shared__ int s_last;
    __shared__ int32_t s_g[65];
    if ((threadIdx.x & 31) == 0) s_k[threadIdx.x >> 5] = key;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 1; w < 8; ++w) key = s_k[w] > key ? s_k[w] : key;
        keys[(size_t)row * nsplit + split] = key;
        __threadfence();                                  // the key is visible before the ticket is
        const int total = (gamma + 1) * nsplit;
        s_last = atomicAdd(&tickets[b], 1) == total - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // last CTA of sequence b: greedy token of each of its gamma + 1 rows (one warp per row, round robin)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = warp; r <= gamma; r += 8) {
        const unsigned long long* kr = keys + ((size_t)b * (gamma + 1) + r) * nsplit;
        unsigned long long k = 0ull;
        for (int s = lane; s < nsplit; s += 32) { const unsigned long long o = __ldcg(kr + s); k = o > k ? o : k; }
        k = warp_max_u64(k);
        if (lane == 0) s_g[r] = argmax_key_index(k);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int a = 0;
        while (a < gamma && draft[(size_t)b * gamma + a] == s_g[a]) ++a;
        accept_len[b] = a;
        s_last = a;                                       // (re-used) the accepted length, for the token rows below
        tickets[b] = 0;                                   // ready for the next call
    }
    __syncthreads();
    if ((int)threadIdx.x <= gamma)
        out_tokens[(size_t)b * (gamma + 1) + threadIdx.x] = (int)threadIdx.x <= s_last ? s_g[threadIdx.x] : -1;
}

int verify_fused_splits(int rows, int V, int sm_count) {
    // one resident wave of 8 CTAs per SM, slices of at least 4096 logits, at most kVerifyMaxSplit per row
    int s = (sm_count * 8) / (rows > 0 ? rows : 1);
    const int cap = (V + 4095) / 4096;
    s = s < cap ? s : cap;
    s = s < kVerifyMaxSplit ? s : kVerifyMaxSplit;
    return s < 1 ? 1 : s;
}

int launch_verify_greedy_fused(int logits_dtype, const void* logits, int B, int gamma, int V, const int32_t* draft,
                               unsigned long long* keys, int* tickets, int sm_count, int32_t* accept_len, int32_t* out_tokens,
                               cudaStream_t stream) {
    if (B <= 0) return 0;
    const int rows = B * (gamma + 1);
    const int nsplit = verify_fused_splits(rows, V, sm_count);
    const int vec = logits_dtype == 0 ? 4 : 8;
    int per = (V + nsplit - 1) / nsplit;
    per = (per + vec - 1) / vec * vec;
    dim3 grid(nsplit, rows);
    if (logits_dtype == 0)
        launch_pdl(verify_greedy_fused_kernel<float>, grid, dim3(256), 0, stream, (const float*)logits, V, nsplit, per, gamma, draft, keys, tickets, accept_len, out_tokens);
    else
        launch_pdl(verify_greedy_fused_kernel<bf16>, grid, dim3(256), 0, stream, (const bf16*)logits, V, nsplit, per, gamma, draft, keys, tickets, accept_len, out_tokens);
    return 1;
}

__global__ void accept_kernel(const int32_t* __restrict__ draft, const int32_t* __restrict__ target_ids, int B, int gamma,
                              int32_t* __restrict__ accept_len, int32_t* __restrict__ out_tokens) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int32_t* g = target_ids + (size_t)b * (gamma + 1);
    const int32_t* t = draft + (size_t)b * gamma;
    int a = 0;
    while (a < gamma && t[a] == g[a]) ++a;
    accept_len[b] = a;
    for (int r = 0; r <= gamma; ++r) out_tokens[(size_t)b * (gamma + 1) + r] = r <= a ? g[r] : -1;
}
int launch_accept(const int32_t* draft, const int32_t* target_ids, int B, int gamma, int32_t* accept_len,
                  int32_t* out_tokens, cudaStream_t stream) {
    if (B <= 0) return 0;
    accept_kernel<<<(B + 63) / 64, 64, 0, stream>>>(draft, target_ids, B, gamma, accept_len, out_tokens);
    return 1;
}

}  // namespace beagle
