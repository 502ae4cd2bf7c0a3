// Draft/verify acceptance under sampling (Section 3): draft i is accepted with probability
// min(1, p_i(t_i) / q_i(t_i)); at the first rejection j (or j = gamma + 1) one token is drawn from the
// normalised max(0, p_j - q_j) (from p_{gamma+1} when nothing was rejected).  p = softmax(target / T),
// q = softmax(draft / T).  The uniforms are inputs, so the kernels are deterministic.
//
// Two launches:
//   1. log-sum-exp of every logit row, rows split into slices of about equal bytes (the only pass that reads all logits);
//   2. eight CTAs per sequence: acceptance tests, accept_len, the accepted drafts and the row j to resample at; the residual
//      mass of row j in 64 chunks (fixed summation order); the CTA that finishes last: inverse CDF -- locate the chunk, then a
//      scan inside it.
#include "kernels.h"

namespace beagle {

namespace {

constexpr int kLseSplit = 16;
constexpr int kChunks = 64;

struct VsScratch {
    float2* lse_p;        // [B*(gamma+1)][kLseSplit]  (max, sum exp) of the target rows
    float2* lse_q;        // [gamma*B][kLseSplit]       of the draft rows
    float* chunk_w;       // [B][kChunks] residual mass per chunk of the row to resample at
    float* chunk_p;       // [B][kChunks] target mass per chunk (fallback when no residual mass is left)
};

// One launch covers the target rows (type T, blockIdx.y < rows_p) and the draft rows (fp32).
template <typename T, typename U>
__device__ __forceinline__ void lse_scan_row(const U* z, int V, int split, int nsplit, float inv_t, bool base_aligned,
                                             size_t row_elems, float& m, float& s) {
    constexpr int VEC = VecOf<U>::N;
    int per = (V + nsplit - 1) / nsplit;
    per = (per + VEC - 1) / VEC * VEC;
    const int lo = split * per, hi = min(V, lo + per);
    auto add = [&](float v) {
        v *= inv_t;
        if (v == -INFINITY) return;                               // a masked entry carries no mass
        if (v > m) { s = s * __expf(m - v) + 1.f; m = v; }      // m = -inf: s = 0 * exp(-inf) + 1
        else s += __expf(v - m);
    };
    if (base_aligned && row_elems % VEC == 0) {
        int i = lo + threadIdx.x * VEC;
        const int stride = blockDim.x * VEC;
        for (; i + 3 * stride + VEC <= hi; i += 4 * stride) {          // four independent 16-byte loads in flight per thread
            uint4 u[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) u[j] = ld_act_stream16(z + i + j * stride);
#pragma unroll
            for (int j = 0; j < 4; ++j) {                               // one piece at a time: few live registers, more CTAs per SM
                float f[VEC];
                unpack16<U>(u[j], f);
                float vm = f[0];
#pragma unroll
                for (int v = 1; v < VEC; ++v) vm = fmaxf(vm, f[v]);
                vm *= inv_t;
                if (vm > m) { s *= __expf(m - vm); m = vm; }           // one rescale per 16 bytes; m = -inf: s stays 0
                if (m != -INFINITY) {
#pragma unroll
                    for (int v = 0; v < VEC; ++v) s += __expf(f[v] * inv_t - m);
                }
            }
        }
        for (; i < hi; i += stride) {
            if (i + VEC <= hi) {
                float f[VEC];
                unpack16<U>(ld_act_stream16(z + i), f);
                float vm = f[0];
#pragma unroll
                for (int v = 1; v < VEC; ++v) vm = fmaxf(vm, f[v]);
                vm *= inv_t;
                if (vm > m) { s *= __expf(m - vm); m = vm; }       // one rescale per 16 bytes; m = -inf: s stays 0
                if (m != -INFINITY) {
#pragma unroll
                    for (int v = 0; v < VEC; ++v) s += __expf(f[v] * inv_t - m);
                }
            } else {
                for (int v = i; v < hi; ++v) add(to_float<U>(z[v]));
            }
        }
    } else {
        for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) add(to_float<U>(z[i]));
    }
}

// Grid: blockIdx.x < rows_p * nsplit_p are the target rows' slices (type T), the rest the draft rows' slices (fp32); the two
// kinds get slice counts of their own so that a slice holds about the same BYTES whatever the row's type.
template <typename T>
__global__ void __launch_bounds__(256, 5) vs_lse_partial_kernel(const T* zp, int rows_p, int nsplit_p, const float* zq,
                                                               int nsplit_q, int V, float inv_t, float2* part_p, float2* part_q) {
    // the grid is sized to about one resident wave (every further CTA costs more in launch, first-load latency and reduction
    // than its shorter slice saves); the unused partial slots are filled with "no mass"
    int row, split, nsplit;
    float m = -INFINITY, s = 0.f;
    float2* part;
    pdl_launch_dependents();
    pdl_wait();                              // the logits may be the output of the kernel before (a draft step's LM head)
    if ((int)blockIdx.x < rows_p * nsplit_p) {
        row = blockIdx.x / nsplit_p; split = blockIdx.x % nsplit_p; nsplit = nsplit_p;
        lse_scan_row<T, T>(zp + (size_t)row * V, V, split, nsplit, inv_t, (reinterpret_cast<uintptr_t>(zp) & 15) == 0, (size_t)row * V, m, s);
        part = part_p;
    } else {
        const int x = blockIdx.x - rows_p * nsplit_p;
        row = x / nsplit_q; split = x % nsplit_q; nsplit = nsplit_q;
        lse_scan_row<T, float>(zq + (size_t)row * V, V, split, nsplit, inv_t, (reinterpret_cast<uintptr_t>(zq) & 15) == 0, (size_t)row * V, m, s);
        part = part_q;
    }
    // merge (m, s) pairs: warp, then CTA, always in the same order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
        const float M = fmaxf(m, m2);
        s = (M == -INFINITY) ? 0.f : s * __expf(m - M) + s2 * __expf(m2 - M);
        m = M;
    }
    __shared__ float sm[8], ss[8];
    if ((threadIdx.x & 31) == 0) { sm[threadIdx.x >> 5] = m; ss[threadIdx.x >> 5] = s; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float M = sm[0], S = ss[0];
        for (int w = 1; w < 8; ++w) {
            const float M2 = fmaxf(M, sm[w]);
            S = (M2 == -INFINITY) ? 0.f : S * __expf(M - M2) + ss[w] * __expf(sm[w] - M2);
            M = M2;
        }
        part[(size_t)row * kLseSplit + split] = make_float2(M, S);
        if (split == 0)
            for (int e = nsplit; e < kLseSplit; ++e) part[(size_t)row * kLseSplit + e] = make_float2(-INFINITY, 0.f);
    }
}

__device__ __forceinline__ float lse_of(const float2* part) {
    float M = -INFINITY;
    for (int i = 0; i < kLseSplit; ++i) M = fmaxf(M, part[i].x);
    float S = 0.f;
    for (int i = 0; i < kLseSplit; ++i) S += (part[i].x == -INFINITY) ? 0.f : part[i].y * __expf(part[i].x - M);
    return M + __logf(S);
}

constexpr int kFinThreads = 256;
constexpr int kSeqCtas = 8;           // CTAs per sequence in the second launch
constexpr int kChunksPerCta = kChunks / kSeqCtas, kWarpsPerChunk = (kFinThreads / 32) / kChunksPerCta;
constexpr int kPiece = 8;             // a chunk is a whole number of 8-entry pieces, so that a thread's loads are 16-byte vectors

// Entries [v0, v0 + 8) of a logit row as floats (16-byte loads when the row allows them; entries past V read as -inf: no mass).
template <typename U>
__device__ __forceinline__ void load_piece(const U* row, int v0, int V, bool vec, float (&f)[kPiece]) {
    if (vec) {
        if (sizeof(U) == 2) {
            unpack16<U>(ld_act16(row + v0), f);
        } else {
            unpack16<U>(ld_act16(row + v0), f);
            unpack16<U>(ld_act16(row + v0 + 4), f + 4);
        }
    } else {
#pragma unroll
        for (int j = 0; j < kPiece; ++j) f[j] = v0 + j < V ? to_float<U>(row[v0 + j]) : -INFINITY;
    }
}

// Residual weights w = max(0, p - q) and target probabilities p of one piece of the row to resample at.
template <typename T>
__device__ __forceinline__ void residual_piece(const T* zp, const float* zq, int v0, int V, bool vec, float inv_t, float lse_p, float lse_q,
                                               float (&w)[kPiece], float (&p)[kPiece]) {
    float fp[kPiece], fq[kPiece];
    load_piece<T>(zp, v0, V, vec, fp);
    if (zq != nullptr) load_piece<float>(zq, v0, V, vec, fq);
#pragma unroll
    for (int j = 0; j < kPiece; ++j) {
        p[j] = __expf(fp[j] * inv_t - lse_p);                       // exp(-inf) = 0 past the row's end
        const float q = (zq != nullptr) ? __expf(fq[j] * inv_t - lse_q) : 0.f;
        w[j] = fmaxf(0.f, p[j] - q);
    }
}

// Everything after the log-sum-exp pass; grid (kSeqCtas, sequences).  Every CTA of a sequence repeats the acceptance tests
// (warp 0: lane i evaluates position i, all positions at once in rounds of 32; the first failing position is the accepted
// length a), then its warps sum the residual mass of row a over the CTA's chunks (lane-strided pieces, then a shuffle tree: a
// fixed order).  The CTA that finishes last for its sequence -- a ticket in global memory, reset by that CTA -- locates the
// chunk whose cumulative mass first exceeds u * total and scans inside it.
template <typename T>
__global__ void __launch_bounds__(kFinThreads) vs_finish_kernel(const int32_t* __restrict__ draft, const float* zq_all, const T* zp_all, int B, int gamma,
                                                               int V, float inv_t, const float* __restrict__ u_accept,
                                                               const float* __restrict__ u_resample, VsScratch sc, int* tickets, int32_t* accept_len,
                                                               int32_t* out_tokens) {
    const int part = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ float s_cw[kChunks], s_warp[kFinThreads / 32], s_warp_p[kFinThreads / 32];
    __shared__ int s_a, s_chunk, s_use_p, s_pick, s_last, s_is_last;
    __shared__ float s_lse_p, s_lse_q, s_before, s_target;
    pdl_launch_dependents();
    pdl_wait();
    if (warp == 0) {
        int a = gamma;
        for (int i0 = 0; i0 < gamma && a == gamma; i0 += 32) {
            const int i = i0 + lane;
            bool pass = true;
            if (i < gamma) {
                const int t = min(max(draft[(size_t)b * gamma + i], 0), V - 1);
                const float lp = to_float<T>(zp_all[((size_t)b * (gamma + 1) + i) * V + t]) * inv_t - lse_of(sc.lse_p + ((size_t)b * (gamma + 1) + i) * kLseSplit);
                const float lq = zq_all[((size_t)i * B + b) * V + t] * inv_t - lse_of(sc.lse_q + ((size_t)i * B + b) * kLseSplit);
                const float ratio = fminf(1.f, __expf(lp - lq));
                pass = u_accept[(size_t)b * gamma + i] < ratio;
            }
            const unsigned fail = ~__ballot_sync(0xffffffffu, pass);
            if (fail) a = i0 + __ffs(fail) - 1;
        }
        if (part == 0) {
            for (int r = lane; r <= gamma; r += 32)
                if (r != a) out_tokens[(size_t)b * (gamma + 1) + r] = r < a ? draft[(size_t)b * gamma + r] : -1;
            if (lane == 0) accept_len[b] = a;
        }
        if (lane == 0) {
            s_a = a;
            s_lse_p = lse_of(sc.lse_p + ((size_t)b * (gamma + 1) + a) * kLseSplit);
            s_lse_q = a < gamma ? lse_of(sc.lse_q + ((size_t)a * B + b) * kLseSplit) : INFINITY;   // unused: no draft row
            s_pick = 0x7fffffff;
            s_last = -1;
        }
    }
    __syncthreads();
    const int a = s_a;
    const T* zp = zp_all + ((size_t)b * (gamma + 1) + a) * V;
    const float* zq = a < gamma ? zq_all + ((size_t)a * B + b) * V : nullptr;
    const float lse_p = s_lse_p, lse_q = s_lse_q;
    // 16-byte loads need every row to start on a 16-byte boundary and to hold whole pieces
    const bool vec = V % kPiece == 0 && ((reinterpret_cast<uintptr_t>(zp_all) | reinterpret_cast<uintptr_t>(zq_all)) & 15) == 0;
    const int row_pieces = (V + kPiece - 1) / kPiece;
    const int ppc = (row_pieces + kChunks - 1) / kChunks;            // pieces per chunk
    {
        // this CTA's chunks, kWarpsPerChunk warps on each: a warp sums every kWarpsPerChunk-th group of 32 pieces
        const int c = part * kChunksPerCta + warp / kWarpsPerChunk, sub = warp % kWarpsPerChunk;
        const int p_lo = c * ppc, p_hi = min(row_pieces, p_lo + ppc);
        float sw = 0.f, sp = 0.f;
#pragma unroll 2
        for (int piece = p_lo + sub * 32 + lane; piece < p_hi; piece += 32 * kWarpsPerChunk) {
            float w[kPiece], p[kPiece];
            residual_piece<T>(zp, zq, piece * kPiece, V, vec, inv_t, lse_p, lse_q, w, p);
#pragma unroll
            for (int j = 0; j < kPiece; ++j) { sw += w[j]; sp += p[j]; }
        }
        sw = warp_sum(sw);
        sp = warp_sum(sp);
        if (lane == 0) { s_warp[warp] = sw; s_warp_p[warp] = sp; }
        __syncthreads();
        if (tid < kChunksPerCta) {
            float tw = 0.f, tp = 0.f;
            for (int k = 0; k < kWarpsPerChunk; ++k) { tw += s_warp[tid * kWarpsPerChunk + k]; tp += s_warp_p[tid * kWarpsPerChunk + k]; }
            sc.chunk_w[(size_t)b * kChunks + part * kChunksPerCta + tid] = tw;
            sc.chunk_p[(size_t)b * kChunks + part * kChunksPerCta + tid] = tp;
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int prev = atomicAdd(&tickets[b], 1);
        s_is_last = (prev == (int)gridDim.x - 1);
        if (s_is_last) tickets[b] = 0;                              // ready for the next call
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();
    if (tid < kChunks) s_cw[tid] = __uint_as_float(ld_act32(sc.chunk_w + (size_t)b * kChunks + tid));
    __syncthreads();
    if (tid == 0) {
        float total = 0.f;
        for (int c = 0; c < kChunks; ++c) total += s_cw[c];
        s_use_p = !(total > 0.f);                   // no residual mass (p == q): draw from p instead
    }
    __syncthreads();
    const bool use_p = s_use_p != 0;
    if (use_p) {
        if (tid < kChunks) s_cw[tid] = __uint_as_float(ld_act32(sc.chunk_p + (size_t)b * kChunks + tid));
        __syncthreads();
    }
    if (tid == 0) {
        float total = 0.f;
        for (int c = 0; c < kChunks; ++c) total += s_cw[c];
        const float target = u_resample[b] * total;
        // chunk whose cumulative mass first exceeds the target (the last non-empty chunk if rounding leaves none)
        float before = 0.f;
        int chunk = -1, last_nonempty = 0;
        for (int c = 0; c < kChunks; ++c) {
            if (s_cw[c] > 0.f) last_nonempty = c;
            if (chunk < 0 && before + s_cw[c] > target) chunk = c;
            if (chunk < 0) before += s_cw[c];
        }
        if (chunk < 0) {
            chunk = last_nonempty;
            before = 0.f;
            for (int c = 0; c < chunk; ++c) before += s_cw[c];
        }
        s_chunk = chunk; s_before = before; s_target = target;
    }
    __syncthreads();
    const int lo = s_chunk * ppc * kPiece, hi = min(V, lo + ppc * kPiece);
    const float target = s_target;
    float run = s_before;                           // mass before the current pass, identical in every thread
    for (int p0 = lo; p0 < hi; p0 += kFinThreads * kPiece) {
        // this thread's piece
        const int v0 = p0 + tid * kPiece;
        float w[kPiece], p[kPiece], seg = 0.f;
        if (v0 < hi) residual_piece<T>(zp, zq, v0, V, vec, inv_t, lse_p, lse_q, w, p);
#pragma unroll
        for (int j = 0; j < kPiece; ++j) {
            w[j] = v0 + j < hi ? (use_p ? p[j] : w[j]) : 0.f;
            seg += w[j];
        }
        // exclusive scan of the piece sums over the CTA
        float inc = seg;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) s_warp[warp] = inc;
        __syncthreads();
        float wbase = 0.f, pass_total = 0.f;
        for (int k = 0; k < kFinThreads / 32; ++k) { if (k < warp) wbase += s_warp[k]; pass_total += s_warp[k]; }
        float c = run + wbase + inc - seg;          // mass before this thread's piece
        int mine = 0x7fffffff, last = -1;
#pragma unroll
        for (int j = 0; j < kPiece; ++j) {
            if (v0 + j < hi) {
                c += w[j];
                if (w[j] > 0.f) last = v0 + j;
                if (mine == 0x7fffffff && c > target) mine = v0 + j;
            }
        }
        if (mine != 0x7fffffff) atomicMin(&s_pick, mine);
        if (last >= 0) atomicMax(&s_last, last);
        __syncthreads();
        if (s_pick != 0x7fffffff) break;
        run += pass_total;
        __syncthreads();
    }
    if (tid == 0) {
        int picked = s_pick;
        if (picked == 0x7fffffff) picked = s_last >= 0 ? s_last : lo;   // rounding: the target lies past the last entry with mass
        out_tokens[(size_t)b * (gamma + 1) + a] = picked;
    }
}

VsScratch carve(void* scratch, int B, int gamma) {
    VsScratch s;
    char* p = static_cast<char*>(scratch);
    auto take = [&](size_t bytes) { char* at = p; p += (bytes + 255) / 256 * 256; return at; };
    s.lse_p = reinterpret_cast<float2*>(take((size_t)B * (gamma + 1) * kLseSplit * sizeof(float2)));
    s.lse_q = reinterpret_cast<float2*>(take((size_t)B * (gamma > 0 ? gamma : 1) * kLseSplit * sizeof(float2)));
    s.chunk_w = reinterpret_cast<float*>(take((size_t)B * kChunks * sizeof(float)));
    s.chunk_p = reinterpret_cast<float*>(take((size_t)B * kChunks * sizeof(float)));
    return s;
}

template <typename T>
int run_verify_sample(const int32_t* draft, const float* zq, const T* zp, int B, int gamma, int V, float temperature, const float* u_accept,
                      const float* u_resample, void* scratch, int* tickets, int32_t* accept_len, int32_t* out_tokens, int sm_count, cudaStream_t stream) {
    const VsScratch sc = carve(scratch, B, gamma);
    const float inv_t = 1.0f / temperature;
    const int rows_p = B * (gamma + 1), rows_q = gamma * B;
    static int per_sm = 0;                                        // resident CTAs of this instantiation per SM (same on every B200)
    if (per_sm == 0 && (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, vs_lse_partial_kernel<T>, 256, 0) != cudaSuccess || per_sm < 1)) {
        cudaGetLastError();
        per_sm = 4;
    }
    // slices: one resident wave, none shorter than 4096 logits; a draft row (fp32) gets as many times the slices of a target row as
    // its elements are wider, so that every CTA scans about the same bytes
    const int wide = (int)(sizeof(float) / sizeof(T));
    const int cap = (V + 4095) / 4096 < kLseSplit ? (V + 4095) / 4096 : kLseSplit;
    int sp = (per_sm * sm_count) / (rows_p + wide * rows_q);
    sp = sp < 1 ? 1 : sp;
    int sq = sp * wide;
    sp = sp > cap ? cap : sp;
    sq = sq > cap ? cap : sq;
    // two dependent launches: each kernel is resident and waiting when the one before it ends
    launch_pdl(vs_lse_partial_kernel<T>, dim3(rows_p * sp + rows_q * sq), dim3(256), 0, stream, zp, rows_p, sp, zq, sq, V, inv_t, sc.lse_p, sc.lse_q);
    launch_pdl(vs_finish_kernel<T>, dim3(kSeqCtas, B), dim3(kFinThreads), 0, stream, draft, zq, zp, B, gamma, V, inv_t, u_accept, u_resample, sc, tickets,
               accept_len, out_tokens);
    return 2;
}

}  // namespace

size_t verify_sample_scratch_bytes(int max_batch, int max_gamma) {
    const size_t rows_p = (size_t)max_batch * (max_gamma + 1), rows_q = (size_t)max_batch * (max_gamma > 0 ? max_gamma : 1);
    return (rows_p + rows_q) * kLseSplit * sizeof(float2) + (size_t)max_batch * 2 * kChunks * sizeof(float) + 4 * 256;
}

int launch_verify_sample(int logits_dtype, const int32_t* draft, const float* draft_logits, const void* target_logits, int B, int gamma, int V,
                         float temperature, const float* u_accept, const float* u_resample, void* scratch, int* tickets, int32_t* accept_len,
                         int32_t* out_tokens, int sm_count, cudaStream_t stream) {
    if (B <= 0) return 0;
    return logits_dtype == 0
        ? run_verify_sample<float>(draft, draft_logits, static_cast<const float*>(target_logits), B, gamma, V, temperature, u_accept,
                                   u_resample, scratch, tickets, accept_len, out_tokens, sm_count, stream)
        : run_verify_sample<bf16>(draft, draft_logits, static_cast<const bf16*>(target_logits), B, gamma, V, temperature, u_accept,
                                  u_resample, scratch, tickets, accept_len, out_tokens, sm_count, stream);
}

}  // namespace beagle
