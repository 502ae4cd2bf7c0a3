// Device-side bookkeeping of dynamic-tree drafting (the dynamic draft attention tree the paper's
// experiments adopt: top-k expansion scored by cumulative log-probability, top-N rerank) and greedy
// acceptance along tree paths.  Everything stays on the device, so a whole tree is drafted without a
// host synchronisation: the forwards of the frontier nodes are the ordinary serve-time kernels, fed
// from the arrays these kernels maintain.
//
//   topk_partial_kernel   per forwarded row and vocabulary slice: (max, exp-sum) of its logits and its k best keys
//   tree_expand_kernel    per row the log-sum-exp and the k best children; appends the k*k children, picks the next
//                         frontier, builds its ancestor lists
//   tree_rerank_kernel    keeps the n best nodes overall, in creation order, parents re-indexed
//   attn_tail_kernel      attention partial over a node's ancestor draft states (an extra split-KV chunk)
//   tree_verify_kernel    walks the tree along the target's greedy tokens
#include "kernels.h"

namespace beagle {

namespace {

__device__ __forceinline__ unsigned long long block_max_u64(unsigned long long key, unsigned long long* s_k) {
    key = warp_max_u64(key);
    const int warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_k[warp] = key;
    __syncthreads();
    unsigned long long r = s_k[0];
    for (int w = 1; w < nwarp; ++w) r = s_k[w] > r ? s_k[w] : r;
    return r;
}

__device__ __forceinline__ float key_value(unsigned long long key) {      // inverse of argmax_key's value transform
    const uint32_t u = static_cast<uint32_t>(key >> 32);
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

constexpr int kTopkSplitElems = 4096;        // logits per CTA of the first pass
constexpr int kTopkPerThread = kTopkSplitElems / 256;

// The k largest of the keys a warp's lanes hold (n_mine each), in decreasing order: round j takes the largest key below
// round j-1's (keys are distinct: the index is part of them).  Lane 0 gets them through `out`.
template <int N>
__device__ __forceinline__ void warp_topk(const unsigned long long (&mine)[N], int k, unsigned long long* out) {
    unsigned long long prev = ~0ull;
    for (int j = 0; j < k; ++j) {
        unsigned long long best = 0ull;
#pragma unroll
        for (int e = 0; e < N; ++e)
            if (mine[e] < prev && mine[e] > best) best = mine[e];
        best = warp_max_u64(best);
        if ((threadIdx.x & 31) == 0) out[j] = best;
        prev = best;
    }
}

// Pass 1, grid (splits, rows): the CTA holds its slice of the row in registers (16 logits per thread), computes the
// slice's (max, exp-sum) and its k best keys: every warp selects the k best of its 512 logits with shuffles only, then
// warp 0 selects among the eight warps' candidates.
__global__ void __launch_bounds__(256) topk_partial_kernel(const float* logits, int V, int k, int per, float2* lse_part,
                                                          unsigned long long* key_part) {
    __shared__ unsigned long long s_k[8][kTreeMaxTopk];
    __shared__ float s_f[8];
    const int split = blockIdx.x, row = blockIdx.y, nsplit = gridDim.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    pdl_wait();                                                 // the logits are the previous kernel's output
    const int lo = split * per, hi = min(V, lo + per), n = max(0, hi - lo);
    const float* z = logits + (size_t)row * V + lo;
    float v[kTopkPerThread];
    unsigned long long key[kTopkPerThread];
    float m = -INFINITY;
#pragma unroll
    for (int e = 0; e < kTopkPerThread; ++e) {
        const int i = threadIdx.x + e * 256;
        v[e] = i < n ? z[i] : -INFINITY;
        key[e] = i < n ? argmax_key(v[e], lo + i) : 0ull;
        m = fmaxf(m, v[e]);
    }
    m = warp_max(m);
    if (lane == 0) s_f[warp] = m;
    __syncthreads();
    m = s_f[0];
    for (int w = 1; w < 8; ++w) m = fmaxf(m, s_f[w]);
    __syncthreads();
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < kTopkPerThread; ++e)
        if (threadIdx.x + e * 256 < n) s += __expf(v[e] - m);
    s = warp_sum(s);
    if (lane == 0) s_f[warp] = s;
    warp_topk(key, k, s_k[warp]);
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += s_f[w];
        lse_part[(size_t)row * nsplit + split] = make_float2(m, t);
    }
    if (warp == 0) {
        unsigned long long cand[8 * kTreeMaxTopk / 32];
#pragma unroll
        for (int e = 0; e < 8 * kTreeMaxTopk / 32; ++e) {
            const int i = lane + e * 32;                         // candidate i = warp i / k, rank i % k
            cand[e] = i < 8 * k ? s_k[i / k][i % k] : 0ull;
        }
        __shared__ unsigned long long s_out[kTreeMaxTopk];
        warp_topk(cand, k, s_out);
        __syncwarp();
        if (lane < k) key_part[((size_t)row * nsplit + split) * k + lane] = s_out[lane];
    }
}

// Pass 2 and the tree's growth in ONE CTA (warp r = forwarded row r): the row's log-sum-exp and its k best children among the
// slices' candidates; then, level 0: the root's children become nodes 0..k-1 and the first frontier (ancestor list = the
// root's state, tail position 0); level e >= 1: the rows of forward e were the frontier, their k*k children are appended at
// `base`, the k best (score, then creation order) become the next frontier, whose ancestor lists are the parent's list plus
// the parent's own state (tail position 1 + (e-1)*k + parent row).
__global__ void __launch_bounds__(32 * kTreeMaxTopk) tree_expand_kernel(TreeArrays t, int nsplit, int k, int rows, int level, int base) {
    __shared__ int s_tok[kTreeMaxTopk * kTreeMaxTopk];
    __shared__ float s_lq[kTreeMaxTopk * kTreeMaxTopk];
    __shared__ unsigned long long s_key[kTreeMaxTopk * kTreeMaxTopk];
    __shared__ unsigned long long s_best[kTreeMaxTopk];
    __shared__ int s_anc[kTreeMaxTopk][kTreeMaxDepth + 1];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_launch_dependents();
    pdl_wait();
    if (warp < rows) {
        const float2* lp = t.topk_lse + (size_t)warp * nsplit;
        float M = -INFINITY;
        for (int i = lane; i < nsplit; i += 32) M = fmaxf(M, lp[i].x);
        M = warp_max(M);
        float S = 0.f;
        for (int i = lane; i < nsplit; i += 32) {
            const float2 p = lp[i];
            S += (p.x == -INFINITY) ? 0.f : p.y * __expf(p.x - M);
        }
        S = warp_sum(S);
        const float lse = M + __logf(S);
        const unsigned long long* cand = t.topk_keys + (size_t)warp * nsplit * k;
        const int ncand = nsplit * k;
        constexpr int kHeld = 16;                              // candidates a lane keeps in registers (512 per row: 32 slices of 16)
        unsigned long long held[kHeld];
#pragma unroll
        for (int e = 0; e < kHeld; ++e) held[e] = lane + e * 32 < ncand ? cand[lane + e * 32] : 0ull;
        unsigned long long prev = ~0ull;
        for (int j = 0; j < k; ++j) {
            unsigned long long best = 0ull;
#pragma unroll
            for (int e = 0; e < kHeld; ++e)
                if (held[e] < prev && held[e] > best) best = held[e];
            for (int i = lane + kHeld * 32; i < ncand; i += 32) {      // larger vocabularies: the rest from memory
                const unsigned long long key = cand[i];
                if (key < prev && key > best) best = key;
            }
            best = warp_max_u64(best);
            if (lane == 0) {
                s_tok[warp * k + j] = best != 0ull ? argmax_key_index(best) : 0;
                s_lq[warp * k + j] = best != 0ull ? key_value(best) - lse : -INFINITY;
            }
            prev = best;
        }
    }
    if (level > 0 && tid < k)
        for (int a = 0; a < level; ++a) s_anc[tid][a] = t.frontier_anc[tid * (kTreeMaxDepth + 1) + a];
    __syncthreads();
    if (level == 0) {
        if (tid < k) {
            t.node_tok[tid] = s_tok[tid];
            t.node_par[tid] = -1;
            t.node_score[tid] = s_lq[tid];
            t.frontier_node[tid] = tid;
            t.frontier_tok[tid] = s_tok[tid];
            t.frontier_anc[tid * (kTreeMaxDepth + 1)] = 0;
        }
        return;
    }
    const int nnew = k * k;
    if (tid < nnew) {
        const int f = t.frontier_node[tid / k];
        const float score = t.node_score[f] + s_lq[tid];
        t.node_tok[base + tid] = s_tok[tid];
        t.node_par[base + tid] = f;
        t.node_score[base + tid] = score;
        s_key[tid] = argmax_key(score, tid);
    }
    __syncthreads();
    if (warp == 0) {
        unsigned long long mine[kTreeMaxTopk * kTreeMaxTopk / 32];
#pragma unroll
        for (int e = 0; e < kTreeMaxTopk * kTreeMaxTopk / 32; ++e) mine[e] = lane + e * 32 < nnew ? s_key[lane + e * 32] : 0ull;
        warp_topk(mine, k, s_best);
    }
    __syncthreads();
    if (tid < k) {
        const int i = argmax_key_index(s_best[tid]), r = i / k;
        t.frontier_node[tid] = base + i;
        t.frontier_tok[tid] = s_tok[i];
        for (int a = 0; a < level; ++a) t.frontier_anc[tid * (kTreeMaxDepth + 1) + a] = s_anc[r][a];
        t.frontier_anc[tid * (kTreeMaxDepth + 1) + level] = 1 + (level - 1) * k + r;
    }
}

// Keeps the n best nodes overall, in creation order, parents re-indexed.  A node's rank is the number of nodes with a larger
// key (score, then creation order); the kept ones are those of rank < n, and a kept node's place in the output is the number
// of kept nodes created before it.
__global__ void __launch_bounds__(1024) tree_rerank_kernel(TreeArrays t, int total, int n, int32_t* out_tok, int32_t* out_par, float* out_score) {
    __shared__ unsigned long long s_key[kTreeMaxNodes];
    __shared__ int s_before[kTreeMaxNodes];           // kept nodes created before node i; bit 30 set when node i itself is kept
    const int tid = threadIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    for (int i = tid; i < total; i += blockDim.x) s_key[i] = argmax_key(t.node_score[i], i);
    __syncthreads();
    for (int i = tid; i < total; i += blockDim.x) {
        const unsigned long long mine = s_key[i];
        int rank = 0;
        for (int j = 0; j < total; ++j) rank += s_key[j] > mine;
        s_before[i] = rank < n ? (1 << 30) : 0;
    }
    __syncthreads();
    int before_me[(kTreeMaxNodes + 1023) / 1024];
    for (int i = tid, e = 0; i < total; i += blockDim.x, ++e) {
        int c = 0;
        for (int j = 0; j < i; ++j) c += s_before[j] >> 30;
        before_me[e] = c;
    }
    __syncthreads();
    for (int i = tid, e = 0; i < total; i += blockDim.x, ++e) s_before[i] |= before_me[e];
    __syncthreads();
    for (int i = tid; i < total; i += blockDim.x) {
        if (!(s_before[i] >> 30)) continue;
        const int at = s_before[i] & ((1 << 30) - 1);
        const int par = t.node_par[i];
        out_tok[at] = t.node_tok[i];
        out_par[at] = (par >= 0 && (s_before[par] >> 30)) ? (s_before[par] & ((1 << 30) - 1)) : -1;
        out_score[at] = t.node_score[i];
    }
}

// One warp per (row, query head): the partial (m, l, unnormalised o) over the row's `nanc` ancestor states,
// written as split-KV chunk `chunk_idx` of that head.  Cache rows of the ancestors: n_true + anc[row][a].
template <int DPL>
__global__ void __launch_bounds__(32) attn_tail_kernel(const bf16* q, const bf16* kcache, const bf16* vcache, const int32_t* anc, int nanc, int slot,
                                                      int n_true, int Hq, int Hkv, int cap, int nch_stride, int chunk_idx, float scale, float* part_o,
                                                      float* part_ml) {
    constexpr int DH = DPL * 32;
    const int h = blockIdx.x, row = blockIdx.y, lane = threadIdx.x;
    pdl_launch_dependents();
    pdl_wait();                                       // the queries, the ancestors' cache rows and the ancestor lists come from kernels before
    const int kvh = h / (Hq / Hkv);
    float qf[DPL];
#pragma unroll
    for (int v = 0; v < DPL; ++v) qf[v] = __bfloat162float(q[((size_t)row * Hq + h) * DH + lane * DPL + v]) * scale;
    float sc[kTreeMaxDepth + 1];
    float m = -INFINITY;
    for (int a = 0; a < nanc; ++a)
        if (!BEAGLE_IN_BOUNDS(anc[row * (kTreeMaxDepth + 1) + a] >= 0 && n_true + anc[row * (kTreeMaxDepth + 1) + a] < cap && BEAGLE_SLOT_OK(slot))) nanc = 0;
    for (int a = 0; a < nanc; ++a) {
        const size_t at = (((size_t)slot * Hkv + kvh) * cap + n_true + anc[row * (kTreeMaxDepth + 1) + a]) * DH + lane * DPL;
        float dot = 0.f;
#pragma unroll
        for (int v = 0; v < DPL; ++v) dot = fmaf(qf[v], __bfloat162float(kcache[at + v]), dot);
        dot = warp_sum(dot);
        sc[a] = dot;
        m = fmaxf(m, dot);
    }
    float l = 0.f, acc[DPL];
#pragma unroll
    for (int v = 0; v < DPL; ++v) acc[v] = 0.f;
    for (int a = 0; a < nanc; ++a) {
        const size_t at = (((size_t)slot * Hkv + kvh) * cap + n_true + anc[row * (kTreeMaxDepth + 1) + a]) * DH + lane * DPL;
        const float p = __expf(sc[a] - m);
        l += p;
#pragma unroll
        for (int v = 0; v < DPL; ++v) acc[v] = fmaf(p, __bfloat162float(vcache[at + v]), acc[v]);
    }
    const size_t pi = ((size_t)row * Hq + h) * nch_stride + chunk_idx;
#pragma unroll
    for (int v = 0; v < DPL; ++v) part_o[pi * DH + lane * DPL + v] = acc[v];
    if (lane == 0) { part_ml[2 * pi] = m; part_ml[2 * pi + 1] = l; }
}

__global__ void tree_verify_kernel(const int32_t* __restrict__ tok, const int32_t* __restrict__ par, int n, const int32_t* __restrict__ target_ids,
                                   int out_cap, int32_t* __restrict__ accept_len, int32_t* __restrict__ out_tokens, int32_t* __restrict__ path) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int cur = -1, want = target_ids[0], a = 0;
    for (int i = 0; i < out_cap; ++i) { out_tokens[i] = -1; if (path != nullptr) path[i] = -1; }
    while (a + 1 < out_cap) {
        int nxt = -1;
        for (int j = 0; j < n && nxt < 0; ++j)
            if (par[j] == cur && tok[j] == want) nxt = j;
        if (nxt < 0) break;
        out_tokens[a] = want;
        if (path != nullptr) path[a] = nxt;
        cur = nxt;
        want = target_ids[1 + cur];
        ++a;
    }
    out_tokens[a] = want;
    *accept_len = a;
}

}  // namespace

int topk_splits(int V);

size_t tree_arrays_bytes(int vocab) {
    const size_t nodes = kTreeMaxNodes;
    const size_t splits = (size_t)topk_splits(vocab) * kTreeMaxTopk;
    return splits * (sizeof(float2) + kTreeMaxTopk * sizeof(unsigned long long)) + 2 * 256 + nodes * (2 * sizeof(int32_t) + sizeof(float)) +
           (size_t)kTreeMaxTopk * (2 + kTreeMaxDepth + 1) * sizeof(int32_t) + 8 * 256;
}

TreeArrays tree_arrays_carve(void* mem, int vocab) {
    TreeArrays t;
    char* p = static_cast<char*>(mem);
    auto take = [&](size_t bytes) { char* at = p; p += (bytes + 255) / 256 * 256; return at; };
    t.node_tok = reinterpret_cast<int32_t*>(take(kTreeMaxNodes * sizeof(int32_t)));
    t.node_par = reinterpret_cast<int32_t*>(take(kTreeMaxNodes * sizeof(int32_t)));
    t.node_score = reinterpret_cast<float*>(take(kTreeMaxNodes * sizeof(float)));
    t.frontier_node = reinterpret_cast<int32_t*>(take(kTreeMaxTopk * sizeof(int32_t)));
    t.frontier_tok = reinterpret_cast<int32_t*>(take(kTreeMaxTopk * sizeof(int32_t)));
    t.frontier_anc = reinterpret_cast<int32_t*>(take((size_t)kTreeMaxTopk * (kTreeMaxDepth + 1) * sizeof(int32_t)));
    const size_t splits = (size_t)topk_splits(vocab) * kTreeMaxTopk;
    t.topk_lse = reinterpret_cast<float2*>(take(splits * sizeof(float2)));
    t.topk_keys = reinterpret_cast<unsigned long long*>(take(splits * kTreeMaxTopk * sizeof(unsigned long long)));
    return t;
}

int topk_splits(int V) { return (V + kTopkSplitElems - 1) / kTopkSplitElems; }

int launch_topk_logprob(const float* logits, int rows, int V, int k, const TreeArrays& t, cudaStream_t stream) {
    const int nsplit = topk_splits(V);
    const int per = (V + nsplit - 1) / nsplit;
    launch_pdl(topk_partial_kernel, dim3(nsplit, rows), dim3(256), 0, stream, logits, V, k, per, t.topk_lse, t.topk_keys);
    return 1;
}
int launch_tree_expand(const TreeArrays& t, int V, int k, int rows, int level, int base, cudaStream_t stream) {
    launch_pdl(tree_expand_kernel, dim3(1), dim3(32 * kTreeMaxTopk), 0, stream, t, topk_splits(V), k, rows, level, base);
    return 1;
}
int launch_tree_rerank(const TreeArrays& t, int total, int n, int32_t* out_tok, int32_t* out_par, float* out_score, cudaStream_t stream) {
    launch_pdl(tree_rerank_kernel, dim3(1), dim3(1024), 0, stream, t, total, n, out_tok, out_par, out_score);
    return 1;
}
int launch_attn_tail(const void* q, const void* kcache, const void* vcache, const int32_t* anc, int nanc, int rows, int slot, int n_true, int Hq,
                     int Hkv, int dh, int cap, int nch_stride, int chunk_idx, float* part_o, float* part_ml, cudaStream_t stream) {
    const float scale = 1.0f / sqrtf((float)dh);
    dim3 grid(Hq, rows);
#define BEAGLE_TAIL(DPL) launch_pdl(attn_tail_kernel<DPL>, grid, dim3(32), 0, stream, (const bf16*)q, (const bf16*)kcache, (const bf16*)vcache, anc, nanc, slot, \
                                    n_true, Hq, Hkv, cap, nch_stride, chunk_idx, scale, part_o, part_ml)
    switch (dh) {
        case 64: BEAGLE_TAIL(2); break;
        case 128: BEAGLE_TAIL(4); break;
        default: return -1;
    }
#undef BEAGLE_TAIL
    return 1;
}
int launch_tree_verify(const int32_t* tok, const int32_t* par, int n, const int32_t* target_ids, int out_cap, int32_t* accept_len,
                       int32_t* out_tokens, int32_t* path, cudaStream_t stream) {
    tree_verify_kernel<<<1, 32, 0, stream>>>(tok, par, n, target_ids, out_cap, accept_len, out_tokens, path);
    return 1;
}

}  // namespace beagle
