// Device-side bookkeeping of dynamic-tree drafting (the dynamic draft attention tree the paper's
// experiments adopt: top-k expansion scored by cumulative log-probability, top-N rerank) and greedy
// acceptance along tree paths.  Everything stays on the device, so a whole tree is drafted without a
// host synchronisation: the forwards of the frontier nodes are the ordinary serve-time kernels, fed
// from the arrays these kernels maintain.
//
//   topk_partial / topk_merge   per forwarded row: log-sum-exp of its logits and its k best children
//   tree_expand_kernel    appends the k*k children, picks the next frontier, builds its ancestor lists
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

constexpr int kTopkSplitElems = 4096;        // logits per CTA of the first pass (16 KB of shared memory)

// Pass 1, grid (splits, rows): the CTA keeps its slice of the row in shared memory, computes the slice's
// (max, exp-sum) and its k best keys (the j-th best is the largest key below the (j-1)-th: no masking).
__global__ void __launch_bounds__(256) topk_partial_kernel(const float* __restrict__ logits, int V, int k, int per, float2* __restrict__ lse_part,
                                                          unsigned long long* __restrict__ key_part) {
    extern __shared__ float s_z[];
    __shared__ unsigned long long s_k[8];
    __shared__ float s_f[8];
    const int split = blockIdx.x, row = blockIdx.y, nsplit = gridDim.x;
    const int lo = split * per, hi = min(V, lo + per), n = max(0, hi - lo);
    const float* z = logits + (size_t)row * V + lo;
    float m = -INFINITY;
    for (int i = threadIdx.x; i < n; i += blockDim.x) { const float v = z[i]; s_z[i] = v; m = fmaxf(m, v); }
    m = warp_max(m);
    if ((threadIdx.x & 31) == 0) s_f[threadIdx.x >> 5] = m;
    __syncthreads();
    m = s_f[0];
    for (int w = 1; w < 8; ++w) m = fmaxf(m, s_f[w]);
    __syncthreads();
    float s = 0.f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) s += __expf(s_z[i] - m);
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) s_f[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += s_f[w];
        lse_part[(size_t)row * nsplit + split] = make_float2(m, t);
    }
    unsigned long long prev = ~0ull;
    for (int j = 0; j < k; ++j) {
        unsigned long long best = 0ull;
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const unsigned long long key = argmax_key(s_z[i], lo + i);
            if (key < prev && key > best) best = key;
        }
        best = block_max_u64(best, s_k);
        if (threadIdx.x == 0) key_part[((size_t)row * nsplit + split) * k + j] = best;
        prev = best;
    }
}

// Pass 2, one CTA per row: log-sum-exp of the row and the k best of the splits' candidates.
__global__ void __launch_bounds__(256) topk_merge_kernel(const float2* __restrict__ lse_part, const unsigned long long* __restrict__ key_part,
                                                        int nsplit, int k, int32_t* __restrict__ child_tok, float* __restrict__ child_lq) {
    __shared__ unsigned long long s_k[8];
    __shared__ float s_lse;
    const int row = blockIdx.x;
    if (threadIdx.x == 0) {
        float M = -INFINITY;
        for (int i = 0; i < nsplit; ++i) M = fmaxf(M, lse_part[(size_t)row * nsplit + i].x);
        float S = 0.f;
        for (int i = 0; i < nsplit; ++i) {
            const float2 p = lse_part[(size_t)row * nsplit + i];
            S += (p.x == -INFINITY) ? 0.f : p.y * __expf(p.x - M);
        }
        s_lse = M + __logf(S);
    }
    const unsigned long long* cand = key_part + (size_t)row * nsplit * k;
    const int ncand = nsplit * k;
    unsigned long long prev = ~0ull;
    for (int j = 0; j < k; ++j) {
        unsigned long long best = 0ull;
        for (int i = threadIdx.x; i < ncand; i += blockDim.x) {
            const unsigned long long key = cand[i];
            if (key < prev && key > best) best = key;
        }
        best = block_max_u64(best, s_k);                    // (contains the barrier that also publishes s_lse)
        if (threadIdx.x == 0) {
            child_tok[(size_t)row * k + j] = best != 0ull ? argmax_key_index(best) : 0;
            child_lq[(size_t)row * k + j] = best != 0ull ? key_value(best) - s_lse : -INFINITY;
        }
        prev = best;
    }
}

// level = 0: the root's children become nodes 0..k-1 and the first frontier (ancestor list = the root's state,
// tail position 0).  level = e >= 1: the rows of forward e were the frontier; their k*k children are appended
// at `base`, the k best (score, then creation order) become the next frontier, whose ancestor lists are the
// parent's list plus the parent's own state (tail position 1 + (e-1)*k + parent row).
__global__ void __launch_bounds__(256) tree_expand_kernel(TreeArrays t, int k, int level, int base) {
    __shared__ unsigned long long s_k[8];
    __shared__ int s_sel[kTreeMaxTopk];
    __shared__ int s_anc[kTreeMaxTopk][kTreeMaxDepth + 1];
    __shared__ int s_node[kTreeMaxTopk];
    const int tid = threadIdx.x;
    if (level == 0) {
        if (tid < k) {
            t.node_tok[tid] = t.child_tok[tid];
            t.node_par[tid] = -1;
            t.node_score[tid] = t.child_lq[tid];
            t.frontier_node[tid] = tid;
            t.frontier_tok[tid] = t.child_tok[tid];
            t.frontier_anc[tid * (kTreeMaxDepth + 1)] = 0;
        }
        return;
    }
    const int nnew = k * k;
    for (int i = tid; i < nnew; i += blockDim.x) {
        const int r = i / k;
        const int f = t.frontier_node[r];
        t.node_tok[base + i] = t.child_tok[i];
        t.node_par[base + i] = f;
        t.node_score[base + i] = t.node_score[f] + t.child_lq[i];
    }
    if (tid < k) {
        s_node[tid] = t.frontier_node[tid];
        for (int a = 0; a < level; ++a) s_anc[tid][a] = t.frontier_anc[tid * (kTreeMaxDepth + 1) + a];
    }
    __syncthreads();
    unsigned long long prev = ~0ull;
    for (int j = 0; j < k; ++j) {
        unsigned long long best = 0ull;
        for (int i = tid; i < nnew; i += blockDim.x) {
            const unsigned long long key = argmax_key(t.node_score[base + i], i);
            if (key < prev && key > best) best = key;
        }
        best = block_max_u64(best, s_k);
        if (tid == 0) s_sel[j] = argmax_key_index(best);
        prev = best;
    }
    __syncthreads();
    if (tid < k) {
        const int i = s_sel[tid], r = i / k;
        t.frontier_node[tid] = base + i;
        t.frontier_tok[tid] = t.node_tok[base + i];
        for (int a = 0; a < level; ++a) t.frontier_anc[tid * (kTreeMaxDepth + 1) + a] = s_anc[r][a];
        t.frontier_anc[tid * (kTreeMaxDepth + 1) + level] = 1 + (level - 1) * k + r;
    }
}

__global__ void __launch_bounds__(1024) tree_rerank_kernel(TreeArrays t, int total, int n, int32_t* __restrict__ out_tok,
                                                          int32_t* __restrict__ out_par, float* __restrict__ out_score) {
    __shared__ unsigned long long s_k[32];
    __shared__ int s_sel[kTreeMaxCandidates], s_sorted[kTreeMaxCandidates];
    const int tid = threadIdx.x;
    unsigned long long prev = ~0ull;
    for (int j = 0; j < n; ++j) {
        unsigned long long best = 0ull;
        for (int i = tid; i < total; i += blockDim.x) {
            const unsigned long long key = argmax_key(t.node_score[i], i);
            if (key < prev && key > best) best = key;
        }
        best = block_max_u64(best, s_k);
        if (tid == 0) s_sel[j] = argmax_key_index(best);
        prev = best;
    }
    __syncthreads();
    if (tid < n) {                                  // creation order: rank by node id
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += s_sel[j] < s_sel[tid];
        s_sorted[rank] = s_sel[tid];
    }
    __syncthreads();
    if (tid < n) {
        const int node = s_sorted[tid];
        const int par = t.node_par[node];
        int pi = -1;
        if (par >= 0)
            for (int j = 0; j < n; ++j) if (s_sorted[j] == par) pi = j;
        out_tok[tid] = t.node_tok[node];
        out_par[tid] = pi;
        out_score[tid] = t.node_score[node];
    }
}

// One warp per (row, query head): the partial (m, l, unnormalised o) over the row's `nanc` ancestor states,
// written as split-KV chunk `chunk_idx` of that head.  Cache rows of the ancestors: n_true + anc[row][a].
template <int DPL>
__global__ void __launch_bounds__(32) attn_tail_kernel(const bf16* __restrict__ q, const bf16* __restrict__ kcache, const bf16* __restrict__ vcache,
                                                      const int32_t* __restrict__ anc, int nanc, int slot, int n_true, int Hq, int Hkv, int cap,
                                                      int nch_stride, int chunk_idx, float scale, float* __restrict__ part_o,
                                                      float* __restrict__ part_ml) {
    constexpr int DH = DPL * 32;
    const int h = blockIdx.x, row = blockIdx.y, lane = threadIdx.x;
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
    return splits * (sizeof(float2) + kTreeMaxTopk * sizeof(unsigned long long)) + 2 * 256 + nodes * (2 * sizeof(int32_t) + sizeof(float)) + (size_t)kTreeMaxTopk * kTreeMaxTopk * (sizeof(int32_t) + sizeof(float)) +
           (size_t)kTreeMaxTopk * (2 + kTreeMaxDepth + 1) * sizeof(int32_t) + 8 * 256;
}

TreeArrays tree_arrays_carve(void* mem, int vocab) {
    TreeArrays t;
    char* p = static_cast<char*>(mem);
    auto take = [&](size_t bytes) { char* at = p; p += (bytes + 255) / 256 * 256; return at; };
    t.node_tok = reinterpret_cast<int32_t*>(take(kTreeMaxNodes * sizeof(int32_t)));
    t.node_par = reinterpret_cast<int32_t*>(take(kTreeMaxNodes * sizeof(int32_t)));
    t.node_score = reinterpret_cast<float*>(take(kTreeMaxNodes * sizeof(float)));
    t.child_tok = reinterpret_cast<int32_t*>(take((size_t)kTreeMaxTopk * kTreeMaxTopk * sizeof(int32_t)));
    t.child_lq = reinterpret_cast<float*>(take((size_t)kTreeMaxTopk * kTreeMaxTopk * sizeof(float)));
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
    topk_partial_kernel<<<dim3(nsplit, rows), 256, (size_t)per * sizeof(float), stream>>>(logits, V, k, per, t.topk_lse, t.topk_keys);
    topk_merge_kernel<<<rows, 256, 0, stream>>>(t.topk_lse, t.topk_keys, nsplit, k, t.child_tok, t.child_lq);
    return 2;
}
int launch_tree_expand(const TreeArrays& t, int k, int level, int base, cudaStream_t stream) {
    tree_expand_kernel<<<1, 256, 0, stream>>>(t, k, level, base);
    return 1;
}
int launch_tree_rerank(const TreeArrays& t, int total, int n, int32_t* out_tok, int32_t* out_par, float* out_score, cudaStream_t stream) {
    tree_rerank_kernel<<<1, 1024, 0, stream>>>(t, total, n, out_tok, out_par, out_score);
    return 1;
}
int launch_attn_tail(const void* q, const void* kcache, const void* vcache, const int32_t* anc, int nanc, int rows, int slot, int n_true, int Hq,
                     int Hkv, int dh, int cap, int nch_stride, int chunk_idx, float* part_o, float* part_ml, cudaStream_t stream) {
    const float scale = 1.0f / sqrtf((float)dh);
    dim3 grid(Hq, rows);
#define BEAGLE_TAIL(DPL) attn_tail_kernel<DPL><<<grid, 32, 0, stream>>>((const bf16*)q, (const bf16*)kcache, (const bf16*)vcache, anc, nanc, slot, \
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
