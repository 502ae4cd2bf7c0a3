// Host-side launchers of the Beagle draft-head kernels.  Every function only enqueues kernels on
// `stream` and returns the number of kernels it launched (negative: unsupported shape).
#pragma once
#include "common.cuh"

namespace beagle {

enum GemvMode {
    GEMV_STORE = 0,     // out[b][n] = W[n,:] . x_b
    GEMV_RESID = 1,     // out[b][n] = W[n,:] . x_b + resid[b][n]      (+ optional second copy out2[orow2[b]][n])
    GEMV_SILU_MUL = 2,  // out[b][n] = SiLU(W[n,:] . x_b) * (W2[n,:] . x_b)
    GEMV_LOGITS = 3,    // logits[b][n] (fp32, optional) and per-block arg-max keys
    GEMV_KV = 4         // blockIdx.y = 0: W -> key cache, 1: W2 -> value cache, at (slot[b], head, pos[b])
};

struct GemvArgs {
    const void* W;
    const void* W2;
    int N, K;
    const void* X;      // activations, storage type, row b at X + xrow.idx[b] * ldx
    int ldx;
    int B;
    void* out;          // [B, ldo]
    int ldo;
    const void* resid;  // [B, ldr]
    int ldr;
    void* out2;         // optional [*, ld2], row orow2.idx[b]
    int ld2;
    float* logits;      // optional fp32 [B, N]
    unsigned long long* partials;   // [B, gridDim.x]
    void* kcache;
    void* vcache;
    int Hkv, dh, cap;   // cache geometry [slot][Hkv][cap][dh]
    RowMap xrow;
    RowMap orow2;       // GEMV_RESID: rows of out2; GEMV_KV: cache slot
    RowMap pos;         // GEMV_KV: position in the slot
};

int gemv_grid_blocks(int mode, int N);   // gridDim.x the launcher uses (size of the partials row)
int launch_gemv(int dtype, int mode, const GemvArgs& a, cudaStream_t stream);

// x = E[token] (or rows of src), xn = RMSNorm(x) * g (or x when do_norm == 0).
// tokens == NULL: row b uses last_token[meta.slot[b]].  src != NULL: no gather, rows of src.
// gather_src != NULL: row b of gather_dst additionally receives row meta.slot[b] of gather_src.
int launch_embed_norm(int dtype, const int32_t* tokens, const int32_t* last_token, const BatchMeta* meta,
                      const void* embed, int vocab, const void* src, const void* gain, int d, float eps, int do_norm,
                      void* x_out, void* xn_out, int rows, const void* gather_src, void* gather_dst, cudaStream_t stream);

// Split-KV cross-attention decode over the cache + combine.  q, o: [B, Hq*dh] storage type.
size_t attn_decode_scratch_bytes(int max_batch, int Hq, int dh, int max_kv);
int launch_attn_decode(int dtype, const void* q, const void* kcache, const void* vcache, const BatchMeta& meta,
                       int B, int Hq, int Hkv, int dh, int cap, int max_kv_len, void* scratch, void* o,
                       cudaStream_t stream);

// Merges the split-KV partials (unnormalised o, running max, exp-sum per chunk of `chunk` keys).
// extra_chunks: partials stored right after a row's regular chunks (the tree's ancestor states) to merge as well.
int launch_attn_combine(int dtype, const float* part_o, const float* part_ml, const BatchMeta& meta, int B, int Hq, int dh,
                        int nchunk_stride, int chunk, void* o, cudaStream_t stream, int extra_chunks = 0);

// tokens_out[b] (optional) and last_token[slot[b]] from the per-block keys.
int launch_argmax_finalize(const unsigned long long* partials, int nblk, const BatchMeta& meta, int B,
                           int32_t* tokens_out, int tokens_out_stride, int32_t* last_token, cudaStream_t stream);

// Row arg-max of [rows, V] logits (fp32 or bf16) into int32 ids; scratch: rows * kRowArgmaxSplit keys.
constexpr int kRowArgmaxSplit = 16;
int launch_row_argmax(int logits_dtype, const void* logits, int rows, int V, unsigned long long* scratch,
                      int32_t* ids_out, cudaStream_t stream);
// Greedy verification from target logits [B, gamma+1, V] (fp32 or bf16) in one launch: arg-max partial keys per (row, slice)
// and the acceptance walk by the CTA that finishes a sequence last.  keys: B * (gamma+1) * kVerifyMaxSplit entries (any
// contents); tickets: B ints, zero before the first launch (the kernel leaves them zero).
constexpr int kVerifyMaxSplit = 64;
int launch_verify_greedy_fused(int logits_dtype, const void* logits, int B, int gamma, int V, const int32_t* draft,
                               unsigned long long* keys, int* tickets, int sm_count, int32_t* accept_len, int32_t* out_tokens,
                               cudaStream_t stream);
// Greedy acceptance from target ids.
int launch_accept(const int32_t* draft, const int32_t* target_ids, int B, int gamma, int32_t* accept_len,
                  int32_t* out_tokens, cudaStream_t stream);

// Acceptance under sampling (Section 3): min(1, p/q) tests with the uniforms u_accept [B, gamma], then one
// token by inverse CDF (u_resample [B]) from the normalised max(0, p_j - q_j).  draft_logits fp32
// [gamma, B, V]; target_logits [B, gamma+1, V] fp32 or bf16.
size_t verify_sample_scratch_bytes(int max_batch, int max_gamma);
int launch_verify_sample(int logits_dtype, const int32_t* draft, const float* draft_logits, const void* target_logits, int B, int gamma, int V,
                         float temperature, const float* u_accept, const float* u_resample, void* scratch, int* tickets, int32_t* accept_len,
                         int32_t* out_tokens, int sm_count, cudaStream_t stream);

// ---- dynamic-tree drafting: device-side bookkeeping -------------------------------------------
constexpr int kTreeMaxTopk = 16, kTreeMaxDepth = 8, kTreeMaxCandidates = 64;
constexpr int kTreeMaxNodes = kTreeMaxTopk + kTreeMaxDepth * kTreeMaxTopk * kTreeMaxTopk;
struct TreeArrays {
    int32_t* node_tok; int32_t* node_par; float* node_score;       // every node created, in creation order
    int32_t* frontier_node; int32_t* frontier_tok;                 // [k] nodes to forward next and their tokens
    int32_t* frontier_anc;                                         // [k][kTreeMaxDepth + 1] tail positions of their ancestors' states
    float2* topk_lse; unsigned long long* topk_keys;               // per (row, vocabulary slice): (max, exp-sum) and the slice's k best keys
};
size_t tree_arrays_bytes(int vocab);
TreeArrays tree_arrays_carve(void* mem, int vocab);
int launch_topk_logprob(const float* logits, int rows, int V, int k, const TreeArrays& t, cudaStream_t stream);
int launch_tree_expand(const TreeArrays& t, int V, int k, int rows, int level, int base, cudaStream_t stream);
int launch_tree_rerank(const TreeArrays& t, int total, int n, int32_t* out_tok, int32_t* out_par, float* out_score, cudaStream_t stream);
// Attention partial over each row's ancestor draft states, stored as split-KV chunk `chunk_idx` (bf16, dh 64 / 128).
int launch_attn_tail(const void* q, const void* kcache, const void* vcache, const int32_t* anc, int nanc, int rows, int slot, int n_true, int Hq,
                     int Hkv, int dh, int cap, int nch_stride, int chunk_idx, float* part_o, float* part_ml, cudaStream_t stream);
// Greedy walk: target_ids[0] is the target's token at the root, target_ids[1 + n] after node n.
int launch_tree_verify(const int32_t* tok, const int32_t* par, int n, const int32_t* target_ids, int out_cap, int32_t* accept_len,
                       int32_t* out_tokens, int32_t* path, cudaStream_t stream);

// ---- optional FP8 LM head: q[r, :] = e4m3(x[r, :] / scale[r]), scale[r] = max|x[r, :]| / 448; cols a multiple of 8 ----
int launch_quantize_rows_e4m3(int dtype, const void* x, long long rows, int cols, void* q, float* scale, cudaStream_t stream);

// ---- optional rotary position embedding (rotate-half; table of (cos, sin) per (position, i < dh/2)) ----
int launch_rope_table(float theta, int dh, int npos, float* table, cudaStream_t stream);
// Rows of a dense [rows, H*dh] matrix in place; row r sits at position pos_base + r % S; inverse: opposite angle.
int launch_rope_rows(int dtype, void* x, long long rows, int H, int dh, int S, int pos_base, int inverse, const float* table,
                     cudaStream_t stream);
// One draft step: query rows b < nq at positions qpos[b]; the key rows appended for b < nk at cache row app[b] (< 0: none), position kpos[b].
int launch_rope_serve(int dtype, void* q, int nq, int Hq, void* kcache, int nk, int Hkv, int dh, int cap, const RowMap& slot, const RowMap& app,
                      const RowMap& qpos, const RowMap& kpos, const float* table, cudaStream_t stream);

// ---- block path ------------------------------------------------------------------------------
enum GemmEpilogue {
    GEMM_STORE = 0,      // C = A W^T                     (storage type)
    GEMM_RESID = 1,      // C = A W^T + R
    GEMM_SILU_MUL = 2,   // C = SiLU(A W^T) * (A W2^T)
    GEMM_F32 = 3,        // C fp32
    GEMM_KV_CACHE = 4,   // scatter rows into the cache: row r -> (slot, pos) through SeqRows
    GEMM_ARGMAX_KEYS = 5,// no C: one packed arg-max key per (row, column tile)   (tensor-core path only)
    GEMM_CE = 6,         // no C: cross-entropy partials per (row, column tile)       (tensor-core path only)
    GEMM_DLOGITS = 7,    // C = row_coef * (softmax(A W^T) - p), storage type, from the rows' softmax statistics (tensor-core path only)
    GEMM_KV_CACHE_PAIR = 8  // A W^T -> `cache` and A W2^T -> `cache2` in ONE pass over A, rows scattered as GEMM_KV_CACHE (tensor-core path only)
};
// Cross-entropy partial of one (row, column range): running max / exp-sum of the draft logits z,
// running max / exp-sum of the target logits t and sum exp(t - tmax) * z (soft targets); with hard
// labels tmax = 0, tsum = 1 if the label lies in the range (else 0) and dot = z[label] (else 0).
constexpr int kCeFields = 5;
struct SeqRows {        // packed-row -> (slot, position) map of a prefill call
    int32_t n;
    int32_t slot[kMaxCallBatch];
    int32_t row_start[kMaxCallBatch + 1];
    int32_t pos_start[kMaxCallBatch];
};
struct GemmArgs {
    const void* A; int lda;       // [M, K]
    const void* W; const void* W2;  // [N, K]
    int M, N, K;
    void* C; int ldc;
    const void* R; int ldr;
    void* cache; int Hkv, dh, cap;  // GEMM_KV_CACHE
    void* cache2;                   // GEMM_KV_CACHE_PAIR: the second matrix's cache
    unsigned long long* keys;       // GEMM_ARGMAX_KEYS
    const void* tgt; int tgt_dtype; int ldt;   // GEMM_CE, soft targets: target logits [M, ldt] (0 fp32, 1 bf16)
    const int32_t* labels;          // GEMM_CE, hard targets: [M] (used when tgt == NULL)
    float* ce_part;                 // GEMM_CE: [M][column tiles][kCeFields]
    const float* row_stats;         // GEMM_DLOGITS: [M][4] = max z, exp-sum z, max t, exp-sum t of every row
    const float* row_coef;          // GEMM_DLOGITS: [M] loss weight of the row times the loss scale
    int* error_word;                // device word set to 1 when a bounded wait ran out
    int w_transient;                // W is a workspace buffer (its tensor map is not cached by pointer)
    // Transposed operands (tensor-core path only, GEMM_STORE / GEMM_RESID / GEMM_F32): a_mn: A is given as [K, M] row-major
    // (row stride lda), i.e. the product is A^T W^T; b_mn: W is given as [K, N] row-major (row stride ldw).
    int a_mn, b_mn, ldw;
    SeqRows rows;
};
int launch_gemm_simt(int dtype, int epi, const GemmArgs& a, cudaStream_t stream);
// Key rows a prefill appended (cache row = position), rotated in place.
int launch_rope_cache_rows(int dtype, void* kcache, long long total_rows, int Hkv, int dh, int cap, const SeqRows& rows, const float* table,
                           cudaStream_t stream);

// ---- block-path losses (Eq. 4 / Eq. 7, forward) -------------------------------------------------
// Cross-entropy partials (one column range = the whole row) from materialised fp32 draft logits.
int launch_row_ce(const float* logits, int rows, int V, const void* tgt, int tgt_dtype, const int32_t* labels, float* ce_part,
                  cudaStream_t stream);
// ce[row] from the partials of `ntiles` column ranges, wce[row] = weight(position) * ce[row], then
// loss = sum(wce) / (batch * windows), summed in a fixed order.  stage: 0 early, 1 late.
// row_stats (optional, 4 floats per row): the row's merged max / exp-sum of z and of the target logits.
int launch_ce_finalize(const float* ce_part, int ntiles, int batch, int S, int block, int offset, int sim_steps, int stage,
                       float* ce_rows, float* wce, float* ce_out, float* loss_out, cudaStream_t stream, float* row_stats = nullptr);

// ---- block-path training step: backward (Eq. 4 / Eq. 7 and the state regression of Appendix B) ----
// out[c][col0 + r] = in[r][c]; columns col0 + rows .. col0 + rows_pad - 1 of every output row are zeroed.
int launch_transpose_pad(int dtype, const void* in, int rows, int cols, int ld_in, void* out, int ld_out, int col0, int rows_pad,
                         cudaStream_t stream);
// The same for `nbatch` matrices: matrix z starts at in + z * in_batch_stride and lands at column col0 + z * col_batch_stride.
int launch_transpose_pad_batched(int dtype, const void* in, int rows, int cols, int ld_in, size_t in_batch_stride, void* out, int ld_out, int col0,
                                 int col_batch_stride, int rows_pad, int nbatch, cudaStream_t stream);
int launch_silu_mul(int dtype, const void* gate, const void* up, void* act, size_t n, cudaStream_t stream);
// In place: gate <- d gate, up <- d up.
int launch_silu_mul_bwd(int dtype, void* gate, void* up, const void* dact, size_t n, cudaStream_t stream);
// d z [row0 .. row0 + rows) = weight(position) * scale * (softmax(z) - p) from a chunk of fp32 logits; columns V..ldz-1 zeroed.
int launch_dlogits(int dtype, const float* logits, int rows, int V, const void* tgt, int tgt_dtype, const int32_t* labels, const float* stats,
                   int row0, int S, int block, int offset, int sim_steps, int stage, float scale, void* dz, int ldz, cudaStream_t stream);
// dh0 = grad_coef * reg * clip(h - h_true, -1, 1); loss3[1] = vscale * sum smooth_l1, loss3[2] = loss3[0] + vcoef * loss3[1].
// coef[row] = loss weight of the row's position (Eq. 4 / Eq. 7) * scale.
int launch_loss_coef(int rows, int S, int block, int offset, int sim_steps, int stage, float scale, float* coef, cudaStream_t stream);
int launch_vloss(int dtype, const void* h, const void* h_true, int rows, int d, int S, int block, int offset, int sim_steps, int stage,
                 float grad_coef, float vscale, float vcoef, void* dh0, float* row_sum, float* loss3, cudaStream_t stream);
int rmsnorm_bwd_parts(int rows);     // rows of the dg_part scratch ([parts][d] fp32)
// out = add + d v of n = RMSNorm(v; gain) given d n (do_norm == 0: out = add + dn); dg_out (optional) = d gain.
int launch_rmsnorm_bwd(int dtype, const void* v, const void* gain, const void* dn, const void* add, int rows, int d, float eps, int do_norm,
                       void* out, float* dg_part, float* dg_out, cudaStream_t stream);
int launch_embed_grad(int dtype, const int32_t* tokens, const void* dx, int rows, int d, float* dembed, cudaStream_t stream);
// Attention backward of the block-masked cross-attention (same visibility rule as launch_attn_block).
// lse, delta: fp32 [B*S, Hq] scratch.  dKp / dVp are written only when step > 1.
int launch_attn_block_bwd(int dtype, const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp, const void* dO, int B, int S,
                          int Hq, int Hkv, int dh, int block, int offset, int step, void* dQ, void* dKt, void* dVt, void* dKp, void* dVp,
                          float* lse, float* delta, cudaStream_t stream);

// Block-masked cross-attention: query row (b, p) reads true keys [0, n(p)) of Kt/Vt and, when
// step > 1, predicted keys n(p) .. n(p)+min(slot, step)-2 of Kp/Vp.  All [B*S, H*dh] row-major.
int launch_attn_block(int dtype, const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp,
                      int B, int S, int Hq, int Hkv, int dh, int block, int offset, int step, void* O,
                      cudaStream_t stream);

}  // namespace beagle
