/*
 * beagle.h -- C ABI of the B200 (sm_100a) forward pass of the Beagle cross-attention draft head.
 *
 * The head is one Transformer block whose queries come from token embeddings and whose keys and
 * values come from higher-level states: the target model's top hidden states ("true states") or
 * the head's own outputs (Section 4.1, Eq. 1 and Eq. 2 of the paper), followed by a linear LM head
 * and greedy draft/verify acceptance (Section 3).  For one query at position p reading the visible
 * state set Vis(p):
 *
 *     x  = E[t_p]                                   embedding
 *     Q  = W_q RMSNorm(x; g_q)                      per head h: rows [h*dh, (h+1)*dh)
 *     K_j, V_j = W_k s_j, W_v s_j                   s_j in Vis(p); head h reads K/V head h / (Hq/Hkv)
 *     o_h = sum_j softmax_j(<Q_h, K_j>/sqrt(dh)) V_j    (softmax over Vis(p) only; Vis empty: o = 0)
 *     y  = W_o [o_1 .. o_Hq] + x
 *     h  = y + W_down( SiLU(W_gate n) * (W_up n) ),  n = RMSNorm(y; g_mlp)
 *     z  = W_lm h,   t^ = argmax z  (lowest index on ties, NaN never wins)
 *
 * Conventions
 *   - Every pointer named "dev" is DEVICE memory owned by the caller; "host" is host memory.  The
 *     library allocates no device memory and creates no stream: the caller passes the key/value
 *     cache, a workspace (sizes from beagle_query_sizes / beagle_block_workspace_bytes) and a
 *     cudaStream_t (as void*; NULL = the legacy default stream).
 *   - dtype 0 = fp32, 1 = bf16 is the storage type of weights, states, cache and hidden outputs;
 *     accumulation, softmax and logits are fp32.  Weights are row-major [out, in].
 *   - Calls only enqueue work on the stream and return; they never synchronise -- with one exception:
 *     the FIRST call on a context that launches anything zeroes a few device words of the workspace
 *     (an error word, completion counters), builds the rotary table if that option is on, and waits
 *     for that once, so that later calls may use any stream.  That first call must be made outside
 *     stream capture (inside one it returns BEAGLE_ERR_STATE and launches nothing); from the second
 *     call on the entry points are capturable.  Argument, shape, capacity and state errors are
 *     detected on the host before anything is launched and leave the context unchanged.  No call
 *     aborts, throws or traps.
 *   - A context belongs to the device that was current when it was created, and every call on it
 *     must be made with that device current.  Several contexts, on one or on several devices, may
 *     live in one process.  A context is not thread-safe; use one per stream.
 */
#ifndef BEAGLE_H
#define BEAGLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct beagle_ctx beagle_ctx;

typedef enum beagle_status {
    BEAGLE_OK = 0,
    BEAGLE_ERR_INVALID_ARG = 1,   /* NULL pointer, negative size, unknown flag                     */
    BEAGLE_ERR_SHAPE = 2,         /* a dimension the kernels do not support (see beagle_config)   */
    BEAGLE_ERR_CAPACITY = 3,      /* cache, workspace, batch or draft depth exceeded              */
    BEAGLE_ERR_STATE = 4,         /* call order: e.g. tokens_in == NULL with no previous step     */
    BEAGLE_ERR_UNSUPPORTED = 5,
    BEAGLE_ERR_CUDA = 6,          /* a CUDA runtime call failed; see beagle_last_error            */
    BEAGLE_ERR_DEVICE = 7         /* a kernel gave up on one of its bounded waits (beagle_check_device) */
} beagle_status;

enum { BEAGLE_FP32 = 0, BEAGLE_BF16 = 1 };

/* Largest `batch` of one beagle_prefill_kv / beagle_draft_step / beagle_verify_greedy call. */
#define BEAGLE_MAX_CALL_BATCH 64

typedef struct beagle_config {
    int32_t hidden;       /* d; multiple of 8                                                      */
    int32_t n_q_heads;    /* Hq                                                                    */
    int32_t n_kv_heads;   /* Hkv; Hq % Hkv == 0, Hq/Hkv in {1,2,4,8}                                */
    int32_t head_dim;     /* dh; bf16: 32|64|128|256, fp32: 16|32|64|128                            */
    int32_t mlp_dim;      /* m; multiple of 8                                                      */
    int32_t vocab;        /* V                                                                     */
    int32_t dtype;        /* BEAGLE_FP32 | BEAGLE_BF16                                             */
    float   rms_eps;
    int32_t norm_q;       /* 1: RMSNorm(g_q) on the query input, 0: none                           */
    int32_t norm_mlp;     /* 1: RMSNorm(g_mlp) on the MLP input, 0: none                           */
    int32_t max_slots;    /* sequences the cache holds                                             */
    int32_t max_ctx;      /* true states per sequence                                              */
    int32_t max_draft;    /* draft states appended per sequence between two resets                 */
    float   rope_theta;   /* 0: no positional term (Eq. 2 as printed).  > 0: rotary position embedding with this base,
                             LLaMA "rotate half" convention: inside each head, components i and i + dh/2 of Q and K are
                             rotated by pos * theta^(-2i/dh), pos = position - 1 (0-based): the query of position p by
                             p - 1, the key made from the state at position j (true, draft or predicted) by j - 1.  Values
                             are not rotated.  In serve-time drafting a slot with n true states queries position
                             n + s at the s-th beagle_draft_step since its last prefill / rollback / reset.          */
} beagle_config;

/* Device pointers, row-major [out, in], BORROWED: they must outlive the context. */
typedef struct beagle_weights {
    const void* embed;    /* [V, d]            */
    const void* g_q;      /* [d]               */
    const void* w_q;      /* [Hq*dh, d]        */
    const void* w_k;      /* [Hkv*dh, d]       */
    const void* w_v;      /* [Hkv*dh, d]       */
    const void* w_o;      /* [d, Hq*dh]        */
    const void* g_mlp;    /* [d]               */
    const void* w_gate;   /* [m, d]            */
    const void* w_up;     /* [m, d]            */
    const void* w_down;   /* [d, m]            */
    const void* w_lm;     /* [V, d]            */
    /* Optional FP8 copy of the LM head (NULL, NULL = none; not part of the paper).  w_lm_fp8: [V, d] bytes, FP8 E4M3;
     * w_lm_scale: fp32 [V]; row v of w_lm ~ w_lm_scale[v] * w_lm_fp8[v, :], as beagle_quantize_rows_e4m3 makes them.
     * When given, beagle_draft_step with more than 8 rows (bf16 configurations) streams these bytes instead of w_lm:
     * the step's states h are quantised the same way per row and z = scale_h * scale_w * (q_h . q_w), accumulated
     * in fp32.  Every other entry point (and smaller batches) keeps using w_lm, which must still be valid. */
    const void* w_lm_fp8;
    const float* w_lm_scale;
} beagle_weights;

/* Bytes of the key/value cache ([2][max_slots][Hkv][max_ctx+max_draft][dh] in the storage type)
 * and of the serve-time workspace.  Both buffers must be 256-byte aligned. */
beagle_status beagle_query_sizes(const beagle_config* cfg, size_t* kv_bytes, size_t* workspace_bytes);

/* Creates the host-side bookkeeping (lengths of every slot start at zero).  kv_dev and
 * workspace_dev stay owned by the caller and must outlive the context; their contents need not be
 * initialised. */
beagle_status beagle_create(const beagle_config* cfg, const beagle_weights* weights_dev,
                            void* kv_dev, size_t kv_bytes, void* workspace_dev, size_t workspace_bytes,
                            beagle_ctx** out);
beagle_status beagle_destroy(beagle_ctx* ctx);

/* Key/value projection and cache append over TRUE states (Eq. 2 first line; Section 4.1, cache
 * paragraph: after every iteration the cache is cut back to the true states).  For each b < batch:
 * the draft tail of slot seq_slot[b] is dropped, then new_len[b] rows of `hidden_dev` are projected
 * with W_k, W_v and appended.  hidden_dev is packed row-major [sum(new_len), d] in the storage type,
 * sequences in call order.  seq_slot and new_len are HOST arrays; slots must be distinct.
 * new_len[b] == 0 only resets.  CAPACITY if a slot would exceed max_ctx. */
beagle_status beagle_prefill_kv(beagle_ctx* ctx, int32_t batch, const int32_t* seq_slot_host,
                                const int32_t* new_len_host, const void* hidden_dev, void* stream);

/* One drafted token for each of `batch` sequences (Eq. 1, Eq. 2, LM head, greedy token).
 * tokens_in_dev: int32 [batch] query tokens, or NULL to continue from each slot's previous greedy
 *   token (STATE error if a slot has none since its last reset).
 * concat != 0: the previous step's output state h of the slot is projected and appended to the
 *   cache tail before attending (the paper's default, "concate"); 0: only states already in the
 *   cache are read and the previous state is discarded.
 * Outputs (any may be NULL): tokens_out_dev int32, row b at tokens_out_dev[b * tokens_out_stride]
 *   (stride 1 = dense [batch]; stride gamma with a base of draft + s fills column s of a
 *   [batch, gamma] draft matrix for beagle_verify_greedy); logits_out_dev fp32 [batch, V];
 *   hidden_out_dev storage type [batch, d]. */
beagle_status beagle_draft_step(beagle_ctx* ctx, int32_t batch, const int32_t* seq_slot_host,
                                const int32_t* tokens_in_dev, int32_t concat,
                                int32_t* tokens_out_dev, int32_t tokens_out_stride,
                                float* logits_out_dev, void* hidden_out_dev, void* stream);

/* Drops the draft tail of the listed slots (cache back to true states only). */
beagle_status beagle_rollback(beagle_ctx* ctx, int32_t batch, const int32_t* seq_slot_host);
/* Forgets a slot entirely (length zero). */
beagle_status beagle_reset_slot(beagle_ctx* ctx, int32_t slot);
/* Current number of true / draft states of a slot (host bookkeeping). */
beagle_status beagle_slot_lengths(const beagle_ctx* ctx, int32_t slot, int32_t* n_true, int32_t* n_draft);

/* Row-wise FP8 quantisation (for beagle_weights.w_lm_fp8 / w_lm_scale): for each of `rows` rows of `cols` elements
 * (cols a multiple of 8) of src_dev (dtype BEAGLE_FP32 | BEAGLE_BF16, dense, 16-byte aligned):
 * scale[r] = max|x[r, :]| / 448 (1 for an all-zero row), q[r, c] = E4M3(x[r, c] / scale[r]) with round to nearest
 * even and saturation; both divisions are IEEE single precision.  q_out_dev: rows * cols bytes; scale_out_dev: fp32
 * [rows].  Needs no context. */
beagle_status beagle_quantize_rows_e4m3(const void* src_dev, int32_t dtype, int64_t rows, int32_t cols, void* q_out_dev,
                                        float* scale_out_dev, void* stream);

/* Tile-major copies of the projection weights for draft steps of 9..64 rows (a re-layout of the same numbers; not part
 * of the paper; bf16 configurations).  Those steps stream every weight matrix once per call in tiles of 128 output rows
 * x 128 bytes of the reduction; in the row-major layout a tile is 128 pieces 2*in bytes apart, in the packed layout it
 * is one contiguous run of 16 KB and the tiles a thread block reads follow one another, which the memory system serves
 * faster.  Results are bit-identical with and without the copies (same tiles, same order of accumulation).
 *
 * beagle_packed_weights_bytes: size of the buffer for w_q, w_k, w_v, w_o, w_gate, w_up, w_down, w_lm (and the FP8 LM
 *   head bytes when with_fp8_lm_head != 0), each padded to whole tiles; 0 for an fp32 configuration.
 * beagle_pack_weights: writes the copies of the context's CURRENT weights into packed_dev (device, 256-byte aligned,
 *   at least that many bytes, owned by the caller, must outlive the context or the next call of this function) on
 *   `stream`, and makes beagle_draft_step / beagle_draft_tree with 9..64 rows read them from then on.  Every other
 *   path keeps reading the row-major weights, which must stay valid.  The copies do NOT follow later changes of the
 *   weights: after an update in place call this again (same buffer allowed, once no earlier call still reads it).
 *   packed_dev == NULL: back to the row-major weights.  An fp32 configuration accepts the call and does nothing.
 * Errors: INVALID_ARG (NULL context / size pointer, misaligned buffer), CAPACITY (buffer too small), CUDA. */
beagle_status beagle_packed_weights_bytes(const beagle_config* cfg, int32_t with_fp8_lm_head, size_t* bytes);
beagle_status beagle_pack_weights(beagle_ctx* ctx, void* packed_dev, size_t bytes, void* stream);

/* Workspace bytes of beagle_block_forward for `batch` sequences of S positions. */
beagle_status beagle_block_workspace_bytes(const beagle_config* cfg, int32_t batch, int32_t S, size_t* bytes);

/* Stateless block-attention forward (Section 4.2 and its mask figure): S data tokens and S true
 * states per sequence.  With n(p) = p-1 for p <= offset, else offset + block*floor((p-1-offset)/block),
 * the query at 1-based position p reads true states 1..n(p) (inverse block mask: keys of its own
 * window are hidden, and Mask_{i,j} = 0 for j >= i).  sim_steps in [1, block]: at simulation step
 * i > 1 the state predicted for window slot i-1 is written in place as the key/value of its
 * position and becomes visible to the later queries of that window, so position p = n+i finally
 * reads true 1..n plus predicted n+1..n+min(i,sim_steps)-1.  Queries are always the data tokens.
 * tokens_dev int32 [batch,S]; hidden_dev storage [batch,S,d]; outputs (nullable): logits fp32
 * [batch,S,V], argmax int32 [batch,S], hidden storage [batch,S,d].  ws_dev: 256-byte aligned. */
beagle_status beagle_block_forward(beagle_ctx* ctx, int32_t batch, int32_t S, const int32_t* tokens_dev,
                                   const void* hidden_dev, int32_t block, int32_t offset, int32_t sim_steps,
                                   float* logits_out_dev, int32_t* argmax_out_dev, void* hidden_out_dev,
                                   void* ws_dev, size_t ws_bytes, void* stream);

/* Forward of the block-attention training losses (Section 4.2): the block forward above, followed by the
 * cross-entropy -E_{t ~ p}[log q(t)] of every position, q = softmax of the draft logits at that position, p the
 * target model's distribution there (it predicts the next token, like the draft state of Eq. 1): the softmax of
 * target_logits_dev [batch, S, V] (logits_dtype BEAGLE_FP32 | BEAGLE_BF16) or the point mass at target_ids_dev
 * int32 [batch, S]; exactly one of the two is non-NULL.  stage 0 = early loss (Eq. 4; sim_steps must be 1): every
 * position inside a window counts once.  stage 1 = late loss (Eq. 7 with l = i and beta*_{i,i} = k - i + 1): the
 * window-slot-i prediction counts block - i + 1 times for i <= sim_steps and not at all beyond.  Positions
 * p <= offset lie in no window.  loss_out_dev fp32 [1] = sum of the weighted terms / (batch * windows), windows =
 * ceil((S - offset) / block), summed in a fixed order; ce_out_dev fp32 [batch, S] (nullable) = every position's
 * unweighted cross-entropy.  The logits are never materialised (bf16 configurations).  Workspace as for
 * beagle_block_forward.  No gradients are computed. */
beagle_status beagle_block_loss(beagle_ctx* ctx, int32_t batch, int32_t S, const int32_t* tokens_dev, const void* hidden_dev,
                                int32_t block, int32_t offset, int32_t sim_steps, int32_t stage, const void* target_logits_dev,
                                int32_t logits_dtype, const int32_t* target_ids_dev, float* loss_out_dev, float* ce_out_dev,
                                void* ws_dev, size_t ws_bytes, void* stream);

/* Gradient buffers of beagle_block_grad: fp32 DEVICE pointers shaped like the parameters of beagle_weights
 * (row-major [out, in]); a NULL entry means that gradient is not wanted and its products are skipped.  Every
 * non-NULL buffer is overwritten (not accumulated into).  Owned by the caller. */
typedef struct beagle_grads {
    float* embed;    /* [V, d]: scatter-add of the query-side input gradients by token id (fp32 atomics: the
                        order of the additions, hence the last bits, may differ between runs) */
    float* g_q;      /* [d]        */
    float* w_q;      /* [Hq*dh, d] */
    float* w_k;      /* [Hkv*dh, d]*/
    float* w_v;      /* [Hkv*dh, d]*/
    float* w_o;      /* [d, Hq*dh] */
    float* g_mlp;    /* [d]        */
    float* w_gate;   /* [m, d]     */
    float* w_up;     /* [m, d]     */
    float* w_down;   /* [d, m]     */
    float* w_lm;     /* [V, d]     */
} beagle_grads;

/* Workspace bytes of beagle_block_grad for `batch` sequences of S positions. */
beagle_status beagle_block_grad_workspace_bytes(const beagle_config* cfg, int32_t batch, int32_t S, size_t* bytes);

/* One training step of the block path (Section 4.2; Appendix B for the regression term): the forward of
 * beagle_block_loss, then the gradient of
 *     total = L + vloss_coef * vloss
 * in every parameter whose entry of `grads` is non-NULL.  L is the early (Eq. 4, stage 0) or late (Eq. 7, stage 1)
 * loss exactly as beagle_block_loss defines it.  vloss is the hidden-state regression of Appendix B (the one of the
 * EAGLE papers): the mean, over the positions that carry a loss term (weight > 0) and over the d components, of
 * smooth_l1(h_hat_p - h_p), smooth_l1(r) = r^2/2 for |r| < 1 and |r| - 1/2 otherwise, h_hat_p the draft state at
 * position p (row p of the block forward's hidden output) and h_p = hidden_dev[b, p], the target's true state at
 * the same position.
 * Simulation (sim_steps > 1): the states predicted at earlier simulation steps enter the final step as key/value
 * inputs, like the true states they replace; they are constants of the differentiation, and W_k / W_v receive the
 * gradient of projecting them.  With sim_steps = 1 nothing is cut.
 * Arguments as for beagle_block_loss; vloss_coef >= 0 (the paper trains with 10).  loss_out_dev fp32 [3] =
 * {L, vloss, total}.  Intermediate gradients are kept in the storage type (bf16 or fp32), accumulated in fp32 inside
 * every product; parameter gradients are fp32 and, except `embed`, summed in a fixed order.  hidden, mlp_dim and
 * head_dim must be multiples of 8 (SHAPE otherwise).  ws_dev: 256-byte aligned, beagle_block_grad_workspace_bytes. */
beagle_status beagle_block_grad(beagle_ctx* ctx, int32_t batch, int32_t S, const int32_t* tokens_dev, const void* hidden_dev,
                                int32_t block, int32_t offset, int32_t sim_steps, int32_t stage, const void* target_logits_dev,
                                int32_t logits_dtype, const int32_t* target_ids_dev, float vloss_coef, const beagle_grads* grads,
                                float* loss_out_dev, void* ws_dev, size_t ws_bytes, void* stream);

/* Greedy acceptance (Section 3: in greedy decoding the draft's and the target's top-1 tokens are
 * matched and only a contiguous prefix is accepted, plus one extra target token).  Exactly one of
 * target_logits_dev ([batch, gamma+1, V], logits_dtype BEAGLE_FP32 or BEAGLE_BF16) and
 * target_ids_dev (int32 [batch, gamma+1]) is non-NULL.  accept_len_dev[b] = a = number of leading
 * drafts equal to the target's top-1; out_tokens_dev[b] = g_1..g_{a+1} then -1 padding
 * ([batch, gamma+1]); tau = a + 1.  draft_tokens_dev int32 [batch, gamma]; gamma <= 64. */
beagle_status beagle_verify_greedy(beagle_ctx* ctx, int32_t batch, int32_t gamma,
                                   const int32_t* draft_tokens_dev, const void* target_logits_dev,
                                   int32_t logits_dtype, const int32_t* target_ids_dev,
                                   int32_t* accept_len_dev, int32_t* out_tokens_dev, void* stream);

/* Acceptance under sampling (Section 3: each draft is accepted with probability min(1, p(t)/q(t)); at the
 * first rejection j, or at j = gamma+1 when nothing was rejected, one token is drawn from the
 * normalised max(0, p_j - q_j), from p_{gamma+1} in the latter case).  p = softmax(target / temperature),
 * q = softmax(draft / temperature).  The random numbers are the caller's: u_accept_dev fp32 [batch, gamma]
 * and u_resample_dev fp32 [batch], uniform in [0, 1); the extra token is the smallest id whose
 * cumulative residual mass exceeds u_resample times the total.  draft_logits_dev: fp32
 * [gamma, batch, V], one [batch, V] block per draft step as beagle_draft_step writes it;
 * target_logits_dev: [batch, gamma+1, V], logits_dtype BEAGLE_FP32 or BEAGLE_BF16; logits are finite.
 * accept_len_dev[b] = a; out_tokens_dev[b] = the a accepted drafts, the extra token, then -1
 * ([batch, gamma+1]).  gamma <= 64, temperature > 0. */
beagle_status beagle_verify_sample(beagle_ctx* ctx, int32_t batch, int32_t gamma, const int32_t* draft_tokens_dev,
                                   const float* draft_logits_dev, const void* target_logits_dev, int32_t logits_dtype,
                                   float temperature, const float* u_accept_dev, const float* u_resample_dev,
                                   int32_t* accept_len_dev, int32_t* out_tokens_dev, void* stream);

/* Dynamic draft tree for one sequence (the draft tree of the experimental setup, Section 5.1, i.e. the
 * method of EAGLE-2 with depth = 1 + `depth`, `topk` children per node and `n_candidates` nodes kept; the paper's
 * runs use 6, 10 and 60).  The root token *root_token_dev (the target's last token) is forwarded over the slot's true
 * states; its topk most likely next tokens become the first frontier, each scored by its log-probability.  `depth`
 * times every frontier node is forwarded -- it reads the true states plus the draft states of the root and of its own
 * ancestors, which are projected into the cache tail as in beagle_draft_step with concat -- and proposes its topk
 * children with score = own score + log-probability; the topk best of all children form the next frontier.  Finally
 * the n_candidates best nodes overall are written in creation order: tree_tokens_dev int32 [n_candidates],
 * tree_parents_dev int32 (index into the same arrays, -1 = child of the root), tree_scores_dev fp32.  Equal values
 * are ordered by the smaller token id / the earlier node.  The whole tree is drafted without a host synchronisation.
 * Limits: topk <= 16, depth <= 8, n_candidates <= 64 and <= topk + depth*topk^2; 1 + (depth-1)*topk <= max_draft;
 * bf16 configurations with head_dim 64 or 128.  Any chain-draft tail of the slot is dropped first; afterwards the
 * slot holds true states only (call beagle_prefill_kv with the accepted states as usual). */
beagle_status beagle_draft_tree(beagle_ctx* ctx, int32_t slot, const int32_t* root_token_dev, int32_t depth, int32_t topk,
                                int32_t n_candidates, int32_t* tree_tokens_dev, int32_t* tree_parents_dev, float* tree_scores_dev,
                                void* stream);

/* Greedy acceptance on a draft tree (Section 3 applied along the tree's paths): target_ids_dev int32 [n_nodes + 1]
 * holds the target's top-1 token at the root ([0]) and after every node n ([1 + n]).  Starting at the root the child
 * whose token equals the target's token at the current node is followed; where none matches the walk stops and the
 * target's token there is emitted.  accept_len_dev[0] = nodes accepted; out_tokens_dev int32 [out_cap] = the emitted
 * tokens then -1 (out_cap >= depth + 2 holds every case); path_dev int32 [out_cap] (nullable) = the accepted nodes. */
beagle_status beagle_verify_tree_greedy(beagle_ctx* ctx, int32_t n_nodes, const int32_t* tree_tokens_dev, const int32_t* tree_parents_dev,
                                        const int32_t* target_ids_dev, int32_t out_cap, int32_t* accept_len_dev, int32_t* out_tokens_dev,
                                        int32_t* path_dev, void* stream);

/* Greedy acceptance from target logits with NO memory handed over by the caller beyond the inputs
 * and outputs.  (The paper has no counterpart: this is a packaging variant of beagle_verify_greedy.)
 *
 * Who needs it: code that must not allocate device memory at the point where it verifies a draft --
 * a serving loop whose framework took the whole GPU for its own pool at start-up, so a fresh
 * cudaMalloc would fail or stall the device; a plug-in that is only lent its input and output
 * tensors; a latency-critical path that may not run an allocator at all.  Such callers also have
 * no workspace to pass to beagle_create, so this entry point needs no context.
 *
 * How: the arg-max scratch (partial keys and row ids) is a fixed array inside the library's device
 * image, BEAGLE_STATIC_VERIFY_MAX_ROWS logit rows large (about 0.55 MB, resident on every GPU that
 * loads the library until the process exits).  The call performs no cudaMalloc/cudaFree and calls
 * no allocating routine.  batch * (gamma + 1) above that limit is rejected with
 * BEAGLE_ERR_CAPACITY and a message in err_buf (optional HOST buffer of err_len bytes).
 *
 * The first call on each device looks up the array's device address (a host-side query, done with
 * that device current); make that first call outside any stream capture.  All calls on a device
 * share the one array: it keeps the previous call's contents, which is harmless because every
 * entry that is read is written first by the same call -- but two calls whose kernels can overlap
 * on the GPU (different streams, no dependency between them) race on it.  Serialise them.
 *
 * Arguments as in beagle_verify_greedy with target logits ([batch, gamma+1, vocab], logits_dtype
 * BEAGLE_FP32 or BEAGLE_BF16); results are identical to that call's. */
#define BEAGLE_STATIC_VERIFY_MAX_ROWS 4160
beagle_status beagle_verify_greedy_static(int32_t batch, int32_t gamma, int32_t vocab,
                                          const int32_t* draft_tokens_dev, const void* target_logits_dev,
                                          int32_t logits_dtype, int32_t* accept_len_dev, int32_t* out_tokens_dev,
                                          void* stream, char* err_buf, size_t err_len);

/* Optional per-stage timing (no counterpart in the paper; measurement support).  While enabled,
 * every stage of every entry point is bracketed by a pair of CUDA events recorded on the call's
 * stream.  beagle_profile_read waits for the recorded events, writes the accumulated milliseconds
 * and the number of bracketed stage instances into two HOST arrays of beagle_profile_stage_count()
 * entries, and clears the record.  Stage names: beagle_profile_stage_name(i). */
beagle_status beagle_profile_enable(beagle_ctx* ctx, int32_t on);
beagle_status beagle_profile_read(beagle_ctx* ctx, float* ms_out_host, int32_t* count_out_host);
int32_t beagle_profile_stage_count(void);
const char* beagle_profile_stage_name(int32_t stage);

/* Inspection of the intermediate vectors (no counterpart in the paper; test support).  Every step of
 * Eq. 1 / Eq. 2 leaves its result in the caller-owned workspace; these calls say where, so that a
 * checker can compare each kernel's output with the definition applied to that kernel's own inputs.
 * Rows are the batch rows of the most recent beagle_draft_step (serve) or the batch*S positions of
 * the most recent beagle_block_forward (block), row-major in the storage type. */
enum {
    BEAGLE_BUF_X = 0,      /* e(t)                              [rows, d]      */
    BEAGLE_BUF_XN = 1,     /* RMSNorm(e(t); g_q)                [rows, d]      */
    BEAGLE_BUF_Q = 2,      /* W_q xn                            [rows, Hq*dh]  */
    BEAGLE_BUF_O = 3,      /* attention output                  [rows, Hq*dh]  */
    BEAGLE_BUF_Y = 4,      /* W_o o + e(t)                      [rows, d]      */
    BEAGLE_BUF_YN = 5,     /* RMSNorm(y; g_mlp)                 [rows, d]      */
    BEAGLE_BUF_ACT = 6,    /* SiLU(W_gate yn) * (W_up yn)       [rows, m]      */
    BEAGLE_BUF_H = 7,      /* W_down act + y                    [rows, d]      */
    BEAGLE_BUF_KT = 8,     /* block path only: K of the true states       [rows, Hkv*dh] */
    BEAGLE_BUF_VT = 9,     /* block path only: V of the true states       [rows, Hkv*dh] */
    BEAGLE_BUF_KP = 10,    /* block path only: K of the predicted states  [rows, Hkv*dh] */
    BEAGLE_BUF_VP = 11,    /* block path only: V of the predicted states  [rows, Hkv*dh] */
    BEAGLE_BUF_COUNT = 12
};
/* Byte offset and row width (elements) of a serve-time buffer inside the workspace given to beagle_create. */
beagle_status beagle_workspace_buffer(const beagle_config* cfg, int32_t which, size_t* offset_bytes, int32_t* row_elems);
/* The same for the workspace of beagle_block_forward(batch, S).  BEAGLE_BUF_H is only meaningful
 * when hidden_out_dev was NULL (otherwise h went to the caller's buffer). */
beagle_status beagle_block_workspace_buffer(const beagle_config* cfg, int32_t batch, int32_t S, int32_t which,
                                            size_t* offset_bytes, int32_t* row_elems);

/* Waits for the stream, then reports BEAGLE_ERR_DEVICE if any kernel of this context abandoned a
 * bounded wait since the last check (its outputs are then undefined); the condition is reported once
 * and cleared, the context stays usable.  Besides the one-time set-up of a context's first launching
 * call, the only call that synchronises. */
beagle_status beagle_check_device(beagle_ctx* ctx, void* stream);

/* Test support for the error path above.  Every wait inside the tensor-core kernels (on a TMA copy, on
 * an MMA commit) is bounded: after a fixed number of polls the kernel raises the context's device
 * error word, lets its outstanding copies land, frees its tensor memory and returns.  This call
 * launches a one-CTA kernel that performs such a wait on a barrier nothing will ever complete, with a
 * short limit and no copy in flight: the wait runs out (nothing hangs, nothing faults) and the next
 * beagle_check_device returns BEAGLE_ERR_DEVICE.  The paper has no counterpart. */
beagle_status beagle_selftest_wait_timeout(beagle_ctx* ctx, void* stream);

/* Text of the last error recorded on this context ("" if none). */
const char* beagle_last_error(const beagle_ctx* ctx);
/* Number of kernels this context has launched so far. */
int64_t beagle_launch_count(const beagle_ctx* ctx);
/* Library version string. */
const char* beagle_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BEAGLE_H */
