// C ABI of the Beagle draft-head library: host-side validation, cache bookkeeping and the launch
// sequence of every entry point.  No device memory is allocated and no stream is created here.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "../../include/beagle.h"
#include "kernels.h"
#include "gemm_tc.h"

using namespace beagle;

enum Stage {
    ST_KV_APPEND = 0, ST_EMBED_NORM, ST_Q_PROJ, ST_ATTN_DECODE, ST_O_PROJ, ST_MLP_NORM, ST_GATE_UP, ST_DOWN, ST_LM_HEAD,
    ST_ARGMAX, ST_PREFILL, ST_VERIFY, ST_BLK_EMBED, ST_BLK_QKV, ST_BLK_PRED_KV, ST_BLK_ATTN, ST_BLK_O, ST_BLK_NORM,
    ST_BLK_GATE_UP, ST_BLK_DOWN, ST_BLK_LM_HEAD, ST_BLK_ARGMAX, ST_BWD_DLOGITS, ST_BWD_DX, ST_BWD_DW, ST_BWD_ATTN,
    ST_BWD_TRANSPOSE, ST_BWD_ELEMENTWISE, ST_QKV_PROJ, ST_COUNT
};
static const char* const kStageNames[ST_COUNT] = {
    "kv_append", "embed_norm", "q_proj", "attn_decode", "o_proj", "mlp_norm", "gate_up", "down_proj", "lm_head",
    "argmax_finalize", "prefill_kv", "verify", "blk_embed", "blk_qkv", "blk_pred_kv", "blk_attn", "blk_o_proj", "blk_norm",
    "blk_gate_up", "blk_down", "blk_lm_head", "blk_argmax", "bwd_dlogits", "bwd_dx_gemm", "bwd_dw_gemm", "bwd_attn",
    "bwd_transpose", "bwd_elementwise", "qkv_proj"};

struct StageRecord { int stage; cudaEvent_t start, stop; };

struct beagle_ctx {
    beagle_config cfg;
    beagle_weights w;
    char* kv = nullptr;
    char* ws = nullptr;
    size_t kv_bytes = 0, ws_bytes = 0;
    int cap = 0;            // rows per (slot, head) of the cache
    size_t elt = 0;         // bytes per stored element
    int qd = 0, kd = 0;
    // cache halves
    void* kcache = nullptr;
    void* vcache = nullptr;
    // serve-time workspace regions
    void *x, *xn, *q, *o, *y, *yn, *act, *h, *h_slot, *hs, *attn_scratch;
    float* sk_partial = nullptr;    // fp32 split partials of the tensor-core serve projections
    int32_t *last_token, *ids;
    unsigned long long *lm_partials, *verify_keys;
    void* vs_scratch = nullptr;     // log-sum-exp partials and chunk masses of beagle_verify_sample
    void* tree_mem = nullptr;       // node / frontier arrays of beagle_draft_tree
    float* tree_logits = nullptr;   // [kTreeMaxTopk, V] logits of the frontier rows
    void* hq = nullptr;             // FP8 LM head: quantised states of the step and their row scales
    float* hscale = nullptr;
    float* rope_table = nullptr;    // (cos, sin) per (position, i < dh/2); rotary option only
    int rope_rows = 0;              // positions the table covers
    std::vector<int32_t> steps;     // draft steps of a slot since its cache was last reset to true states
    int* dev_error = nullptr;       // device word raised by a kernel whose bounded wait ran out; the zero-initialised counters follow it
    int sm_count = 148;
    bool dev_ready = false;         // device_setup_once has run
    int lm_blocks = 0;
    // host bookkeeping
    std::vector<int32_t> n_true, n_draft;
    std::vector<char> pending;      // slot has an output state not yet appended
    std::vector<char> has_token;    // slot has a previous greedy token
    std::string err;
    int64_t launches = 0;
    TcPlan* tc = nullptr;           // tensor-core GEMM plans (bf16 only)
    // optional per-stage timing with CUDA events (off by default)
    bool profiling = false;
    std::vector<StageRecord> records;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> free_events;
};

#ifdef BEAGLE_BOUNDS_CHECK
namespace beagle {
__device__ int* g_bounds_word = nullptr;
__device__ int g_bounds_slots = 0;
}  // namespace beagle
#endif

namespace {
// Brackets one stage with events on the call's stream while profiling is on.
struct StageTimer {
    beagle_ctx* ctx;
    cudaStream_t stream;
    StageRecord rec;
    bool on;
    StageTimer(beagle_ctx* c, int stage, cudaStream_t s) : ctx(c), stream(s), on(c->profiling) {
        if (!on) return;
        rec.stage = stage;
        if (!ctx->free_events.empty()) {
            rec.start = ctx->free_events.back().first;
            rec.stop = ctx->free_events.back().second;
            ctx->free_events.pop_back();
        } else if (cudaEventCreate(&rec.start) != cudaSuccess || cudaEventCreate(&rec.stop) != cudaSuccess) {
            on = false;
            return;
        }
        cudaEventRecord(rec.start, stream);
    }
    ~StageTimer() {
        if (!on) return;
        cudaEventRecord(rec.stop, stream);
        ctx->records.push_back(rec);
    }
};
}  // namespace

namespace {

constexpr size_t kAlign = 256;
constexpr int kServeTcMinBatch = 8;     // serve-time batches above this use the tensor-core projections
constexpr int kPrefillSkinnyMaxRows = 512;   // prefill calls up to this many rows use the same kernels in chunks
size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

beagle_status fail(beagle_ctx* ctx, beagle_status st, const char* fmt, ...) {
    if (ctx != nullptr) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof(buf), fmt, ap);
        va_end(ap);
        ctx->err = buf;
    }
    return st;
}

beagle_status check_config(const beagle_config* c) {
    if (c == nullptr) return BEAGLE_ERR_INVALID_ARG;
    if (c->dtype != BEAGLE_FP32 && c->dtype != BEAGLE_BF16) return BEAGLE_ERR_INVALID_ARG;
    if (c->hidden <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->head_dim <= 0 || c->mlp_dim <= 0 ||
        c->vocab <= 0 || c->max_slots <= 0 || c->max_ctx <= 0 || c->max_draft < 0)
        return BEAGLE_ERR_INVALID_ARG;
    if (!(c->rms_eps >= 0.f)) return BEAGLE_ERR_INVALID_ARG;
    if (!(c->rope_theta >= 0.f) || (c->rope_theta > 0.f && c->rope_theta < 1.f)) return BEAGLE_ERR_INVALID_ARG;
    if (c->hidden % 8 || c->mlp_dim % 8) return BEAGLE_ERR_SHAPE;
    if (c->n_q_heads % c->n_kv_heads) return BEAGLE_ERR_SHAPE;
    const int g = c->n_q_heads / c->n_kv_heads;
    if (g != 1 && g != 2 && g != 4 && g != 8) return BEAGLE_ERR_SHAPE;
    const int vec = c->dtype == BEAGLE_BF16 ? 8 : 4;
    const int lpk = c->head_dim / vec;
    if (c->head_dim % vec || (lpk != 4 && lpk != 8 && lpk != 16 && lpk != 32)) return BEAGLE_ERR_SHAPE;
    // the widest rows (32 pieces of 16 bytes) with eight grouped query heads would need more static shared memory than
    // a decode-attention CTA has (bf16, head_dim 256, Hq / Hkv = 8): no kernel serves that shape
    if (lpk == 32 && g * c->head_dim > 1024) return BEAGLE_ERR_SHAPE;
    return BEAGLE_OK;
}

struct ServeLayout {
    size_t x, xn, q, o, y, yn, act, h, h_slot, hs, attn, sk_partial, last_token, ids, lm_partials, verify_keys, vs_scratch, tree_mem, tree_logits, rope, hq, hscale, dev_error, total;
    int lm_blocks;
};
// Device words that must read zero before the first kernel uses them: the error word (first 256 bytes), one completion
// counter per (row, K/V head) of the decode attention, one ticket per row of the greedy verification.
size_t dev_words_bytes(const beagle_config& c) {
    return 256 + (size_t)BEAGLE_MAX_CALL_BATCH * c.n_kv_heads * sizeof(int32_t) + (size_t)BEAGLE_MAX_CALL_BATCH * sizeof(int32_t);
}
ServeLayout serve_layout(const beagle_config& c) {
    ServeLayout L;
    const size_t elt = c.dtype == BEAGLE_BF16 ? 2 : 4;
    const size_t B = BEAGLE_MAX_CALL_BATCH;
    const size_t d = c.hidden, qd = (size_t)c.n_q_heads * c.head_dim, m = c.mlp_dim;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes); return at; };
    L.x = take(B * d * elt); L.xn = take(B * d * elt);
    L.q = take(B * qd * elt); L.o = take(B * qd * elt);
    L.y = take(B * d * elt); L.yn = take(B * d * elt);
    L.act = take(B * m * elt); L.h = take(B * d * elt);
    L.h_slot = take((size_t)c.max_slots * d * elt);
    L.hs = take(B * d * elt);
    {
        const int kd = c.n_kv_heads * c.head_dim;
        size_t need = 0;
        if (c.dtype == BEAGLE_BF16) {
            const size_t cand[5] = {tc_skinny_partial_bytes((int)qd, (int)d, 1), tc_skinny_partial_bytes(kd, (int)d, 2),
                                    tc_skinny_partial_bytes((int)d, (int)qd, 1), tc_skinny_partial_bytes((int)m, (int)d, 2),
                                    tc_skinny_partial_bytes((int)d, (int)m, 1)};
            for (size_t v : cand) need = v > need ? v : need;
        }
        L.sk_partial = take(need);
    }
    L.attn = take(attn_decode_scratch_bytes((int)B, c.n_q_heads, c.head_dim, c.max_ctx + c.max_draft));
    L.last_token = take((size_t)c.max_slots * sizeof(int32_t));
    L.ids = take(B * 65 * sizeof(int32_t));
    L.lm_blocks = gemv_grid_blocks(GEMV_LOGITS, c.vocab);
    L.lm_partials = take(B * (size_t)L.lm_blocks * sizeof(unsigned long long));
    L.verify_keys = take(B * 65 * kVerifyMaxSplit * sizeof(unsigned long long));
    L.vs_scratch = take(verify_sample_scratch_bytes((int)B, 64));
    L.tree_mem = take(tree_arrays_bytes(c.vocab));
    L.tree_logits = take(c.dtype == BEAGLE_BF16 ? (size_t)kTreeMaxTopk * c.vocab * sizeof(float) : 0);
    L.rope = take(c.rope_theta > 0.f ? ((size_t)c.max_ctx + c.max_draft + 1) * (c.head_dim / 2) * 2 * sizeof(float) : 0);
    L.hq = take(B * d); L.hscale = take(B * sizeof(float));                    // FP8 LM head: the step's states as E4M3 bytes + row scales
    L.dev_error = take(dev_words_bytes(c));    // error word, the attention completion counters, the verification tickets
    L.total = off;
    return L;
}

struct BlockLayout {
    size_t x, xn, q, kt, vt, kp, vp, vtT, vpT, o, y, yn, act, h, logits, keys, ids, ce_part, ce_rows, wce, rope, total;
    int Sp;             // positions per sequence padded to a multiple of 8 (columns of a sequence in the transposed values)
    int lm_chunk_rows;
};
constexpr int kLmChunkRows = 2048;
BlockLayout block_layout(const beagle_config& c, int batch, int S) {
    BlockLayout L;
    const size_t elt = c.dtype == BEAGLE_BF16 ? 2 : 4;
    const size_t M = (size_t)batch * S;
    const size_t d = c.hidden, qd = (size_t)c.n_q_heads * c.head_dim, kd = (size_t)c.n_kv_heads * c.head_dim, m = c.mlp_dim;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes); return at; };
    L.x = take(M * d * elt); L.xn = take(M * d * elt); L.q = take(M * qd * elt);
    L.kt = take(M * kd * elt); L.vt = take(M * kd * elt); L.kp = take(M * kd * elt); L.vp = take(M * kd * elt);
    L.Sp = (S + 7) / 8 * 8;
    L.vtT = take(0); L.vpT = take(0);          // (transposed values: no longer made)
    L.o = take(M * qd * elt); L.y = take(M * d * elt); L.yn = take(M * d * elt);
    L.act = take(M * m * elt); L.h = take(M * d * elt);
    L.lm_chunk_rows = (int)(M < (size_t)kLmChunkRows ? M : (size_t)kLmChunkRows);
    L.logits = take((size_t)L.lm_chunk_rows * c.vocab * sizeof(float));
    const size_t key_cols = (size_t)(tc_argmax_tiles(c.vocab) > kRowArgmaxSplit ? tc_argmax_tiles(c.vocab) : kRowArgmaxSplit);
    L.keys = take(M * key_cols * sizeof(unsigned long long));
    L.ids = take(M * sizeof(int32_t));
    L.ce_part = take(M * (size_t)tc_argmax_tiles(c.vocab) * kCeFields * sizeof(float));     // loss forward: per (row, column tile)
    L.ce_rows = take(M * sizeof(float));
    L.wce = take(M * sizeof(float));
    L.rope = take(c.rope_theta > 0.f ? (size_t)S * (c.head_dim / 2) * 2 * sizeof(float) : 0);
    L.total = off;
    return L;
}

// Workspace of one training step: the forward's regions, then what the backward adds.
struct GradLayout {
    BlockLayout fwd;
    size_t gate, up, dact, dz, dh0, dh, dyn, dy, d_o, dq, dkt, dvt, dkp, dvp, dxn, ta, tb, wt, qT, doT, ktT, kpT, lse, delta, stats, coef, vrow, dgpart, total;
    int Mp, Vp;        // rows and vocabulary padded to a multiple of 8 (contraction lengths of the transposed products)
};
GradLayout grad_layout(const beagle_config& c, int batch, int S) {
    GradLayout L;
    L.fwd = block_layout(c, batch, S);
    const size_t elt = c.dtype == BEAGLE_BF16 ? 2 : 4;
    const size_t M = (size_t)batch * S;
    const size_t d = c.hidden, qd = (size_t)c.n_q_heads * c.head_dim, kd = (size_t)c.n_kv_heads * c.head_dim, m = c.mlp_dim, V = c.vocab;
    L.Mp = (int)((M + 7) / 8 * 8);
    L.Vp = (int)((V + 7) / 8 * 8);
    size_t off = L.fwd.total;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes); return at; };
    auto max2 = [](size_t a, size_t b) { return a > b ? a : b; };
    L.gate = take(M * m * elt); L.up = take(M * m * elt); L.dact = take(M * m * elt);
    L.dz = take(M * (size_t)L.Vp * elt);
    L.dh0 = take(M * d * elt); L.dh = take(M * d * elt); L.dyn = take(M * d * elt); L.dy = take(M * d * elt);
    L.d_o = take(M * qd * elt); L.dq = take(M * qd * elt);
    L.dkt = take(M * kd * elt); L.dvt = take(M * kd * elt); L.dkp = take(M * kd * elt); L.dvp = take(M * kd * elt);
    L.dxn = take(M * d * elt);
    // transposed operands: TA holds d(out)^T [features, rows], TB the layer input^T; K/V use two row blocks side by side
    const size_t widest = max2(max2(V, m), max2(qd, d));
    L.ta = take(max2(widest * (size_t)L.Mp, kd * 2 * (size_t)L.Mp) * elt);
    L.tb = take(max2(max2(m, qd) * (size_t)L.Mp, d * 2 * (size_t)L.Mp) * elt);
    // one transposed weight at a time: [in, out] (hidden, mlp_dim and head_dim are multiples of 8; the vocabulary is padded)
    L.wt = take(max2(d * (size_t)L.Vp, max2(m, qd) * d) * elt);
    // transposed copies for the tcgen05 attention backward (bf16 only)
    L.qT = take(0); L.doT = take(0); L.ktT = take(0); L.kpT = take(0);      // (transposed copies for the attention backward: no longer made)
    L.lse = take(M * c.n_q_heads * sizeof(float)); L.delta = take(M * c.n_q_heads * sizeof(float));
    L.stats = take(M * 4 * sizeof(float)); L.coef = take(M * sizeof(float)); L.vrow = take(M * sizeof(float));
    L.dgpart = take((size_t)rmsnorm_bwd_parts((int)M) * d * sizeof(float));
    L.total = off;
    return L;
}

int* attn_done_counters(beagle_ctx* ctx) { return ctx->dev_error + 64; }
int* verify_tickets(beagle_ctx* ctx) { return ctx->dev_error + 64 + BEAGLE_MAX_CALL_BATCH * ctx->cfg.n_kv_heads; }

beagle_status cuda_ok(beagle_ctx* ctx, const char* what) {
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ctx, BEAGLE_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    return BEAGLE_OK;
}

// One-time device set-up of a context, done by the first call that launches anything: the device words (error word,
// completion counters, verification tickets) are zeroed and, with the rotary option, the (cos, sin) table is built; the
// call then waits for both, so that later calls find them ready whatever stream they use.  Work enqueued inside a
// stream capture would be recorded, not run, so a first call inside a capture is refused.
beagle_status device_setup_once(beagle_ctx* ctx, cudaStream_t stream) {
    if (ctx->dev_ready) return BEAGLE_OK;
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess)
        return fail(ctx, BEAGLE_ERR_CUDA, "device set-up: %s", cudaGetErrorString(cudaGetLastError()));
    if (cs != cudaStreamCaptureStatusNone)
        return fail(ctx, BEAGLE_ERR_STATE, "the first launching call on a context must be made outside stream capture");
    if (cudaMemsetAsync(ctx->dev_error, 0, dev_words_bytes(ctx->cfg), stream) != cudaSuccess)
        return fail(ctx, BEAGLE_ERR_CUDA, "device set-up: %s", cudaGetErrorString(cudaGetLastError()));
    if (ctx->cfg.rope_theta > 0.f)
        ctx->launches += launch_rope_table(ctx->cfg.rope_theta, ctx->cfg.head_dim, ctx->rope_rows, ctx->rope_table, stream);
#ifdef BEAGLE_BOUNDS_CHECK
    {   // bounds-checking build: the kernels' index checks report into this context's error word
        int* word = ctx->dev_error;
        int slots = ctx->cfg.max_slots;
        if (cudaMemcpyToSymbolAsync(g_bounds_word, &word, sizeof(word), 0, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
            cudaMemcpyToSymbolAsync(g_bounds_slots, &slots, sizeof(slots), 0, cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return fail(ctx, BEAGLE_ERR_CUDA, "device set-up: %s", cudaGetErrorString(cudaGetLastError()));
    }
#endif
    if (cudaStreamSynchronize(stream) != cudaSuccess)
        return fail(ctx, BEAGLE_ERR_CUDA, "device set-up: %s", cudaGetErrorString(cudaGetLastError()));
    ctx->dev_ready = true;
    return BEAGLE_OK;
}

// One dense projection C = A W^T of the block / prefill path: tensor cores when the plan covers the
// shape (bf16), the CUDA-core kernel otherwise.
int dense_gemm(beagle_ctx* ctx, int epi, const GemmArgs& a, cudaStream_t stream) {
    if (ctx->tc != nullptr) {
        GemmArgs t = a;
        t.error_word = ctx->dev_error;
        const int rc = tc_gemm(ctx->tc, epi, t, stream);
        if (rc >= 0) return rc;
    }
    if (epi == GEMM_ARGMAX_KEYS || epi == GEMM_CE || epi == GEMM_DLOGITS || epi == GEMM_KV_CACHE_PAIR || a.a_mn || a.b_mn) return -1;
    return launch_gemm_simt(ctx->cfg.dtype, epi, a, stream);
}

}  // namespace

extern "C" {

#ifdef BEAGLE_BOUNDS_CHECK
const char* beagle_version(void) { return "beagle-b200 0.2 (sm_100a, bounds-checking build)"; }
#else
const char* beagle_version(void) { return "beagle-b200 0.2 (sm_100a)"; }
#endif

beagle_status beagle_query_sizes(const beagle_config* cfg, size_t* kv_bytes, size_t* workspace_bytes) {
    const beagle_status st = check_config(cfg);
    if (st != BEAGLE_OK) return st;
    if (kv_bytes == nullptr || workspace_bytes == nullptr) return BEAGLE_ERR_INVALID_ARG;
    const size_t elt = cfg->dtype == BEAGLE_BF16 ? 2 : 4;
    const size_t cap = (size_t)cfg->max_ctx + cfg->max_draft;
    *kv_bytes = 2 * align_up((size_t)cfg->max_slots * cfg->n_kv_heads * cap * cfg->head_dim * elt);
    *workspace_bytes = serve_layout(*cfg).total;
    return BEAGLE_OK;
}

beagle_status beagle_workspace_buffer(const beagle_config* cfg, int32_t which, size_t* offset_bytes, int32_t* row_elems) {
    const beagle_status st = check_config(cfg);
    if (st != BEAGLE_OK) return st;
    if (offset_bytes == nullptr || row_elems == nullptr) return BEAGLE_ERR_INVALID_ARG;
    const ServeLayout L = serve_layout(*cfg);
    const int d = cfg->hidden, qd = cfg->n_q_heads * cfg->head_dim, m = cfg->mlp_dim;
    switch (which) {
        case BEAGLE_BUF_X: *offset_bytes = L.x; *row_elems = d; break;
        case BEAGLE_BUF_XN: *offset_bytes = L.xn; *row_elems = d; break;
        case BEAGLE_BUF_Q: *offset_bytes = L.q; *row_elems = qd; break;
        case BEAGLE_BUF_O: *offset_bytes = L.o; *row_elems = qd; break;
        case BEAGLE_BUF_Y: *offset_bytes = L.y; *row_elems = d; break;
        case BEAGLE_BUF_YN: *offset_bytes = L.yn; *row_elems = d; break;
        case BEAGLE_BUF_ACT: *offset_bytes = L.act; *row_elems = m; break;
        case BEAGLE_BUF_H: *offset_bytes = L.h; *row_elems = d; break;
        default: return BEAGLE_ERR_INVALID_ARG;
    }
    return BEAGLE_OK;
}

beagle_status beagle_block_workspace_buffer(const beagle_config* cfg, int32_t batch, int32_t S, int32_t which,
                                            size_t* offset_bytes, int32_t* row_elems) {
    const beagle_status st = check_config(cfg);
    if (st != BEAGLE_OK) return st;
    if (offset_bytes == nullptr || row_elems == nullptr || batch <= 0 || S <= 0) return BEAGLE_ERR_INVALID_ARG;
    if ((long long)batch * S > (1ll << 24)) return BEAGLE_ERR_CAPACITY;
    const BlockLayout L = block_layout(*cfg, batch, S);
    const int d = cfg->hidden, qd = cfg->n_q_heads * cfg->head_dim, kd = cfg->n_kv_heads * cfg->head_dim, m = cfg->mlp_dim;
    switch (which) {
        case BEAGLE_BUF_X: *offset_bytes = L.x; *row_elems = d; break;
        case BEAGLE_BUF_XN: *offset_bytes = L.xn; *row_elems = d; break;
        case BEAGLE_BUF_Q: *offset_bytes = L.q; *row_elems = qd; break;
        case BEAGLE_BUF_O: *offset_bytes = L.o; *row_elems = qd; break;
        case BEAGLE_BUF_Y: *offset_bytes = L.y; *row_elems = d; break;
        case BEAGLE_BUF_YN: *offset_bytes = L.yn; *row_elems = d; break;
        case BEAGLE_BUF_ACT: *offset_bytes = L.act; *row_elems = m; break;
        case BEAGLE_BUF_H: *offset_bytes = L.h; *row_elems = d; break;
        case BEAGLE_BUF_KT: *offset_bytes = L.kt; *row_elems = kd; break;
        case BEAGLE_BUF_VT: *offset_bytes = L.vt; *row_elems = kd; break;
        case BEAGLE_BUF_KP: *offset_bytes = L.kp; *row_elems = kd; break;
        case BEAGLE_BUF_VP: *offset_bytes = L.vp; *row_elems = kd; break;
        default: return BEAGLE_ERR_INVALID_ARG;
    }
    return BEAGLE_OK;
}

beagle_status beagle_create(const beagle_config* cfg, const beagle_weights* w, void* kv_dev, size_t kv_bytes,
                            void* workspace_dev, size_t workspace_bytes, beagle_ctx** out) {
    if (out == nullptr) return BEAGLE_ERR_INVALID_ARG;
    *out = nullptr;
    const beagle_status st = check_config(cfg);
    if (st != BEAGLE_OK) return st;
    if (w == nullptr || kv_dev == nullptr || workspace_dev == nullptr) return BEAGLE_ERR_INVALID_ARG;
    const void* const* wp = reinterpret_cast<const void* const*>(w);
    for (size_t i = 0; i < 11; ++i)                              // the eleven parameters; the FP8 copy of the LM head is optional
        if (wp[i] == nullptr || (reinterpret_cast<uintptr_t>(wp[i]) & 15)) return BEAGLE_ERR_INVALID_ARG;
    if ((w->w_lm_fp8 == nullptr) != (w->w_lm_scale == nullptr)) return BEAGLE_ERR_INVALID_ARG;
    if (w->w_lm_fp8 != nullptr && ((reinterpret_cast<uintptr_t>(w->w_lm_fp8) & 15) || cfg->hidden % 16)) return BEAGLE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(kv_dev) & (kAlign - 1)) || (reinterpret_cast<uintptr_t>(workspace_dev) & (kAlign - 1)))
        return BEAGLE_ERR_INVALID_ARG;
    size_t need_kv, need_ws;
    beagle_query_sizes(cfg, &need_kv, &need_ws);
    if (kv_bytes < need_kv || workspace_bytes < need_ws) return BEAGLE_ERR_CAPACITY;

    beagle_ctx* c = new beagle_ctx();
    c->cfg = *cfg;
    c->w = *w;
    c->kv = static_cast<char*>(kv_dev);
    c->ws = static_cast<char*>(workspace_dev);
    c->kv_bytes = kv_bytes;
    c->ws_bytes = workspace_bytes;
    c->cap = cfg->max_ctx + cfg->max_draft;
    c->elt = cfg->dtype == BEAGLE_BF16 ? 2 : 4;
    c->qd = cfg->n_q_heads * cfg->head_dim;
    c->kd = cfg->n_kv_heads * cfg->head_dim;
    c->kcache = c->kv;
    c->vcache = c->kv + need_kv / 2;
    const ServeLayout L = serve_layout(*cfg);
    c->x = c->ws + L.x; c->xn = c->ws + L.xn; c->q = c->ws + L.q; c->o = c->ws + L.o;
    c->y = c->ws + L.y; c->yn = c->ws + L.yn; c->act = c->ws + L.act; c->h = c->ws + L.h;
    c->h_slot = c->ws + L.h_slot; c->hs = c->ws + L.hs; c->attn_scratch = c->ws + L.attn;
    c->sk_partial = reinterpret_cast<float*>(c->ws + L.sk_partial);
    c->last_token = reinterpret_cast<int32_t*>(c->ws + L.last_token);
    c->ids = reinterpret_cast<int32_t*>(c->ws + L.ids);
    c->lm_partials = reinterpret_cast<unsigned long long*>(c->ws + L.lm_partials);
    c->verify_keys = reinterpret_cast<unsigned long long*>(c->ws + L.verify_keys);
    c->vs_scratch = c->ws + L.vs_scratch;
    c->tree_mem = c->ws + L.tree_mem;
    c->tree_logits = reinterpret_cast<float*>(c->ws + L.tree_logits);
    c->hq = c->ws + L.hq;
    c->hscale = reinterpret_cast<float*>(c->ws + L.hscale);
    c->rope_table = reinterpret_cast<float*>(c->ws + L.rope);
    c->rope_rows = cfg->max_ctx + cfg->max_draft + 1;
    c->dev_error = reinterpret_cast<int*>(c->ws + L.dev_error);
    c->lm_blocks = L.lm_blocks;
    c->n_true.assign(cfg->max_slots, 0);
    c->n_draft.assign(cfg->max_slots, 0);
    c->pending.assign(cfg->max_slots, 0);
    c->steps.assign(cfg->max_slots, 0);
    c->has_token.assign(cfg->max_slots, 0);
    int hard = 0;
    c->tc = (cfg->dtype == BEAGLE_BF16) ? tc_plan_create(*cfg, *w, &hard) : nullptr;
    if (hard) {
        delete c;
        return BEAGLE_ERR_CUDA;     // a GPU is present but the tensor-map encoder is not: never fall back silently
    }
    {
        int dev = 0, sms = 0;       // grid sizing only; without a device (host-only use) the default stays
        if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
            c->sm_count = sms;
        else
            cudaGetLastError();
    }
    if (c->tc != nullptr)
        tc_attn_bind_cache(c->tc, c->kcache, c->vcache, (long long)cfg->max_slots * cfg->n_kv_heads * c->cap, cfg->head_dim);
    *out = c;
    return BEAGLE_OK;
}

static void release_events(beagle_ctx* ctx) {
    for (auto& r : ctx->records) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
    for (auto& e : ctx->free_events) { cudaEventDestroy(e.first); cudaEventDestroy(e.second); }
    ctx->records.clear();
    ctx->free_events.clear();
}

beagle_status beagle_profile_enable(beagle_ctx* ctx, int32_t on) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    ctx->profiling = on != 0;
    return BEAGLE_OK;
}

int32_t beagle_profile_stage_count(void) { return ST_COUNT; }
const char* beagle_profile_stage_name(int32_t stage) { return (stage >= 0 && stage < ST_COUNT) ? kStageNames[stage] : ""; }

beagle_status beagle_profile_read(beagle_ctx* ctx, float* ms_out, int32_t* count_out) {
    if (ctx == nullptr || ms_out == nullptr || count_out == nullptr) return BEAGLE_ERR_INVALID_ARG;
    for (int i = 0; i < ST_COUNT; ++i) { ms_out[i] = 0.f; count_out[i] = 0; }
    for (auto& r : ctx->records) {
        if (cudaEventSynchronize(r.stop) != cudaSuccess) return fail(ctx, BEAGLE_ERR_CUDA, "profile_read: event sync failed");
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, r.start, r.stop) != cudaSuccess) return fail(ctx, BEAGLE_ERR_CUDA, "profile_read: elapsed time failed");
        ms_out[r.stage] += ms;
        count_out[r.stage] += 1;
        ctx->free_events.emplace_back(r.start, r.stop);
    }
    ctx->records.clear();
    return BEAGLE_OK;
}

beagle_status beagle_destroy(beagle_ctx* ctx) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    release_events(ctx);
    tc_plan_destroy(ctx->tc);
    delete ctx;
    return BEAGLE_OK;
}

beagle_status beagle_check_device(beagle_ctx* ctx, void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (cudaStreamSynchronize(stream) != cudaSuccess) return fail(ctx, BEAGLE_ERR_CUDA, "check_device: %s", cudaGetErrorString(cudaGetLastError()));
    if (!ctx->dev_ready) return BEAGLE_OK;
    int word = 0;
    if (cudaMemcpy(&word, ctx->dev_error, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return fail(ctx, BEAGLE_ERR_CUDA, "check_device: %s", cudaGetErrorString(cudaGetLastError()));
    if (word != 0) {
        // reported once: the word is cleared so that the context stays usable and a later check speaks of later kernels; the
        // counters behind it are cleared too, since a kernel that gave up may have left its tickets half-way
        if (cudaMemset(ctx->dev_error, 0, dev_words_bytes(ctx->cfg)) != cudaSuccess)
            return fail(ctx, BEAGLE_ERR_CUDA, "check_device: %s", cudaGetErrorString(cudaGetLastError()));
        return fail(ctx, BEAGLE_ERR_DEVICE, word == 2 ? "a kernel's index check failed (bounds-checking build): the access was skipped"
                                                      : "a kernel gave up on a bounded wait (pipeline barrier never completed)");
    }
    return BEAGLE_OK;
}

beagle_status beagle_selftest_wait_timeout(beagle_ctx* ctx, void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const beagle_status st = device_setup_once(ctx, stream);
    if (st != BEAGLE_OK) return st;
    ctx->launches += launch_wait_timeout_selftest(ctx->dev_error, stream);
    return cuda_ok(ctx, "selftest_wait_timeout");
}

// The matrices that the 9..64-row serve path streams, in the order their tile-major copies lie in the caller's buffer.
namespace {
struct PackItem { const void* W; int N, K, elt_bytes; };
int pack_items(const beagle_config& c, const beagle_weights* w, bool fp8, PackItem out[9]) {
    const int qd = c.n_q_heads * c.head_dim, kd = c.n_kv_heads * c.head_dim;
    int n = 0;
    out[n++] = {w ? w->w_q : nullptr, qd, c.hidden, 2};
    out[n++] = {w ? w->w_k : nullptr, kd, c.hidden, 2};
    out[n++] = {w ? w->w_v : nullptr, kd, c.hidden, 2};
    out[n++] = {w ? w->w_o : nullptr, c.hidden, qd, 2};
    out[n++] = {w ? w->w_gate : nullptr, c.mlp_dim, c.hidden, 2};
    out[n++] = {w ? w->w_up : nullptr, c.mlp_dim, c.hidden, 2};
    out[n++] = {w ? w->w_down : nullptr, c.hidden, c.mlp_dim, 2};
    out[n++] = {w ? w->w_lm : nullptr, c.vocab, c.hidden, 2};
    if (fp8) out[n++] = {w ? w->w_lm_fp8 : nullptr, c.vocab, c.hidden, 1};
    return n;
}
}  // namespace

beagle_status beagle_packed_weights_bytes(const beagle_config* cfg, int32_t with_fp8_lm_head, size_t* bytes) {
    if (bytes == nullptr) return BEAGLE_ERR_INVALID_ARG;
    *bytes = 0;
    const beagle_status st = check_config(cfg);
    if (st != BEAGLE_OK) return st;
    if (cfg->dtype != BEAGLE_BF16) return BEAGLE_OK;
    PackItem items[9];
    const int n = pack_items(*cfg, nullptr, with_fp8_lm_head != 0, items);
    size_t total = 0;
    for (int i = 0; i < n; ++i) total += tc_skinny_packed_bytes(items[i].N, items[i].K, items[i].elt_bytes);
    *bytes = total;
    return BEAGLE_OK;
}

beagle_status beagle_pack_weights(beagle_ctx* ctx, void* packed_dev, size_t bytes, void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    if (ctx->tc == nullptr) return BEAGLE_OK;                          // fp32 configuration: nothing reads packed weights
    tc_skinny_forget_packed(ctx->tc);
    if (packed_dev == nullptr) return BEAGLE_OK;
    if (reinterpret_cast<uintptr_t>(packed_dev) & (kAlign - 1)) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "packed weights buffer is not 256-byte aligned");
    const bool fp8 = ctx->w.w_lm_fp8 != nullptr;
    size_t need = 0;
    beagle_packed_weights_bytes(&ctx->cfg, fp8 ? 1 : 0, &need);
    if (bytes < need) return fail(ctx, BEAGLE_ERR_CAPACITY, "packed weights need %zu bytes, got %zu", need, bytes);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    PackItem items[9];
    const int n = pack_items(ctx->cfg, &ctx->w, fp8, items);
    char* dst = static_cast<char*>(packed_dev);
    for (int i = 0; i < n; ++i) {
        // a matrix whose shape the tiled kernels do not take (row pitch not a multiple of 16 bytes) simply keeps its row-major form
        const int r = tc_skinny_pack(ctx->tc, items[i].W, items[i].N, items[i].K, items[i].elt_bytes, dst, stream);
        if (r > 0) ctx->launches += r;
        dst += tc_skinny_packed_bytes(items[i].N, items[i].K, items[i].elt_bytes);
    }
    return cuda_ok(ctx, "pack_weights");
}

const char* beagle_last_error(const beagle_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }
int64_t beagle_launch_count(const beagle_ctx* ctx) { return ctx ? ctx->launches : 0; }

static beagle_status check_slots(beagle_ctx* ctx, int32_t batch, const int32_t* seq_slot) {
    if (batch < 0 || batch > BEAGLE_MAX_CALL_BATCH) return fail(ctx, BEAGLE_ERR_CAPACITY, "batch %d outside [0, %d]", batch, BEAGLE_MAX_CALL_BATCH);
    if (batch > 0 && seq_slot == nullptr) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "seq_slot is NULL");
    for (int b = 0; b < batch; ++b) {
        if (seq_slot[b] < 0 || seq_slot[b] >= ctx->cfg.max_slots) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "slot %d out of range", seq_slot[b]);
        for (int c = 0; c < b; ++c)
            if (seq_slot[c] == seq_slot[b]) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "slot %d listed twice", seq_slot[b]);
    }
    return BEAGLE_OK;
}

beagle_status beagle_rollback(beagle_ctx* ctx, int32_t batch, const int32_t* seq_slot) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    const beagle_status st = check_slots(ctx, batch, seq_slot);
    if (st != BEAGLE_OK) return st;
    for (int b = 0; b < batch; ++b) {
        ctx->n_draft[seq_slot[b]] = 0;
        ctx->pending[seq_slot[b]] = 0;
        ctx->has_token[seq_slot[b]] = 0;
        ctx->steps[seq_slot[b]] = 0;
    }
    return BEAGLE_OK;
}

beagle_status beagle_reset_slot(beagle_ctx* ctx, int32_t slot) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    if (slot < 0 || slot >= ctx->cfg.max_slots) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "slot %d out of range", slot);
    ctx->n_true[slot] = ctx->n_draft[slot] = 0;
    ctx->pending[slot] = ctx->has_token[slot] = 0;
    ctx->steps[slot] = 0;
    return BEAGLE_OK;
}

beagle_status beagle_slot_lengths(const beagle_ctx* ctx, int32_t slot, int32_t* n_true, int32_t* n_draft) {
    if (ctx == nullptr || slot < 0 || slot >= ctx->cfg.max_slots) return BEAGLE_ERR_INVALID_ARG;
    if (n_true) *n_true = ctx->n_true[slot];
    if (n_draft) *n_draft = ctx->n_draft[slot];
    return BEAGLE_OK;
}

beagle_status beagle_prefill_kv(beagle_ctx* ctx, int32_t batch, const int32_t* seq_slot, const int32_t* new_len,
                                const void* hidden_dev, void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    beagle_status st = check_slots(ctx, batch, seq_slot);
    if (st != BEAGLE_OK) return st;
    if (batch > 0 && new_len == nullptr) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "new_len is NULL");
    long long total = 0;
    for (int b = 0; b < batch; ++b) {
        if (new_len[b] < 0) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "new_len[%d] < 0", b);
        if ((long long)ctx->n_true[seq_slot[b]] + new_len[b] > ctx->cfg.max_ctx)
            return fail(ctx, BEAGLE_ERR_CAPACITY, "slot %d: %d + %d true states exceed max_ctx %d", seq_slot[b],
                        ctx->n_true[seq_slot[b]], new_len[b], ctx->cfg.max_ctx);
        total += new_len[b];
    }
    if (total > 0 && hidden_dev == nullptr) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "hidden is NULL");
    if (total > (1ll << 30)) return fail(ctx, BEAGLE_ERR_CAPACITY, "too many rows");
    if (total > 0 && (reinterpret_cast<uintptr_t>(hidden_dev) & 15)) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "hidden must be 16-byte aligned");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const beagle_config& c = ctx->cfg;

    if (total > 0) {
        st = device_setup_once(ctx, stream);
        if (st != BEAGLE_OK) return st;
        StageTimer timer_(ctx, ST_PREFILL, stream);
        SeqRows rows;
        memset(&rows, 0, sizeof(rows));
        int n = 0, r = 0;
        for (int b = 0; b < batch; ++b) {
            if (new_len[b] == 0) continue;
            rows.slot[n] = seq_slot[b];
            rows.row_start[n] = r;
            rows.pos_start[n] = ctx->n_true[seq_slot[b]];
            r += new_len[b];
            ++n;
        }
        rows.n = n;
        rows.row_start[n] = r;
        const bool small = ctx->tc != nullptr ? total <= kServeTcMinBatch : total <= 16;
        if (small) {
            // few rows (the states accepted by one verification): weight-streaming path
            GemvArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_k; a.W2 = ctx->w.w_v; a.N = ctx->kd; a.K = c.hidden;
            a.X = hidden_dev; a.ldx = c.hidden; a.B = (int)total;
            a.kcache = ctx->kcache; a.vcache = ctx->vcache; a.Hkv = c.n_kv_heads; a.dh = c.head_dim; a.cap = ctx->cap;
            for (int s = 0; s < n; ++s)
                for (int i = rows.row_start[s]; i < rows.row_start[s + 1]; ++i) {
                    a.xrow.idx[i] = i;
                    a.orow2.idx[i] = rows.slot[s];
                    a.pos.idx[i] = rows.pos_start[s] + (i - rows.row_start[s]);
                }
            ctx->launches += launch_gemv(c.dtype, GEMV_KV, a, stream);
        } else if (ctx->tc != nullptr && total <= kPrefillSkinnyMaxRows) {
            // up to a few hundred rows (one verification of a whole batch): chunks of 64 rows on the
            // tensor cores with the weights as the wide operand; W_k, W_v stay in L2 between chunks
            int s = 0;
            for (int r0 = 0; r0 < (int)total; r0 += kMaxCallBatch) {
                const int nb = (int)total - r0 < kMaxCallBatch ? (int)total - r0 : kMaxCallBatch;
                SkinnyArgs a;
                memset(&a, 0, sizeof(a));
                a.W = ctx->w.w_k; a.W2 = ctx->w.w_v; a.N = ctx->kd; a.K = c.hidden;
                a.X = static_cast<const char*>(hidden_dev) + (size_t)r0 * c.hidden * ctx->elt; a.ldx = c.hidden; a.B = nb;
                a.kcache = ctx->kcache; a.vcache = ctx->vcache; a.Hkv = c.n_kv_heads; a.dh = c.head_dim; a.cap = ctx->cap;
                a.partial = ctx->sk_partial; a.error_word = ctx->dev_error;
                for (int i = 0; i < nb; ++i) {
                    while (r0 + i >= rows.row_start[s + 1]) ++s;
                    a.slot.idx[i] = rows.slot[s];
                    a.pos.idx[i] = rows.pos_start[s] + (r0 + i - rows.row_start[s]);
                }
                const int rc = tc_skinny(ctx->tc, SK_KV, a, stream);
                if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "K/V projection: unsupported shape");
                ctx->launches += rc;
            }
        } else {
            GemmArgs g;
            memset(&g, 0, sizeof(g));
            g.A = hidden_dev; g.lda = c.hidden; g.M = (int)total; g.N = ctx->kd; g.K = c.hidden;
            g.Hkv = c.n_kv_heads; g.dh = c.head_dim; g.cap = ctx->cap; g.rows = rows;
            // tensor cores: both projections in one pass over the states (the K and V weight tiles side by side in one MMA);
            // otherwise one product per matrix
            g.W = ctx->w.w_k; g.cache = ctx->kcache; g.W2 = ctx->w.w_v; g.cache2 = ctx->vcache;
            int rc = ctx->tc != nullptr ? dense_gemm(ctx, GEMM_KV_CACHE_PAIR, g, stream) : -1;
            if (rc < 0) {
                rc = dense_gemm(ctx, GEMM_KV_CACHE, g, stream);
                if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "K projection: unsupported shape");
                ctx->launches += rc;
                g.W = ctx->w.w_v; g.cache = ctx->vcache;
                rc = dense_gemm(ctx, GEMM_KV_CACHE, g, stream);
                if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "V projection: unsupported shape");
            }
            ctx->launches += rc;
        }
        if (c.rope_theta > 0.f) {       // rotary option: the new key rows are rotated in place by their positions
            ctx->launches += launch_rope_cache_rows(c.dtype, ctx->kcache, total, c.n_kv_heads, c.head_dim, ctx->cap, rows, ctx->rope_table, stream);
        }
        st = cuda_ok(ctx, "prefill_kv");
        if (st != BEAGLE_OK) return st;
    }
    for (int b = 0; b < batch; ++b) {
        const int s = seq_slot[b];
        ctx->n_true[s] += new_len[b];
        ctx->n_draft[s] = 0;
        ctx->pending[s] = 0;
        ctx->has_token[s] = 0;
        ctx->steps[s] = 0;
    }
    return BEAGLE_OK;
}

beagle_status beagle_draft_step(beagle_ctx* ctx, int32_t batch, const int32_t* seq_slot, const int32_t* tokens_in_dev,
                                int32_t concat, int32_t* tokens_out_dev, int32_t tokens_out_stride, float* logits_out_dev,
                                void* hidden_out_dev, void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    beagle_status st = check_slots(ctx, batch, seq_slot);
    if (st != BEAGLE_OK) return st;
    if (batch == 0) return BEAGLE_OK;
    if (tokens_out_dev != nullptr && tokens_out_stride < 1) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "tokens_out_stride must be >= 1");
    const beagle_config& c = ctx->cfg;
    bool any_append = false;
    for (int b = 0; b < batch; ++b) {
        const int s = seq_slot[b];
        if (tokens_in_dev == nullptr && !ctx->has_token[s])
            return fail(ctx, BEAGLE_ERR_STATE, "slot %d has no previous draft token; pass tokens_in", s);
        if (concat && ctx->pending[s]) {
            if (ctx->n_draft[s] >= c.max_draft)
                return fail(ctx, BEAGLE_ERR_CAPACITY, "slot %d: draft tail already holds max_draft = %d states", s, c.max_draft);
            any_append = true;
        }
    }
    if (c.rope_theta > 0.f)
        for (int b = 0; b < batch; ++b)
            if (ctx->n_true[seq_slot[b]] + ctx->steps[seq_slot[b]] >= ctx->rope_rows)
                return fail(ctx, BEAGLE_ERR_CAPACITY, "slot %d: position %d exceeds max_ctx + max_draft", seq_slot[b],
                            ctx->n_true[seq_slot[b]] + ctx->steps[seq_slot[b]] + 1);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int dt = c.dtype;
    st = device_setup_once(ctx, stream);
    if (st != BEAGLE_OK) return st;

    BatchMeta meta;
    memset(&meta, 0, sizeof(meta));
    RowMap ident, slots, app_pos;
    memset(&app_pos, 0, sizeof(app_pos));
    int max_kv = 0;
    for (int b = 0; b < kMaxCallBatch; ++b) { ident.idx[b] = b; slots.idx[b] = 0; }
    for (int b = 0; b < batch; ++b) {
        const int s = seq_slot[b];
        const bool app = concat && ctx->pending[s];
        app_pos.idx[b] = app ? ctx->n_true[s] + ctx->n_draft[s] : -1;
        meta.slot[b] = s;
        meta.kv_len[b] = ctx->n_true[s] + ctx->n_draft[s] + (app ? 1 : 0);
        slots.idx[b] = s;
        if (meta.kv_len[b] > max_kv) max_kv = meta.kv_len[b];
    }

    // Batches above 8 rows run their projections on the tensor cores (weights streamed once);
    // smaller ones on the weight-streaming CUDA-core kernel.
    const bool use_tc = ctx->tc != nullptr && batch > kServeTcMinBatch;
    int rc = 0;
#define BEAGLE_SKINNY(MODE, ARGS, WHAT)                                                   \
    do {                                                                                  \
        ARGS.partial = ctx->sk_partial;                                                   \
        ARGS.error_word = ctx->dev_error;                                                 \
        rc = tc_skinny(ctx->tc, MODE, ARGS, stream);                                      \
        if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, WHAT ": unsupported shape");      \
        ctx->launches += rc;                                                              \
    } while (0)

    // (1) x = E[t], xn = RMSNorm(x); the tensor-core path also gathers the slots' previous states
    {
        StageTimer timer_(ctx, ST_EMBED_NORM, stream);
        ctx->launches += launch_embed_norm(dt, tokens_in_dev, ctx->last_token, &meta, ctx->w.embed, c.vocab, nullptr, ctx->w.g_q,
                                           c.hidden, c.rms_eps, c.norm_q, ctx->x, ctx->xn, batch,
                                           (use_tc && any_append) ? ctx->h_slot : nullptr, ctx->hs, stream);
    }
    // (2) + (3) on the tensor-core path: the K/V append and the query projection read different inputs and write different
    // outputs, so they share one launch
    bool merged_qkv = false;
    if (use_tc && any_append) {
        StageTimer timer_(ctx, ST_QKV_PROJ, stream);
        SkinnyArgs q, kv;
        memset(&q, 0, sizeof(q)); memset(&kv, 0, sizeof(kv));
        q.W = ctx->w.w_q; q.N = ctx->qd; q.K = c.hidden; q.X = ctx->xn; q.ldx = c.hidden; q.B = batch;
        q.out = ctx->q; q.ldo = ctx->qd; q.error_word = ctx->dev_error;
        kv.W = ctx->w.w_k; kv.W2 = ctx->w.w_v; kv.N = ctx->kd; kv.K = c.hidden; kv.X = ctx->hs; kv.ldx = c.hidden; kv.B = batch;
        kv.kcache = ctx->kcache; kv.vcache = ctx->vcache; kv.Hkv = c.n_kv_heads; kv.dh = c.head_dim; kv.cap = ctx->cap;
        kv.slot = slots; kv.pos = app_pos;
        rc = tc_skinny_qkv(ctx->tc, q, kv, stream);
        if (rc > 0) { ctx->launches += rc; merged_qkv = true; }
    }
    // (2) concat: K/V of the previous step's state joins the cache tail (Section 4.1, cache paragraph)
    if (any_append && !merged_qkv) {
        StageTimer timer_(ctx, ST_KV_APPEND, stream);
        if (use_tc) {
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_k; a.W2 = ctx->w.w_v; a.N = ctx->kd; a.K = c.hidden; a.X = ctx->hs; a.ldx = c.hidden; a.B = batch;
            a.kcache = ctx->kcache; a.vcache = ctx->vcache; a.Hkv = c.n_kv_heads; a.dh = c.head_dim; a.cap = ctx->cap;
            a.slot = slots; a.pos = app_pos;
            BEAGLE_SKINNY(SK_KV, a, "K/V append");
        } else {
            GemvArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_k; a.W2 = ctx->w.w_v; a.N = ctx->kd; a.K = c.hidden;
            a.X = ctx->h_slot; a.ldx = c.hidden; a.B = batch; a.xrow = slots;
            a.kcache = ctx->kcache; a.vcache = ctx->vcache; a.Hkv = c.n_kv_heads; a.dh = c.head_dim; a.cap = ctx->cap;
            a.orow2 = slots; a.pos = app_pos;
            ctx->launches += launch_gemv(dt, GEMV_KV, a, stream);
        }
    }
    // (3) Q = W_q xn
    if (!merged_qkv) {
        StageTimer timer_(ctx, ST_Q_PROJ, stream);
        if (use_tc) {
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_q; a.N = ctx->qd; a.K = c.hidden; a.X = ctx->xn; a.ldx = c.hidden; a.B = batch;
            a.out = ctx->q; a.ldo = ctx->qd;
            BEAGLE_SKINNY(SK_STORE, a, "Q projection");
        } else {
            GemvArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_q; a.N = ctx->qd; a.K = c.hidden; a.X = ctx->xn; a.ldx = c.hidden; a.B = batch; a.xrow = ident;
            a.out = ctx->q; a.ldo = ctx->qd;
            ctx->launches += launch_gemv(dt, GEMV_STORE, a, stream);
        }
    }
    // (3') rotary option: the s-th step since the reset queries position n + s; the state appended now sits one before it
    if (c.rope_theta > 0.f) {
        StageTimer timer_(ctx, ST_Q_PROJ, stream);
        RowMap qpos, kpos;
        memset(&qpos, 0, sizeof(qpos)); memset(&kpos, 0, sizeof(kpos));
        for (int b = 0; b < batch; ++b) {
            qpos.idx[b] = ctx->n_true[seq_slot[b]] + ctx->steps[seq_slot[b]];
            kpos.idx[b] = qpos.idx[b] > 0 ? qpos.idx[b] - 1 : 0;
        }
        ctx->launches += launch_rope_serve(dt, ctx->q, batch, c.n_q_heads, ctx->kcache, any_append ? batch : 0, c.n_kv_heads, c.head_dim, ctx->cap,
                                           slots, app_pos, qpos, kpos, ctx->rope_table, stream);
    }
    // (4) o = softmax(Q K^T / sqrt(dh)) V over the cache
    {
        StageTimer timer_(ctx, ST_ATTN_DECODE, stream);
        rc = -1;
        if (ctx->tc != nullptr) {       // bf16, head_dim 64 / 128: TMA-staged tiles
            int32_t stable[kMaxCallBatch];
            for (int b = 0; b < batch; ++b) stable[b] = ctx->n_true[seq_slot[b]];
            rc = tc_attn_decode(ctx->tc, ctx->q, meta, stable, batch, c.n_q_heads, c.n_kv_heads, c.head_dim, ctx->cap, max_kv,
                                ctx->attn_scratch, attn_done_counters(ctx), ctx->o, ctx->dev_error, stream);
        }
        if (rc < 0)
            rc = launch_attn_decode(dt, ctx->q, ctx->kcache, ctx->vcache, meta, batch, c.n_q_heads, c.n_kv_heads,
                                    c.head_dim, ctx->cap, max_kv, ctx->attn_scratch, ctx->o, stream);
        if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "attention: unsupported head shape");
        ctx->launches += rc;
    }
    // (5) y = W_o o + x   (6) yn = RMSNorm(y)
    if (use_tc) {
        {
            StageTimer timer_(ctx, ST_O_PROJ, stream);
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_o; a.N = c.hidden; a.K = ctx->qd; a.X = ctx->o; a.ldx = ctx->qd; a.B = batch;
            a.out = ctx->y; a.ldo = c.hidden; a.resid = ctx->x; a.ldr = c.hidden;      // cluster variant: residual added in the reduction
            BEAGLE_SKINNY(SK_RESID, a, "O projection");
        }
        // a row kernel over the 32 x d result is cheaper than a finishing kernel that re-reads all fp32 split partials
        StageTimer timer_(ctx, ST_MLP_NORM, stream);
        ctx->launches += launch_embed_norm(dt, nullptr, nullptr, nullptr, nullptr, 0, ctx->y, ctx->w.g_mlp, c.hidden, c.rms_eps,
                                           c.norm_mlp, nullptr, ctx->yn, batch, nullptr, nullptr, stream);
    } else {
        {
            StageTimer timer_(ctx, ST_O_PROJ, stream);
            GemvArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_o; a.N = c.hidden; a.K = ctx->qd; a.X = ctx->o; a.ldx = ctx->qd; a.B = batch; a.xrow = ident;
            a.out = ctx->y; a.ldo = c.hidden; a.resid = ctx->x; a.ldr = c.hidden;
            ctx->launches += launch_gemv(dt, GEMV_RESID, a, stream);
        }
        StageTimer timer_(ctx, ST_MLP_NORM, stream);
        ctx->launches += launch_embed_norm(dt, nullptr, nullptr, nullptr, nullptr, 0, ctx->y, ctx->w.g_mlp, c.hidden, c.rms_eps,
                                           c.norm_mlp, nullptr, ctx->yn, batch, nullptr, nullptr, stream);
    }
    // (7) act = SiLU(W_gate yn) * (W_up yn)
    {
        StageTimer timer_(ctx, ST_GATE_UP, stream);
        if (use_tc) {
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_gate; a.W2 = ctx->w.w_up; a.N = c.mlp_dim; a.K = c.hidden; a.X = ctx->yn; a.ldx = c.hidden; a.B = batch;
            a.out = ctx->act; a.ldo = c.mlp_dim;
            BEAGLE_SKINNY(SK_SILU_MUL, a, "gate/up projection");
        } else {
            GemvArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_gate; a.W2 = ctx->w.w_up; a.N = c.mlp_dim; a.K = c.hidden; a.X = ctx->yn; a.ldx = c.hidden;
            a.B = batch; a.xrow = ident; a.out = ctx->act; a.ldo = c.mlp_dim;
            ctx->launches += launch_gemv(dt, GEMV_SILU_MUL, a, stream);
        }
    }
    // (8) h = W_down act + y ; kept per slot for the next step's K/V append
    {
        StageTimer timer_(ctx, ST_DOWN, stream);
        if (use_tc) {
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_down; a.N = c.hidden; a.K = c.mlp_dim; a.X = ctx->act; a.ldx = c.mlp_dim; a.B = batch;
            a.out = ctx->h; a.ldo = c.hidden; a.resid = ctx->y; a.ldr = c.hidden;
            a.out2 = ctx->h_slot; a.ld2 = c.hidden; a.orow2 = slots;
            BEAGLE_SKINNY(SK_RESID, a, "down projection");
        } else {
            GemvArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_down; a.N = c.hidden; a.K = c.mlp_dim; a.X = ctx->act; a.ldx = c.mlp_dim; a.B = batch; a.xrow = ident;
            a.out = ctx->h; a.ldo = c.hidden; a.resid = ctx->y; a.ldr = c.hidden;
            a.out2 = ctx->h_slot; a.ld2 = c.hidden; a.orow2 = slots;
            ctx->launches += launch_gemv(dt, GEMV_RESID, a, stream);
        }
    }
    if (hidden_out_dev != nullptr) {
        cudaMemcpyAsync(hidden_out_dev, ctx->h, (size_t)batch * c.hidden * ctx->elt, cudaMemcpyDeviceToDevice, stream);
    }
    // (9) z = W_lm h, greedy token
    {
        int nblk = ctx->lm_blocks;
        {
            StageTimer timer_(ctx, ST_LM_HEAD, stream);
            if (use_tc) {
                SkinnyArgs a;
                memset(&a, 0, sizeof(a));
                a.W = ctx->w.w_lm; a.N = c.vocab; a.K = c.hidden; a.X = ctx->h; a.ldx = c.hidden; a.B = batch;
                a.logits = logits_out_dev; a.keys = ctx->lm_partials;
                if (ctx->w.w_lm_fp8 != nullptr) {       // optional FP8 LM head: quantise this step's states, stream the byte weights
                    rc = launch_quantize_rows_e4m3(dt, ctx->h, batch, c.hidden, ctx->hq, ctx->hscale, stream);
                    if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "FP8 LM head: hidden must be a multiple of 8");
                    ctx->launches += rc;
                    a.W8 = ctx->w.w_lm_fp8; a.w_scale = ctx->w.w_lm_scale; a.X8 = ctx->hq; a.x_scale = ctx->hscale;
                }
                BEAGLE_SKINNY(SK_LOGITS, a, "LM head");
                nblk = tc_skinny_key_tiles(c.vocab);
            } else {
                GemvArgs a;
                memset(&a, 0, sizeof(a));
                a.W = ctx->w.w_lm; a.N = c.vocab; a.K = c.hidden; a.X = ctx->h; a.ldx = c.hidden; a.B = batch; a.xrow = ident;
                a.logits = logits_out_dev; a.partials = ctx->lm_partials;
                ctx->launches += launch_gemv(dt, GEMV_LOGITS, a, stream);
            }
        }
        StageTimer timer_(ctx, ST_ARGMAX, stream);
        ctx->launches += launch_argmax_finalize(ctx->lm_partials, nblk, meta, batch, tokens_out_dev, tokens_out_stride, ctx->last_token, stream);
    }
#undef BEAGLE_SKINNY
    st = cuda_ok(ctx, "draft_step");
    if (st != BEAGLE_OK) return st;
    for (int b = 0; b < batch; ++b) {
        const int s = seq_slot[b];
        if (concat && ctx->pending[s]) ctx->n_draft[s] += 1;
        ctx->pending[s] = 1;
        ctx->has_token[s] = 1;
        ctx->steps[s] += 1;
    }
    return BEAGLE_OK;
}

beagle_status beagle_quantize_rows_e4m3(const void* src_dev, int32_t dtype, int64_t rows, int32_t cols, void* q_out_dev,
                                        float* scale_out_dev, void* stream_) {
    if (src_dev == nullptr || q_out_dev == nullptr || scale_out_dev == nullptr || rows < 0 || cols <= 0) return BEAGLE_ERR_INVALID_ARG;
    if (dtype != BEAGLE_FP32 && dtype != BEAGLE_BF16) return BEAGLE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(src_dev) & 15) || (reinterpret_cast<uintptr_t>(q_out_dev) & 7)) return BEAGLE_ERR_INVALID_ARG;
    if (launch_quantize_rows_e4m3(dtype, src_dev, rows, cols, q_out_dev, scale_out_dev, static_cast<cudaStream_t>(stream_)) < 0)
        return BEAGLE_ERR_SHAPE;
    return cudaGetLastError() == cudaSuccess ? BEAGLE_OK : BEAGLE_ERR_CUDA;
}

beagle_status beagle_block_workspace_bytes(const beagle_config* cfg, int32_t batch, int32_t S, size_t* bytes) {
    const beagle_status st = check_config(cfg);
    if (st != BEAGLE_OK) return st;
    if (bytes == nullptr || batch <= 0 || S <= 0) return BEAGLE_ERR_INVALID_ARG;
    if ((long long)batch * S > (1ll << 24)) return BEAGLE_ERR_CAPACITY;
    *bytes = block_layout(*cfg, batch, S).total;
    return BEAGLE_OK;
}

struct LossSpec {                  // beagle_block_loss: what replaces the LM head's outputs
    int stage;                     // 0 early (Eq. 4), 1 late (Eq. 7)
    const void* tgt; int tgt_dtype;
    const int32_t* labels;
    float* loss_out; float* ce_out;
    void* gate; void* up;          // training step: the final pass keeps W_gate n and W_up n (NULL: fused SiLU-mul GEMM)
    float* row_stats;              // training step: every row's merged softmax statistics (4 floats), or NULL
    float* lse2;                   // training step: the attention rows' base-2 log-sum-exp (tensor-core attention only), or NULL
    bool lse2_written;             // set when the last pass ran the tensor-core attention and filled lse2
};

static beagle_status block_forward_impl(beagle_ctx* ctx, int32_t batch, int32_t S, const int32_t* tokens_dev,
                                        const void* hidden_dev, int32_t block, int32_t offset, int32_t sim_steps,
                                        float* logits_out_dev, int32_t* argmax_out_dev, void* hidden_out_dev,
                                        void* ws_dev, size_t ws_bytes, void* stream_, LossSpec* loss) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    if (batch <= 0 || S <= 0 || tokens_dev == nullptr || hidden_dev == nullptr || ws_dev == nullptr)
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_forward: NULL or empty argument");
    if ((long long)batch * S > (1ll << 24)) return fail(ctx, BEAGLE_ERR_CAPACITY, "block_forward: too many positions");
    if (block < 1 || offset < 0 || offset >= S || sim_steps < 1 || sim_steps > block)
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_forward: need block >= 1, 0 <= offset < S, 1 <= sim_steps <= block");
    if (ctx->cfg.head_dim % 32) return fail(ctx, BEAGLE_ERR_SHAPE, "block_forward: head_dim must be a multiple of 32");
    if (reinterpret_cast<uintptr_t>(ws_dev) & (kAlign - 1)) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    if ((reinterpret_cast<uintptr_t>(hidden_dev) & 15) || (hidden_out_dev && (reinterpret_cast<uintptr_t>(hidden_out_dev) & 15)))
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "hidden buffers must be 16-byte aligned");
    const beagle_config& c = ctx->cfg;
    const BlockLayout L = block_layout(c, batch, S);
    if (ws_bytes < L.total) return fail(ctx, BEAGLE_ERR_CAPACITY, "block_forward: workspace %zu < %zu bytes", ws_bytes, L.total);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    {
        const beagle_status st0 = device_setup_once(ctx, stream);
        if (st0 != BEAGLE_OK) return st0;
    }
    char* ws = static_cast<char*>(ws_dev);
    const int dt = c.dtype;
    const int M = batch * S;
    void *X = ws + L.x, *Xn = ws + L.xn, *Q = ws + L.q, *Kt = ws + L.kt, *Vt = ws + L.vt, *Kp = ws + L.kp, *Vp = ws + L.vp;
    void *O = ws + L.o, *Y = ws + L.y, *Yn = ws + L.yn, *ACT = ws + L.act;
    void* H = hidden_out_dev != nullptr ? hidden_out_dev : (void*)(ws + L.h);
    int rc;
#define BEAGLE_GEMM(STAGE, EPI, ARGS, WHAT)                                            \
    do {                                                                               \
        StageTimer timer_(ctx, STAGE, stream);                                         \
        rc = dense_gemm(ctx, EPI, ARGS, stream);                                       \
        if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, WHAT ": unsupported shape");   \
        ctx->launches += rc;                                                           \
    } while (0)

    // queries: every position's data token (Section 4.2: no new queries are generated)
    {
        StageTimer timer_(ctx, ST_BLK_EMBED, stream);
        ctx->launches += launch_embed_norm(dt, tokens_dev, nullptr, nullptr, ctx->w.embed, c.vocab, nullptr,
                                           ctx->w.g_q, c.hidden, c.rms_eps, c.norm_q, X, Xn, M, nullptr, nullptr, stream);
    }
    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.M = M;
    g.A = Xn; g.lda = c.hidden; g.K = c.hidden; g.W = ctx->w.w_q; g.N = ctx->qd; g.C = Q; g.ldc = ctx->qd;
    BEAGLE_GEMM(ST_BLK_QKV, GEMM_STORE, g, "Q projection");
    // keys / values of the true states
    g.A = hidden_dev; g.W = ctx->w.w_k; g.N = ctx->kd; g.C = Kt; g.ldc = ctx->kd;
    BEAGLE_GEMM(ST_BLK_QKV, GEMM_STORE, g, "K projection");
    g.W = ctx->w.w_v; g.C = Vt;
    BEAGLE_GEMM(ST_BLK_QKV, GEMM_STORE, g, "V projection");
    // rotary option: position p - 1 for the query of position p and for the key of the state at position p
    float* rope = reinterpret_cast<float*>(ws + L.rope);
    if (c.rope_theta > 0.f) {
        StageTimer timer_(ctx, ST_BLK_QKV, stream);
        ctx->launches += launch_rope_table(c.rope_theta, c.head_dim, S, rope, stream);
        ctx->launches += launch_rope_rows(dt, Q, M, c.n_q_heads, c.head_dim, S, 0, 0, rope, stream);
        ctx->launches += launch_rope_rows(dt, Kt, M, c.n_kv_heads, c.head_dim, S, 0, 0, rope, stream);
    }

    for (int step = 1; step <= sim_steps; ++step) {
        if (step > 1) {
            // the states predicted so far become keys / values at their own positions (in place)
            memset(&g, 0, sizeof(g));
            g.M = M; g.A = H; g.lda = c.hidden; g.K = c.hidden; g.N = ctx->kd; g.ldc = ctx->kd;
            g.W = ctx->w.w_k; g.C = Kp;
            BEAGLE_GEMM(ST_BLK_PRED_KV, GEMM_STORE, g, "predicted K projection");
            g.W = ctx->w.w_v; g.C = Vp;
            BEAGLE_GEMM(ST_BLK_PRED_KV, GEMM_STORE, g, "predicted V projection");
            if (c.rope_theta > 0.f) ctx->launches += launch_rope_rows(dt, Kp, M, c.n_kv_heads, c.head_dim, S, 0, 0, rope, stream);
        }
        {
            StageTimer timer_(ctx, ST_BLK_ATTN, stream);
            rc = -1;
            if (ctx->tc != nullptr) {       // bf16, head_dim 64 / 128: tensor-core tiles
                    float* lse2 = (loss != nullptr && step == sim_steps) ? loss->lse2 : nullptr;
                if (c.head_dim == 64 || c.head_dim == 128) {
                    // tcgen05 path: the values are read as they lie (MN-major operand of P V)
                    rc = tc_attn_block_umma(ctx->tc, Q, Kt, Vt, Kp, step > 1 ? Vp : Vt, batch, S, c.n_q_heads, c.n_kv_heads, c.head_dim,
                                            block, offset, step, O, ctx->dev_error, stream, lse2);
                }
                if (rc >= 0 && lse2 != nullptr) loss->lse2_written = true;
            }
            if (rc < 0)
                rc = launch_attn_block(dt, Q, Kt, Vt, Kp, Vp, batch, S, c.n_q_heads, c.n_kv_heads, c.head_dim, block, offset, step, O, stream);
            if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "block attention: unsupported head_dim");
            ctx->launches += rc;
        }
        memset(&g, 0, sizeof(g));
        g.M = M; g.A = O; g.lda = ctx->qd; g.K = ctx->qd; g.W = ctx->w.w_o; g.N = c.hidden; g.C = Y; g.ldc = c.hidden;
        g.R = X; g.ldr = c.hidden;
        BEAGLE_GEMM(ST_BLK_O, GEMM_RESID, g, "O projection");
        {
            StageTimer timer_(ctx, ST_BLK_NORM, stream);
            ctx->launches += launch_embed_norm(dt, nullptr, nullptr, nullptr, nullptr, 0, Y, ctx->w.g_mlp, c.hidden, c.rms_eps,
                                               c.norm_mlp, nullptr, Yn, M, nullptr, nullptr, stream);
        }
        memset(&g, 0, sizeof(g));
        g.M = M; g.A = Yn; g.lda = c.hidden; g.K = c.hidden; g.W = ctx->w.w_gate; g.W2 = ctx->w.w_up; g.N = c.mlp_dim;
        g.C = ACT; g.ldc = c.mlp_dim;
        if (loss != nullptr && loss->gate != nullptr && step == sim_steps) {
            g.W2 = nullptr; g.C = loss->gate;
            BEAGLE_GEMM(ST_BLK_GATE_UP, GEMM_STORE, g, "gate projection");
            g.W = ctx->w.w_up; g.C = loss->up;
            BEAGLE_GEMM(ST_BLK_GATE_UP, GEMM_STORE, g, "up projection");
            ctx->launches += launch_silu_mul(dt, loss->gate, loss->up, ACT, (size_t)M * c.mlp_dim, stream);
        } else {
            BEAGLE_GEMM(ST_BLK_GATE_UP, GEMM_SILU_MUL, g, "gate/up projection");
        }
        memset(&g, 0, sizeof(g));
        g.M = M; g.A = ACT; g.lda = c.mlp_dim; g.K = c.mlp_dim; g.W = ctx->w.w_down; g.N = c.hidden; g.C = H; g.ldc = c.hidden;
        g.R = Y; g.ldr = c.hidden;
        BEAGLE_GEMM(ST_BLK_DOWN, GEMM_RESID, g, "down projection");
    }

    // loss forward: cross-entropy partials straight from the LM-head GEMM, merged, weighted and reduced
    if (loss != nullptr) {
        float* part = reinterpret_cast<float*>(ws + L.ce_part);
        int ntiles = 1;
        if (ctx->tc != nullptr) {
            memset(&g, 0, sizeof(g));
            g.M = M; g.A = H; g.lda = c.hidden; g.K = c.hidden; g.W = ctx->w.w_lm; g.N = c.vocab;
            g.tgt = loss->tgt; g.tgt_dtype = loss->tgt_dtype; g.ldt = c.vocab; g.labels = loss->labels; g.ce_part = part;
            BEAGLE_GEMM(ST_BLK_LM_HEAD, GEMM_CE, g, "LM head (loss)");
            ntiles = tc_argmax_tiles(c.vocab);
        } else {
            float* chunk = reinterpret_cast<float*>(ws + L.logits);
            const size_t trow = (size_t)c.vocab * (loss->tgt_dtype == BEAGLE_BF16 ? 2 : 4);
            for (int r0 = 0; r0 < M; r0 += L.lm_chunk_rows) {
                const int rows = M - r0 < L.lm_chunk_rows ? M - r0 : L.lm_chunk_rows;
                memset(&g, 0, sizeof(g));
                g.M = rows; g.A = static_cast<const char*>(H) + (size_t)r0 * c.hidden * ctx->elt; g.lda = c.hidden; g.K = c.hidden;
                g.W = ctx->w.w_lm; g.N = c.vocab; g.C = chunk; g.ldc = c.vocab;
                BEAGLE_GEMM(ST_BLK_LM_HEAD, GEMM_F32, g, "LM head");
                ctx->launches += launch_row_ce(chunk, rows, c.vocab,
                                               loss->tgt != nullptr ? static_cast<const char*>(loss->tgt) + (size_t)r0 * trow : nullptr,
                                               loss->tgt_dtype, loss->labels != nullptr ? loss->labels + r0 : nullptr,
                                               part + (size_t)r0 * kCeFields, stream);
            }
        }
        StageTimer timer_(ctx, ST_BLK_ARGMAX, stream);
        ctx->launches += launch_ce_finalize(part, ntiles, batch, S, block, offset, sim_steps, loss->stage,
                                            reinterpret_cast<float*>(ws + L.ce_rows), reinterpret_cast<float*>(ws + L.wce), loss->ce_out,
                                            loss->loss_out, stream, loss->row_stats);
    }
    // LM head at every position
    if (loss == nullptr && (logits_out_dev != nullptr || argmax_out_dev != nullptr)) {
        unsigned long long* keys = reinterpret_cast<unsigned long long*>(ws + L.keys);
        int32_t* ids = argmax_out_dev != nullptr ? argmax_out_dev : reinterpret_cast<int32_t*>(ws + L.ids);
        if (logits_out_dev != nullptr) {
            memset(&g, 0, sizeof(g));
            g.M = M; g.A = H; g.lda = c.hidden; g.K = c.hidden; g.W = ctx->w.w_lm; g.N = c.vocab; g.C = logits_out_dev; g.ldc = c.vocab;
            BEAGLE_GEMM(ST_BLK_LM_HEAD, GEMM_F32, g, "LM head");
            if (argmax_out_dev != nullptr) {
                StageTimer timer_(ctx, ST_BLK_ARGMAX, stream);
                ctx->launches += launch_row_argmax(0, logits_out_dev, M, c.vocab, keys, ids, stream);
            }
        } else if (ctx->tc != nullptr) {
            // arg-max only: the LM-head GEMM emits one packed key per (row, column tile); no logits are written
            memset(&g, 0, sizeof(g));
            g.M = M; g.A = H; g.lda = c.hidden; g.K = c.hidden; g.W = ctx->w.w_lm; g.N = c.vocab; g.keys = keys;
            BEAGLE_GEMM(ST_BLK_LM_HEAD, GEMM_ARGMAX_KEYS, g, "LM head");
            StageTimer timer_(ctx, ST_BLK_ARGMAX, stream);
            ctx->launches += tc_keys_to_ids(keys, M, tc_argmax_tiles(c.vocab), ids, stream);
        } else {
            float* chunk = reinterpret_cast<float*>(ws + L.logits);
            for (int r0 = 0; r0 < M; r0 += L.lm_chunk_rows) {
                const int rows = M - r0 < L.lm_chunk_rows ? M - r0 : L.lm_chunk_rows;
                memset(&g, 0, sizeof(g));
                g.M = rows; g.A = static_cast<const char*>(H) + (size_t)r0 * c.hidden * ctx->elt; g.lda = c.hidden; g.K = c.hidden;
                g.W = ctx->w.w_lm; g.N = c.vocab; g.C = chunk; g.ldc = c.vocab;
                BEAGLE_GEMM(ST_BLK_LM_HEAD, GEMM_F32, g, "LM head");
                StageTimer timer_(ctx, ST_BLK_ARGMAX, stream);
                ctx->launches += launch_row_argmax(0, chunk, rows, c.vocab, keys + (size_t)r0 * kRowArgmaxSplit, ids + r0, stream);
            }
        }
    }
#undef BEAGLE_GEMM
    return cuda_ok(ctx, "block_forward");
}

beagle_status beagle_block_forward(beagle_ctx* ctx, int32_t batch, int32_t S, const int32_t* tokens_dev,
                                   const void* hidden_dev, int32_t block, int32_t offset, int32_t sim_steps,
                                   float* logits_out_dev, int32_t* argmax_out_dev, void* hidden_out_dev,
                                   void* ws_dev, size_t ws_bytes, void* stream_) {
    return block_forward_impl(ctx, batch, S, tokens_dev, hidden_dev, block, offset, sim_steps, logits_out_dev, argmax_out_dev,
                              hidden_out_dev, ws_dev, ws_bytes, stream_, nullptr);
}

beagle_status beagle_block_loss(beagle_ctx* ctx, int32_t batch, int32_t S, const int32_t* tokens_dev, const void* hidden_dev,
                                int32_t block, int32_t offset, int32_t sim_steps, int32_t stage, const void* target_logits_dev,
                                int32_t logits_dtype, const int32_t* target_ids_dev, float* loss_out_dev, float* ce_out_dev,
                                void* ws_dev, size_t ws_bytes, void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    if (stage != 0 && stage != 1) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_loss: stage must be 0 (early) or 1 (late)");
    if (stage == 0 && sim_steps != 1) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_loss: the early-stage loss uses sim_steps = 1");
    if ((target_logits_dev == nullptr) == (target_ids_dev == nullptr))
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_loss: give exactly one of target_logits / target_ids");
    if (target_logits_dev != nullptr && logits_dtype != BEAGLE_FP32 && logits_dtype != BEAGLE_BF16)
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_loss: unknown logits_dtype");
    if (loss_out_dev == nullptr) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_loss: loss_out is NULL");
    LossSpec spec;
    spec.stage = stage; spec.tgt = target_logits_dev; spec.tgt_dtype = target_logits_dev != nullptr ? logits_dtype : 0;
    spec.labels = target_ids_dev; spec.loss_out = loss_out_dev; spec.ce_out = ce_out_dev;
    spec.gate = nullptr; spec.up = nullptr; spec.row_stats = nullptr; spec.lse2 = nullptr; spec.lse2_written = false;
    return block_forward_impl(ctx, batch, S, tokens_dev, hidden_dev, block, offset, sim_steps, nullptr, nullptr, nullptr, ws_dev,
                              ws_bytes, stream_, &spec);
}

beagle_status beagle_block_grad_workspace_bytes(const beagle_config* cfg, int32_t batch, int32_t S, size_t* bytes) {
    const beagle_status st = check_config(cfg);
    if (st != BEAGLE_OK) return st;
    if (bytes == nullptr || batch <= 0 || S <= 0) return BEAGLE_ERR_INVALID_ARG;
    if ((long long)batch * S > (1ll << 24)) return BEAGLE_ERR_CAPACITY;
    *bytes = grad_layout(*cfg, batch, S).total;
    return BEAGLE_OK;
}

beagle_status beagle_block_grad(beagle_ctx* ctx, int32_t batch, int32_t S, const int32_t* tokens_dev, const void* hidden_dev,
                                int32_t block, int32_t offset, int32_t sim_steps, int32_t stage, const void* target_logits_dev,
                                int32_t logits_dtype, const int32_t* target_ids_dev, float vloss_coef, const beagle_grads* grads,
                                float* loss_out_dev, void* ws_dev, size_t ws_bytes, void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    if (grads == nullptr || loss_out_dev == nullptr) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_grad: grads / loss_out is NULL");
    if (batch <= 0 || S <= 0) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_grad: empty batch");
    if ((long long)batch * S > (1ll << 24)) return fail(ctx, BEAGLE_ERR_CAPACITY, "block_grad: too many positions");
    if (stage != 0 && stage != 1) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_grad: stage must be 0 (early) or 1 (late)");
    if (stage == 0 && sim_steps != 1) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_grad: the early-stage loss uses sim_steps = 1");
    if ((target_logits_dev == nullptr) == (target_ids_dev == nullptr))
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_grad: give exactly one of target_logits / target_ids");
    if (target_logits_dev != nullptr && logits_dtype != BEAGLE_FP32 && logits_dtype != BEAGLE_BF16)
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_grad: unknown logits_dtype");
    if (!(vloss_coef >= 0.f)) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "block_grad: vloss_coef must be >= 0");
    const beagle_config& c = ctx->cfg;
    if (c.hidden % 8 || c.mlp_dim % 8 || c.head_dim % 8) return fail(ctx, BEAGLE_ERR_SHAPE, "block_grad: hidden, mlp_dim and head_dim must be multiples of 8");
    const GradLayout L = grad_layout(c, batch, S);
    if (ws_dev == nullptr || ws_bytes < L.total) return fail(ctx, BEAGLE_ERR_CAPACITY, "block_grad: workspace %zu < %zu bytes", ws_bytes, L.total);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    char* ws = static_cast<char*>(ws_dev);
    const int dt = c.dtype;
    const int M = batch * S, Mp = L.Mp, Vp = L.Vp;
    const int d = c.hidden, qd = ctx->qd, kd = ctx->kd, m = c.mlp_dim, V = c.vocab;

    // ---- forward of the training step: keeps every activation, W_gate n and W_up n, and the rows' softmax statistics
    LossSpec spec;
    spec.stage = stage; spec.tgt = target_logits_dev; spec.tgt_dtype = target_logits_dev != nullptr ? logits_dtype : 0;
    spec.labels = target_ids_dev; spec.loss_out = loss_out_dev; spec.ce_out = nullptr;
    spec.gate = ws + L.gate; spec.up = ws + L.up; spec.row_stats = reinterpret_cast<float*>(ws + L.stats);
    spec.lse2 = reinterpret_cast<float*>(ws + L.lse); spec.lse2_written = false;
    beagle_status st = block_forward_impl(ctx, batch, S, tokens_dev, hidden_dev, block, offset, sim_steps, nullptr, nullptr, nullptr, ws_dev,
                                          ws_bytes, stream_, &spec);
    if (st != BEAGLE_OK) return st;

    const BlockLayout& F = L.fwd;
    void *X = ws + F.x, *Xn = ws + F.xn, *Q = ws + F.q, *Kt = ws + F.kt, *Vt = ws + F.vt, *Kp = ws + F.kp, *Vp_ = ws + F.vp;
    void *O = ws + F.o, *Y = ws + F.y, *Yn = ws + F.yn, *ACT = ws + F.act, *H = ws + F.h;
    void *G = ws + L.gate, *U = ws + L.up, *DACT = ws + L.dact, *DZ = ws + L.dz, *DH0 = ws + L.dh0, *DH = ws + L.dh, *DYN = ws + L.dyn;
    void *DY = ws + L.dy, *DO = ws + L.d_o, *DQ = ws + L.dq, *DKT = ws + L.dkt, *DVT = ws + L.dvt, *DKP = ws + L.dkp, *DVP = ws + L.dvp;
    void *DXN = ws + L.dxn, *TA = ws + L.ta, *TB = ws + L.tb, *WT = ws + L.wt;
    float* dgpart = reinterpret_cast<float*>(ws + L.dgpart);
    int rc;
    GemmArgs g;
#define BEAGLE_BWD_GEMM(STAGE, EPI, WHAT)                                              \
    do {                                                                               \
        StageTimer timer_(ctx, STAGE, stream);                                         \
        rc = dense_gemm(ctx, EPI, g, stream);                                          \
        if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, WHAT ": unsupported shape");   \
        ctx->launches += rc;                                                           \
    } while (0)
    auto transpose = [&](const void* in, int rows, int cols, int ld_in, void* out, int ld_out, int col0, int rows_pad) {
        StageTimer timer_(ctx, ST_BWD_TRANSPOSE, stream);
        ctx->launches += launch_transpose_pad(dt, in, rows, cols, ld_in, out, ld_out, col0, rows_pad, stream);
    };
    // dX = dY W: A = dY [M, n_out_pad], "weight" = W^T [n_in, n_out_pad] (transposed here, padded columns zero)
    auto dx_gemm = [&](int epi, const void* dYm, int ldy, const void* W, int n_out, int n_in, void* out, const void* resid) -> int {
        if (ctx->tc != nullptr) {
            // tensor cores: the weight [n_out, n_in] is read as it lies, as an MN-major operand (no transposed copy)
            memset(&g, 0, sizeof(g));
            g.M = M; g.A = dYm; g.lda = ldy; g.K = n_out; g.W = W; g.ldw = n_in; g.b_mn = 1; g.N = n_in; g.C = out; g.ldc = n_in;
            g.R = resid; g.ldr = n_in;
            StageTimer timer_(ctx, ST_BWD_DX, stream);
            const int r = dense_gemm(ctx, epi, g, stream);
            if (r > 0) { ctx->launches += r; return r; }
        }
        const int np = (n_out + 7) / 8 * 8;
        transpose(W, n_out, n_in, n_in, WT, np, 0, np);
        memset(&g, 0, sizeof(g));
        g.M = M; g.A = dYm; g.lda = ldy; g.K = np; g.W = WT; g.N = n_in; g.C = out; g.ldc = n_in; g.R = resid; g.ldr = n_in;
        g.w_transient = 1;
        StageTimer timer_(ctx, ST_BWD_DX, stream);
        const int r = dense_gemm(ctx, epi, g, stream);
        if (r > 0) ctx->launches += r;
        return r;
    };
    // dW = dY^T X: A = dY^T [n_out, K], "weight" = X^T [n_in, K], K = Mp (or 2 Mp with two row blocks side by side), fp32 out
    // dW = dY^T X on the tensor cores without transposed copies: both operands MN-major, contraction over the M rows
    auto dw_gemm_mn = [&](const void* dYm, int ldy, int n_out, const void* Xm, int ldx, int n_in, float* out) -> int {
        if (ctx->tc == nullptr) return -1;
        memset(&g, 0, sizeof(g));
        g.M = n_out; g.A = dYm; g.lda = ldy; g.a_mn = 1; g.K = M; g.W = Xm; g.ldw = ldx; g.b_mn = 1; g.N = n_in; g.C = out; g.ldc = n_in;
        StageTimer timer_(ctx, ST_BWD_DW, stream);
        const int r = dense_gemm(ctx, GEMM_F32, g, stream);
        if (r > 0) ctx->launches += r;
        return r;
    };
    auto dw_gemm = [&](int n_out, int n_in, int Kc, float* out) -> int {
        memset(&g, 0, sizeof(g));
        g.M = n_out; g.A = TA; g.lda = Kc; g.K = Kc; g.W = TB; g.N = n_in; g.C = out; g.ldc = n_in; g.w_transient = 1;
        StageTimer timer_(ctx, ST_BWD_DW, stream);
        const int r = dense_gemm(ctx, GEMM_F32, g, stream);
        if (r > 0) ctx->launches += r;
        return r;
    };
#define BEAGLE_NEED(EXPR, WHAT) do { if ((EXPR) < 0) return fail(ctx, BEAGLE_ERR_SHAPE, WHAT ": unsupported shape"); } while (0)

    // ---- d z = weight * (softmax(z) - p) / (batch * windows), from re-materialised logits, chunk by chunk
    const int windows = (S - offset + block - 1) / block;
    const float ce_scale = 1.0f / ((float)batch * (float)windows);
    bool dz_done = false;
    if (ctx->tc != nullptr) {      // fused: the LM-head GEMM is run again and its epilogue turns the logits into d z
        float* coef = reinterpret_cast<float*>(ws + L.coef);
        StageTimer timer_(ctx, ST_BWD_DLOGITS, stream);
        ctx->launches += launch_loss_coef(M, S, block, offset, sim_steps, stage, ce_scale, coef, stream);
        memset(&g, 0, sizeof(g));
        g.M = M; g.A = H; g.lda = d; g.K = d; g.W = ctx->w.w_lm; g.N = V; g.C = DZ; g.ldc = Vp;
        g.tgt = target_logits_dev; g.tgt_dtype = spec.tgt_dtype; g.ldt = V; g.labels = target_ids_dev;
        g.row_stats = reinterpret_cast<const float*>(ws + L.stats); g.row_coef = coef;
        rc = dense_gemm(ctx, GEMM_DLOGITS, g, stream);
        if (rc > 0) { ctx->launches += rc; dz_done = true; }
    }
    if (!dz_done) {
        float* chunk = reinterpret_cast<float*>(ws + F.logits);
        for (int r0 = 0; r0 < M; r0 += F.lm_chunk_rows) {
            const int rows = M - r0 < F.lm_chunk_rows ? M - r0 : F.lm_chunk_rows;
            memset(&g, 0, sizeof(g));
            g.M = rows; g.A = static_cast<const char*>(H) + (size_t)r0 * d * ctx->elt; g.lda = d; g.K = d;
            g.W = ctx->w.w_lm; g.N = V; g.C = chunk; g.ldc = V;
            BEAGLE_BWD_GEMM(ST_BWD_DLOGITS, GEMM_F32, "LM head (backward)");
            StageTimer timer_(ctx, ST_BWD_DLOGITS, stream);
            ctx->launches += launch_dlogits(dt, chunk, rows, V, target_logits_dev, spec.tgt_dtype, target_ids_dev,
                                            reinterpret_cast<const float*>(ws + L.stats), r0, S, block, offset, sim_steps, stage, ce_scale, DZ, Vp,
                                            stream);
        }
    }
    // ---- regression term (Appendix B): value and its gradient in h
    {
        int reg_rows = 0;      // positions with a loss term, per sequence
        for (int p = offset + 1; p <= S; ++p) {
            const int slot = p - (offset + block * ((p - 1 - offset) / block));
            if (stage == 0 || slot <= sim_steps) ++reg_rows;
        }
        const float n_reg = (float)batch * (float)reg_rows * (float)d;
        const float vscale = reg_rows > 0 ? 1.0f / n_reg : 0.f;
        StageTimer timer_(ctx, ST_BWD_ELEMENTWISE, stream);
        ctx->launches += launch_vloss(dt, H, hidden_dev, M, d, S, block, offset, sim_steps, stage, vloss_coef * vscale, vscale, vloss_coef, DH0,
                                      reinterpret_cast<float*>(ws + L.vrow), loss_out_dev, stream);
    }
    // ---- LM head: dh = dz W_lm + dh0;  dW_lm = dz^T h
    BEAGLE_NEED(dx_gemm(GEMM_RESID, DZ, Vp, ctx->w.w_lm, V, d, DH, DH0), "dh");
    if (grads->w_lm != nullptr && dw_gemm_mn(DZ, Vp, V, H, d, d, grads->w_lm) < 0) {
        transpose(DZ, M, V, Vp, TA, Mp, 0, Mp);
        transpose(H, M, d, d, TB, Mp, 0, Mp);
        BEAGLE_NEED(dw_gemm(V, d, Mp, grads->w_lm), "dW_lm");
    }
    // ---- MLP: h = y + W_down act
    BEAGLE_NEED(dx_gemm(GEMM_STORE, DH, d, ctx->w.w_down, d, m, DACT, nullptr), "dact");
    if (grads->w_down != nullptr && dw_gemm_mn(DH, d, d, ACT, m, m, grads->w_down) < 0) {
        transpose(DH, M, d, d, TA, Mp, 0, Mp);
        transpose(ACT, M, m, m, TB, Mp, 0, Mp);
        BEAGLE_NEED(dw_gemm(d, m, Mp, grads->w_down), "dW_down");
    }
    {
        StageTimer timer_(ctx, ST_BWD_ELEMENTWISE, stream);
        ctx->launches += launch_silu_mul_bwd(dt, G, U, DACT, (size_t)M * m, stream);     // G <- d gate, U <- d up
    }
    BEAGLE_NEED(dx_gemm(GEMM_STORE, G, m, ctx->w.w_gate, m, d, DYN, nullptr), "dyn (gate)");
    BEAGLE_NEED(dx_gemm(GEMM_RESID, U, m, ctx->w.w_up, m, d, DYN, DYN), "dyn (up)");
    if (grads->w_gate != nullptr || grads->w_up != nullptr) {
        bool yn_t = false;          // Yn^T made (only the path with transposed copies needs it)
        if (grads->w_gate != nullptr && dw_gemm_mn(G, m, m, Yn, d, d, grads->w_gate) < 0) {
            transpose(Yn, M, d, d, TB, Mp, 0, Mp);
            yn_t = true;
            transpose(G, M, m, m, TA, Mp, 0, Mp);
            BEAGLE_NEED(dw_gemm(m, d, Mp, grads->w_gate), "dW_gate");
        }
        if (grads->w_up != nullptr && dw_gemm_mn(U, m, m, Yn, d, d, grads->w_up) < 0) {
            if (!yn_t) transpose(Yn, M, d, d, TB, Mp, 0, Mp);
            transpose(U, M, m, m, TA, Mp, 0, Mp);
            BEAGLE_NEED(dw_gemm(m, d, Mp, grads->w_up), "dW_up");
        }
    }
    {   // dy = dh + RMSNorm backward of dyn
        StageTimer timer_(ctx, ST_BWD_ELEMENTWISE, stream);
        rc = launch_rmsnorm_bwd(dt, Y, ctx->w.g_mlp, DYN, DH, M, d, c.rms_eps, c.norm_mlp, DY, dgpart, grads->g_mlp, stream);
        if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "block_grad: hidden too large for the RMSNorm backward");
        ctx->launches += rc;
    }
    // ---- output projection: y = W_O o + x
    BEAGLE_NEED(dx_gemm(GEMM_STORE, DY, d, ctx->w.w_o, d, qd, DO, nullptr), "do");
    if (grads->w_o != nullptr && dw_gemm_mn(DY, d, d, O, qd, qd, grads->w_o) < 0) {
        transpose(DY, M, d, d, TA, Mp, 0, Mp);
        transpose(O, M, qd, qd, TB, Mp, 0, Mp);
        BEAGLE_NEED(dw_gemm(d, qd, Mp, grads->w_o), "dW_o");
    }
    // ---- attention
    {
        StageTimer timer_(ctx, ST_BWD_ATTN, stream);
        rc = -1;
        if (spec.lse2_written) {     // bf16, head_dim 64 / 128: tcgen05, from the forward's log-sum-exp
            rc = tc_attn_block_bwd_umma(ctx->tc, Q, Kt, Vt, Kp, Vp_, O, DO, spec.lse2, batch, S,
                                        c.n_q_heads, c.n_kv_heads, c.head_dim, block, offset, sim_steps, reinterpret_cast<float*>(ws + L.delta), DQ,
                                        DKT, DVT, DKP, DVP, ctx->dev_error, stream);
        }
        if (rc < 0)
            rc = launch_attn_block_bwd(dt, Q, Kt, Vt, Kp, Vp_, DO, batch, S, c.n_q_heads, c.n_kv_heads, c.head_dim, block, offset, sim_steps, DQ,
                                       DKT, DVT, DKP, DVP, reinterpret_cast<float*>(ws + L.lse), reinterpret_cast<float*>(ws + L.delta), stream);
        if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "block_grad: unsupported head_dim");
        ctx->launches += rc;
    }
    if (c.rope_theta > 0.f) {      // back through the rotations: the transpose of a rotation is the opposite angle
        StageTimer timer_(ctx, ST_BWD_ELEMENTWISE, stream);
        const float* rope = reinterpret_cast<const float*>(ws + F.rope);
        ctx->launches += launch_rope_rows(dt, DQ, M, c.n_q_heads, c.head_dim, S, 0, 1, rope, stream);
        ctx->launches += launch_rope_rows(dt, DKT, M, c.n_kv_heads, c.head_dim, S, 0, 1, rope, stream);
        if (sim_steps > 1) ctx->launches += launch_rope_rows(dt, DKP, M, c.n_kv_heads, c.head_dim, S, 0, 1, rope, stream);
    }
    // ---- projections: dW_q = dq^T xn;  dW_k = dk_true^T h_true + dk_pred^T h_hat (same for V)
    if (grads->w_q != nullptr && dw_gemm_mn(DQ, qd, qd, Xn, d, d, grads->w_q) < 0) {
        transpose(DQ, M, qd, qd, TA, Mp, 0, Mp);
        transpose(Xn, M, d, d, TB, Mp, 0, Mp);
        BEAGLE_NEED(dw_gemm(qd, d, Mp, grads->w_q), "dW_q");
    }
    // (under simulation the contraction runs over two row blocks, true and predicted: that case keeps the transposed copies)
    bool kv_done = false;
    if (sim_steps == 1 && ctx->tc != nullptr) {
        kv_done = true;
        if (grads->w_k != nullptr) kv_done = kv_done && dw_gemm_mn(DKT, kd, kd, hidden_dev, d, d, grads->w_k) > 0;
        if (kv_done && grads->w_v != nullptr) kv_done = dw_gemm_mn(DVT, kd, kd, hidden_dev, d, d, grads->w_v) > 0;
    }
    if (!kv_done && (grads->w_k != nullptr || grads->w_v != nullptr)) {
        const int Kc = sim_steps > 1 ? 2 * Mp : Mp;
        transpose(hidden_dev, M, d, d, TB, Kc, 0, Mp);
        if (sim_steps > 1) transpose(H, M, d, d, TB, Kc, Mp, Mp);
        if (grads->w_k != nullptr) {
            transpose(DKT, M, kd, kd, TA, Kc, 0, Mp);
            if (sim_steps > 1) transpose(DKP, M, kd, kd, TA, Kc, Mp, Mp);
            BEAGLE_NEED(dw_gemm(kd, d, Kc, grads->w_k), "dW_k");
        }
        if (grads->w_v != nullptr) {
            transpose(DVT, M, kd, kd, TA, Kc, 0, Mp);
            if (sim_steps > 1) transpose(DVP, M, kd, kd, TA, Kc, Mp, Mp);
            BEAGLE_NEED(dw_gemm(kd, d, Kc, grads->w_v), "dW_v");
        }
    }
    // ---- query side down to the embedding: dxn = dq W_q, dx = dy + RMSNorm backward
    if (grads->g_q != nullptr || grads->embed != nullptr) {
        BEAGLE_NEED(dx_gemm(GEMM_STORE, DQ, qd, ctx->w.w_q, qd, d, DXN, nullptr), "dxn");
        StageTimer timer_(ctx, ST_BWD_ELEMENTWISE, stream);
        rc = launch_rmsnorm_bwd(dt, X, ctx->w.g_q, DXN, DY, M, d, c.rms_eps, c.norm_q, DYN, dgpart, grads->g_q, stream);   // DYN <- dx
        if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "block_grad: hidden too large for the RMSNorm backward");
        ctx->launches += rc;
        if (grads->embed != nullptr) {
            cudaMemsetAsync(grads->embed, 0, (size_t)V * d * sizeof(float), stream);
            ctx->launches += launch_embed_grad(dt, tokens_dev, DYN, M, d, grads->embed, stream);
        }
    }
#undef BEAGLE_BWD_GEMM
#undef BEAGLE_NEED
    return cuda_ok(ctx, "block_grad");
}

beagle_status beagle_verify_greedy(beagle_ctx* ctx, int32_t batch, int32_t gamma, const int32_t* draft_tokens_dev,
                                   const void* target_logits_dev, int32_t logits_dtype, const int32_t* target_ids_dev,
                                   int32_t* accept_len_dev, int32_t* out_tokens_dev, void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    if (batch < 0 || batch > BEAGLE_MAX_CALL_BATCH) return fail(ctx, BEAGLE_ERR_CAPACITY, "batch %d outside [0, %d]", batch, BEAGLE_MAX_CALL_BATCH);
    if (gamma < 0 || gamma > 64) return fail(ctx, BEAGLE_ERR_CAPACITY, "gamma %d outside [0, 64]", gamma);
    if (batch == 0) return BEAGLE_OK;
    if ((gamma > 0 && draft_tokens_dev == nullptr) || accept_len_dev == nullptr || out_tokens_dev == nullptr)
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "verify: NULL argument");
    if ((target_logits_dev == nullptr) == (target_ids_dev == nullptr))
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "verify: give exactly one of target_logits / target_ids");
    if (target_logits_dev != nullptr && logits_dtype != BEAGLE_FP32 && logits_dtype != BEAGLE_BF16)
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "verify: unknown logits_dtype");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (target_logits_dev != nullptr) {
        // one launch: arg-max partials of every logit row + the acceptance walk by the CTA that finishes a sequence last
        const beagle_status st = device_setup_once(ctx, stream);
        if (st != BEAGLE_OK) return st;
        StageTimer timer_(ctx, ST_VERIFY, stream);
        ctx->launches += launch_verify_greedy_fused(logits_dtype, target_logits_dev, batch, gamma, ctx->cfg.vocab, draft_tokens_dev,
                                                    ctx->verify_keys, verify_tickets(ctx), ctx->sm_count, accept_len_dev, out_tokens_dev, stream);
    } else {
        StageTimer timer_(ctx, ST_VERIFY, stream);
        ctx->launches += launch_accept(draft_tokens_dev, target_ids_dev, batch, gamma, accept_len_dev, out_tokens_dev, stream);
    }
    return cuda_ok(ctx, "verify_greedy");
}

beagle_status beagle_verify_sample(beagle_ctx* ctx, int32_t batch, int32_t gamma, const int32_t* draft_tokens_dev,
                                   const float* draft_logits_dev, const void* target_logits_dev, int32_t logits_dtype,
                                   float temperature, const float* u_accept_dev, const float* u_resample_dev,
                                   int32_t* accept_len_dev, int32_t* out_tokens_dev, void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    if (batch < 0 || batch > BEAGLE_MAX_CALL_BATCH) return fail(ctx, BEAGLE_ERR_CAPACITY, "batch %d outside [0, %d]", batch, BEAGLE_MAX_CALL_BATCH);
    if (gamma < 0 || gamma > 64) return fail(ctx, BEAGLE_ERR_CAPACITY, "gamma %d outside [0, 64]", gamma);
    if (!(temperature > 0.f)) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "verify_sample: temperature must be > 0");
    if (batch == 0) return BEAGLE_OK;
    if (target_logits_dev == nullptr || u_resample_dev == nullptr || accept_len_dev == nullptr || out_tokens_dev == nullptr ||
        (gamma > 0 && (draft_tokens_dev == nullptr || draft_logits_dev == nullptr || u_accept_dev == nullptr)))
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "verify_sample: NULL argument");
    if (logits_dtype != BEAGLE_FP32 && logits_dtype != BEAGLE_BF16) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "verify_sample: unknown logits_dtype");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const beagle_status st0 = device_setup_once(ctx, stream);          // the sequences' tickets must read zero
    if (st0 != BEAGLE_OK) return st0;
    StageTimer timer_(ctx, ST_VERIFY, stream);
    ctx->launches += launch_verify_sample(logits_dtype, draft_tokens_dev, draft_logits_dev, target_logits_dev, batch, gamma, ctx->cfg.vocab,
                                          temperature, u_accept_dev, u_resample_dev, ctx->vs_scratch, verify_tickets(ctx), accept_len_dev, out_tokens_dev, ctx->sm_count, stream);
    return cuda_ok(ctx, "verify_sample");
}

beagle_status beagle_draft_tree(beagle_ctx* ctx, int32_t slot, const int32_t* root_token_dev, int32_t depth, int32_t topk,
                                int32_t n_candidates, int32_t* tree_tokens_dev, int32_t* tree_parents_dev, float* tree_scores_dev,
                                void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    const beagle_config& c = ctx->cfg;
    if (slot < 0 || slot >= c.max_slots) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "slot %d out of range", slot);
    if (root_token_dev == nullptr || tree_tokens_dev == nullptr || tree_parents_dev == nullptr || tree_scores_dev == nullptr)
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "draft_tree: NULL argument");
    if (depth < 0 || depth > kTreeMaxDepth || topk < 1 || topk > kTreeMaxTopk || topk > c.vocab)
        return fail(ctx, BEAGLE_ERR_CAPACITY, "draft_tree: need 0 <= depth <= %d and 1 <= topk <= %d", kTreeMaxDepth, kTreeMaxTopk);
    const int total = topk + depth * topk * topk;
    if (n_candidates < 1 || n_candidates > kTreeMaxCandidates || n_candidates > total)
        return fail(ctx, BEAGLE_ERR_CAPACITY, "draft_tree: n_candidates must be in [1, min(%d, %d)]", kTreeMaxCandidates, total);
    if (ctx->tc == nullptr || (c.head_dim != 64 && c.head_dim != 128))
        return fail(ctx, BEAGLE_ERR_UNSUPPORTED, "draft_tree: needs the bf16 tensor-core path with head_dim 64 or 128");
    const int tail = depth > 0 ? 1 + (depth - 1) * topk : 0;          // draft states that enter the cache
    if (tail > c.max_draft) return fail(ctx, BEAGLE_ERR_CAPACITY, "draft_tree: %d draft states exceed max_draft %d", tail, c.max_draft);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const TreeArrays T = tree_arrays_carve(ctx->tree_mem, c.vocab);
    const int n_true = ctx->n_true[slot];
    if (c.rope_theta > 0.f && n_true + depth >= ctx->rope_rows)
        return fail(ctx, BEAGLE_ERR_CAPACITY, "draft_tree: positions up to %d exceed max_ctx + max_draft", n_true + depth + 1);
    const beagle_status st0 = device_setup_once(ctx, stream);
    if (st0 != BEAGLE_OK) return st0;
    // every check has passed: the tree starts from the true states, whatever chain-draft tail the slot had is dropped
    ctx->n_draft[slot] = 0; ctx->pending[slot] = 0; ctx->has_token[slot] = 0; ctx->steps[slot] = 0;
    const int dt = c.dtype;
    int rc = 0;
#define BEAGLE_TREE_SKINNY(MODE, ARGS, WHAT)                                              \
    do {                                                                                  \
        ARGS.partial = ctx->sk_partial;                                                   \
        ARGS.error_word = ctx->dev_error;                                                 \
        rc = tc_skinny(ctx->tc, MODE, ARGS, stream);                                      \
        if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, WHAT ": unsupported shape");      \
        ctx->launches += rc;                                                              \
    } while (0)

    for (int e = 0; e <= depth; ++e) {
        const int rows = e == 0 ? 1 : topk;                           // forward 0: the root; forward e: the frontier of level e
        const int nanc = e;                                           // ancestor states a row reads: the root's + e - 1 of its own line
        BatchMeta meta;
        memset(&meta, 0, sizeof(meta));
        RowMap slots, pos;
        for (int b = 0; b < kMaxCallBatch; ++b) { slots.idx[b] = slot; pos.idx[b] = -1; meta.slot[b] = slot; meta.kv_len[b] = n_true; }
        // x = E[token], xn = RMSNorm(x)
        ctx->launches += launch_embed_norm(dt, e == 0 ? root_token_dev : T.frontier_tok, nullptr, &meta, ctx->w.embed, c.vocab, nullptr, ctx->w.g_q,
                                           c.hidden, c.rms_eps, c.norm_q, ctx->x, ctx->xn, rows, nullptr, nullptr, stream);
        // the states produced by the previous forward join the cache tail (concatenation, Section 4.1)
        bool merged_qkv = false;
        if (e >= 1) {
            const int nprev = e == 1 ? 1 : topk;
            for (int r = 0; r < nprev; ++r) pos.idx[r] = n_true + (e == 1 ? 0 : 1 + (e - 2) * topk + r);
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_k; a.W2 = ctx->w.w_v; a.N = ctx->kd; a.K = c.hidden; a.X = ctx->h; a.ldx = c.hidden; a.B = nprev;
            a.kcache = ctx->kcache; a.vcache = ctx->vcache; a.Hkv = c.n_kv_heads; a.dh = c.head_dim; a.cap = ctx->cap;
            a.slot = slots; a.pos = pos;
            // one launch with the query projection when possible (rows beyond nprev have pos = -1 and are skipped)
            SkinnyArgs q;
            memset(&q, 0, sizeof(q));
            q.W = ctx->w.w_q; q.N = ctx->qd; q.K = c.hidden; q.X = ctx->xn; q.ldx = c.hidden; q.B = rows;
            q.out = ctx->q; q.ldo = ctx->qd; q.error_word = ctx->dev_error;
            SkinnyArgs kv = a;
            kv.B = rows;
            rc = tc_skinny_qkv(ctx->tc, q, kv, stream);
            if (rc > 0) { ctx->launches += rc; merged_qkv = true; }
            else BEAGLE_TREE_SKINNY(SK_KV, a, "K/V append");
        }
        if (!merged_qkv) {
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_q; a.N = ctx->qd; a.K = c.hidden; a.X = ctx->xn; a.ldx = c.hidden; a.B = rows;
            a.out = ctx->q; a.ldo = ctx->qd;
            BEAGLE_TREE_SKINNY(SK_STORE, a, "Q projection");
        }
        if (c.rope_theta > 0.f) {      // rotary option: the rows of forward e are tokens at position n_true + e + 1; the states appended now sit one before
            RowMap qpos, kpos;
            for (int b = 0; b < kMaxCallBatch; ++b) { qpos.idx[b] = n_true + e; kpos.idx[b] = n_true + (e > 0 ? e - 1 : 0); }
            ctx->launches += launch_rope_serve(dt, ctx->q, rows, c.n_q_heads, ctx->kcache, e >= 1 ? (e == 1 ? 1 : topk) : 0, c.n_kv_heads, c.head_dim,
                                               ctx->cap, slots, pos, qpos, kpos, ctx->rope_table, stream);
        }
        // attention: the true states (shared by the rows) in chunks, the ancestors' states as one extra chunk
        {
            int32_t stable[kMaxCallBatch];
            for (int b = 0; b < rows; ++b) stable[b] = n_true;
            float *po = nullptr, *pml = nullptr;
            int nch = 0;
            rc = tc_attn_decode(ctx->tc, ctx->q, meta, stable, rows, c.n_q_heads, c.n_kv_heads, c.head_dim, ctx->cap, n_true,
                                ctx->attn_scratch, nullptr, ctx->o, ctx->dev_error, stream, 1, &po, &pml, &nch);
            if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "attention: unsupported head shape");
            ctx->launches += rc;
            if (nanc > 0) {
                rc = launch_attn_tail(ctx->q, ctx->kcache, ctx->vcache, T.frontier_anc, nanc, rows, slot, n_true, c.n_q_heads, c.n_kv_heads,
                                      c.head_dim, ctx->cap, nch, (n_true + tc_attn_chunk() - 1) / tc_attn_chunk(), po, pml, stream);
                if (rc < 0) return fail(ctx, BEAGLE_ERR_SHAPE, "tree attention: unsupported head_dim");
                ctx->launches += rc;
            }
            ctx->launches += launch_attn_combine(1, po, pml, meta, rows, c.n_q_heads, c.head_dim, nch, tc_attn_chunk(), ctx->o, stream,
                                                 nanc > 0 ? 1 : 0);
        }
        {
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_o; a.N = c.hidden; a.K = ctx->qd; a.X = ctx->o; a.ldx = ctx->qd; a.B = rows;
            a.out = ctx->y; a.ldo = c.hidden; a.resid = ctx->x; a.ldr = c.hidden;
            BEAGLE_TREE_SKINNY(SK_RESID, a, "O projection");
        }
        ctx->launches += launch_embed_norm(dt, nullptr, nullptr, nullptr, nullptr, 0, ctx->y, ctx->w.g_mlp, c.hidden, c.rms_eps, c.norm_mlp,
                                           nullptr, ctx->yn, rows, nullptr, nullptr, stream);
        {
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_gate; a.W2 = ctx->w.w_up; a.N = c.mlp_dim; a.K = c.hidden; a.X = ctx->yn; a.ldx = c.hidden; a.B = rows;
            a.out = ctx->act; a.ldo = c.mlp_dim;
            BEAGLE_TREE_SKINNY(SK_SILU_MUL, a, "gate/up projection");
        }
        {
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_down; a.N = c.hidden; a.K = c.mlp_dim; a.X = ctx->act; a.ldx = c.mlp_dim; a.B = rows;
            a.out = ctx->h; a.ldo = c.hidden; a.resid = ctx->y; a.ldr = c.hidden;
            BEAGLE_TREE_SKINNY(SK_RESID, a, "down projection");
        }
        {
            SkinnyArgs a;
            memset(&a, 0, sizeof(a));
            a.W = ctx->w.w_lm; a.N = c.vocab; a.K = c.hidden; a.X = ctx->h; a.ldx = c.hidden; a.B = rows;
            a.logits = ctx->tree_logits; a.keys = ctx->lm_partials;
            BEAGLE_TREE_SKINNY(SK_LOGITS, a, "LM head");
        }
        ctx->launches += launch_topk_logprob(ctx->tree_logits, rows, c.vocab, topk, T, stream);
        ctx->launches += launch_tree_expand(T, c.vocab, topk, rows, e, e == 0 ? 0 : topk + (e - 1) * topk * topk, stream);
    }
#undef BEAGLE_TREE_SKINNY
    ctx->launches += launch_tree_rerank(T, total, n_candidates, tree_tokens_dev, tree_parents_dev, tree_scores_dev, stream);
    return cuda_ok(ctx, "draft_tree");
}

beagle_status beagle_verify_tree_greedy(beagle_ctx* ctx, int32_t n_nodes, const int32_t* tree_tokens_dev, const int32_t* tree_parents_dev,
                                        const int32_t* target_ids_dev, int32_t out_cap, int32_t* accept_len_dev, int32_t* out_tokens_dev,
                                        int32_t* path_dev, void* stream_) {
    if (ctx == nullptr) return BEAGLE_ERR_INVALID_ARG;
    if (n_nodes < 0 || n_nodes > 4096) return fail(ctx, BEAGLE_ERR_CAPACITY, "verify_tree: n_nodes %d outside [0, 4096]", n_nodes);
    if (out_cap < 1) return fail(ctx, BEAGLE_ERR_INVALID_ARG, "verify_tree: out_cap must be >= 1");
    if (target_ids_dev == nullptr || accept_len_dev == nullptr || out_tokens_dev == nullptr ||
        (n_nodes > 0 && (tree_tokens_dev == nullptr || tree_parents_dev == nullptr)))
        return fail(ctx, BEAGLE_ERR_INVALID_ARG, "verify_tree: NULL argument");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    ctx->launches += launch_tree_verify(tree_tokens_dev, tree_parents_dev, n_nodes, target_ids_dev, out_cap, accept_len_dev, out_tokens_dev,
                                        path_dev, stream);
    return cuda_ok(ctx, "verify_tree_greedy");
}

}  // extern "C"
