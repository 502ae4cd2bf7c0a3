// bf16 tensor-core GEMM (tcgen05 + TMEM + TMA) behind the dense projections.
#pragma once
#include "../../include/beagle.h"
#include "kernels.h"

namespace beagle {

struct TcPlan;   // tensor maps of the weight matrices and launch constants

// Returns nullptr when the tensor-core path cannot serve this configuration.
// *hard_error = 1 when a device is present but the tensor-map encoder could not be obtained.
TcPlan* tc_plan_create(const beagle_config& cfg, const beagle_weights& w, int* hard_error);
void tc_plan_destroy(TcPlan* plan);
// C = A W^T with the fused epilogue `epi` (GemmEpilogue).  Returns the number of kernels launched,
// or -1 when this shape is not covered (the caller then uses the CUDA-core kernel).
int tc_gemm(TcPlan* plan, int epi, const GemmArgs& a, cudaStream_t stream);
// GEMM_ARGMAX_KEYS writes one packed key per (row, 256-column tile): keys [M, tc_argmax_tiles(N)].
int tc_argmax_tiles(int N);
int tc_keys_to_ids(const unsigned long long* keys, int rows, int ntiles, int32_t* ids, cudaStream_t stream);

// Test support: a one-CTA kernel whose bounded mbarrier wait (short limit, nothing ever arrives, no copy in flight) runs
// out and raises `error_word`, as the tensor-core kernels do when a wait of theirs gives up.
int launch_wait_timeout_selftest(int* error_word, cudaStream_t stream);

// ---- serve-time projections for 9..64 rows ("swap-AB") -----------------------------------------
// The weight matrix supplies the 128 MMA rows and the batch's activations the (<= 64) columns, so
// the weights are streamed exactly once whatever the batch.  The reduction dimension may be split
// across CTAs; each split writes fp32 partial sums that a finishing kernel adds in a fixed order
// and passes through the projection's epilogue.  The LM head writes logits and arg-max keys directly.
enum SkinnyMode {
    SK_STORE = 0,      // out[b][n] = W[n,:] . x_b
    SK_RESID = 1,      // out[b][n] = W[n,:] . x_b + resid[b][n]  (+ copy to out2[orow2[b]], + RMSNorm of the result to norm_out)
    SK_SILU_MUL = 2,   // out[b][n] = SiLU(W[n,:] . x_b) * (W2[n,:] . x_b)
    SK_KV = 3,         // W -> key cache, W2 -> value cache at (slot[b], head, pos[b]); pos[b] < 0 skips row b
    SK_LOGITS = 4      // logits[b][n] fp32 (optional) and one arg-max key per (b, 128-row tile)
};
struct SkinnyArgs {
    const void* W; const void* W2; int N, K;     // weights [N, K] row-major
    const void* X; int ldx; int B;               // activations [B, K], row stride ldx, B <= 64
    float* partial;                              // scratch, tc_skinny_partial_bytes() bytes
    void* out; int ldo;
    const void* resid; int ldr;
    void* out2; int ld2; RowMap orow2;
    void* norm_out; const void* gain; float eps; int do_norm;
    void* kcache; void* vcache; int Hkv, dh, cap; RowMap slot; RowMap pos;
    float* logits; unsigned long long* keys;     // keys: [B, tc_skinny_key_tiles(N)]
    // SK_LOGITS with FP8 operands (optional): W8 [N, K] and X8 [B, K] (dense) hold E4M3 bytes, w_scale [N] / x_scale [B] the
    // rows' scales; logits = w_scale[n] * x_scale[b] * sum_k W8[n, k] X8[b, k].  W / X are then unused.
    const void* W8; const float* w_scale; const void* X8; const float* x_scale;
    int* error_word;
};
// Kernels launched, or -1 when the shape is not covered.
int tc_skinny(TcPlan* plan, int mode, const SkinnyArgs& a, cudaStream_t stream);
// The query projection (SK_STORE arguments `q`) and the K/V append (SK_KV arguments `kv`) of one draft step as ONE launch;
// same reduction length and batch.  1, or -1 when not covered (the caller then launches the two separately).
int tc_skinny_qkv(TcPlan* plan, const SkinnyArgs& q, const SkinnyArgs& kv, cudaStream_t stream);
// Bytes of fp32 partial sums a projection [N, K] with `nmat` weight matrices needs for 64 rows.
size_t tc_skinny_partial_bytes(int N, int K, int nmat);
int tc_skinny_key_tiles(int N);
// Tile-major copy of a K-major weight matrix [N, K] (elt_bytes 2: bf16, 1: FP8 bytes) for the kernels above: tile (ta, kb) = rows
// [128 ta, +128) x bytes [128 kb, +128) of the matrix, 16 KB contiguous, at ((ta * ceil(K * elt_bytes / 128)) + kb) * 16 KB; rows and
// bytes past the matrix are zero.  tc_skinny_packed_bytes: size of the copy.  tc_skinny_pack: writes it (one launch) and registers
// it, so that tc_skinny / tc_skinny_qkv given W read `dst` instead; dst == nullptr forgets W's copy.  Returns launches or -1.
size_t tc_skinny_packed_bytes(int N, int K, int elt_bytes);
int tc_skinny_pack(TcPlan* plan, const void* W, int N, int K, int elt_bytes, void* dst, cudaStream_t stream);
void tc_skinny_forget_packed(TcPlan* plan);

// ---- TMA-staged decode attention over the bf16 cache (head_dim 64 or 128) ----------------------
// Binds the cache halves ([rows, head_dim] each); false when the shape is not covered.
bool tc_attn_bind_cache(TcPlan* plan, const void* kcache, const void* vcache, long long rows, int dh);
// Split-KV partials + combine, as launch_attn_decode; -1 when not covered (caller falls back).
// stable_len[b] (host, nullable): leading cache rows of row b's slot that no kernel still in flight writes.
int tc_attn_decode(TcPlan* plan, const void* q, const BatchMeta& meta, const int32_t* stable_len, int B, int Hq, int Hkv, int dh,
                   int cap, int max_kv_len, void* scratch, int* done_count, void* o, int* error_word, cudaStream_t stream,
                   int defer_merge = 0, float** part_o_out = nullptr, float** part_ml_out = nullptr, int* nch_stride_out = nullptr);
// defer_merge: only the chunk partials are written; the caller adds its own chunks and merges (tree drafting).
// done_count: B*Hkv device ints, zero before the first launch (the kernel leaves them zero).
int tc_attn_chunk(void);

// ---- block-masked cross-attention of the multi-token forward (bf16, head_dim 64 or 128) -------
// Same contract as launch_attn_block, on tcgen05 (both products as tcgen05.mma, accumulators in tensor memory); -1 when not
// covered (caller falls back).  Vt / Vp are read as they lie ([B*S, Hkv*dh]).  lse2 (optional, fp32 [B*S, Hq]): base-2
// log-sum-exp of every row's scaled scores, for the backward below.
int tc_attn_block_umma(TcPlan* plan, const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp, int B, int S, int Hq,
                       int Hkv, int dh, int block, int offset, int step, void* O, int* error_word, cudaStream_t stream, float* lse2 = nullptr);
// Attention backward on tcgen05 (same contract as launch_attn_block_bwd, bf16, head_dim 64 / 128); delta: fp32 [B*S, Hq] scratch.
int tc_attn_block_bwd_umma(TcPlan* plan, const void* Q, const void* Kt, const void* Vt, const void* Kp, const void* Vp, const void* O,
                           const void* dO, const float* lse2, int B, int S, int Hq, int Hkv, int dh, int block, int offset, int step,
                           float* delta, void* dQ, void* dKt, void* dVt, void* dKp, void* dVp, int* error_word, cudaStream_t stream);

}  // namespace beagle
