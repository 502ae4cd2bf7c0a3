"""CPU oracle of the Beagle cross-attention draft head.

TEST INFRASTRUCTURE ONLY.  Nothing here is on the product path: the CUDA
library never imports, links or calls this package, and this package never
imports the CUDA binding.  Only the tests, the smoke check and the benchmark's
CPU-baseline / reference legs may use it.
"""
from .beagle_oracle import (  # noqa: F401
    HeadConfig,
    OracleHead,
    OracleSequence,
    rms_norm,
    round_bf16,
    silu,
    visible_true_count,
    project_kv,
    attention_weights,
    cross_attention,
    embed_tokens,
    query_projection,
    attention_rows,
    output_projection,
    mlp_block,
    down_projection,
    lm_head,
    draft_block,
    prefill_kv,
    rollback,
    draft_step,
    block_forward,
    argmax_lowest,
    verify_greedy,
    softmax_rows,
    residual_distribution,
    inverse_cdf,
    verify_sample,
    cross_entropy_rows,
    loss_weights,
    block_loss,
    rope_rotate,
    smooth_l1,
    rms_norm_backward,
    block_loss_grad,
    log_softmax_rows,
    top_k_lowest,
    draft_tree,
    verify_tree_greedy,
)
