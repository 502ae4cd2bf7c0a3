"""Helpers of the GPU parity tests: drive the CUDA library and the CPU oracle on the same seeded
inputs and compare them under the stated tolerances.

Tolerances (written here once, used by every parity test):
  * token ids, arg-max, accepted lengths: bit-exact wherever the oracle's top-2 logit margin
    exceeds 1e-2; below that margin either of the oracle's two best ids is accepted and the chain
    continues teacher-forced with the oracle's token;
  * bf16 storage: |gpu - ref| <= 2e-2 + 1e-2 |ref| on logits and hidden states;
  * fp32 storage: |gpu - ref| <= 1e-5 + 1e-5 |ref|.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle as O
from paper_2505_24544_b200 import workloads as WL

MARGIN = 1e-2


def tolerances(dtype: str):
    return (2e-2, 1e-2) if dtype == "bf16" else (1e-5, 1e-5)


def oracle_head(w: WL.Workload, weights_np) -> O.OracleHead:
    cfg = O.HeadConfig(w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.mlp_dim, w.vocab, rms_eps=w.rms_eps)
    return O.OracleHead(cfg, weights_np)


def to_dev(a: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    if a.dtype == np.float32:
        t = t.to(torch.bfloat16 if dtype == "bf16" else torch.float32)
    return t.contiguous()


def assert_close(gpu: np.ndarray, ref: np.ndarray, dtype: str, what: str, scale: float = 1.0):
    atol, rtol = tolerances(dtype)
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (what, gpu.shape, ref.shape)
    assert np.all(np.isfinite(gpu)), f"{what}: non-finite GPU values"
    err = np.abs(gpu - ref)
    bound = scale * (atol + rtol * np.abs(ref))
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    assert np.all(err <= bound), (f"{what}: max abs err {err.max():.3e} (at {worst}: gpu {gpu[worst]:.6f} ref {ref[worst]:.6f}), "
                                  f"allowed {bound[worst]:.3e}")
    return float(err.max())


def check_tokens(gpu_tok: np.ndarray, ref_logits: np.ndarray, what: str):
    """Token ids against the oracle's logits under the top-2 margin rule.  Returns the oracle ids."""
    ref_logits = np.asarray(ref_logits, dtype=np.float64)
    flat = ref_logits.reshape(-1, ref_logits.shape[-1])
    gt = np.asarray(gpu_tok).reshape(-1)
    ref_ids = O.argmax_lowest(flat)
    for r in range(flat.shape[0]):
        if gt[r] == ref_ids[r]:
            continue
        top = np.partition(flat[r], -2)[-2:]
        margin = top[1] - top[0]
        second = [i for i in np.argsort(flat[r])[-2:]]
        assert margin <= MARGIN and gt[r] in second, (
            f"{what}: row {r}: gpu id {gt[r]}, oracle id {ref_ids[r]}, oracle top-2 margin {margin:.3e}")
    return ref_ids.reshape(ref_logits.shape[:-1])


def run_chain_parity(head_gpu, head_cpu: O.OracleHead, w: WL.Workload, slots, seqs_cpu, first_tokens: np.ndarray,
                     depth: int, concat: bool = True, check_rows=None):
    """Drafts ``depth`` tokens on both sides from the current cache state and compares every step.
    ``check_rows``: batch rows that also exist on the oracle side (all by default); seqs_cpu lists
    the oracle sequences of exactly those rows."""
    B = len(slots)
    rows = list(range(B)) if check_rows is None else list(check_rows)
    tok_dev = to_dev(first_tokens.astype(np.int32), w.dtype)
    cpu_tokens = [int(first_tokens[r]) for r in rows]
    drafted_gpu = np.zeros((B, depth), dtype=np.int64)
    drafted_ref = np.zeros((len(rows), depth), dtype=np.int64)
    max_err = 0.0
    for s in range(depth):
        t_out, logits, hidden = head_gpu.draft_step(slots, tokens_in=tok_dev, concat=concat, want_logits=True, want_hidden=True)
        torch.cuda.synchronize()
        out = O.draft_step(head_cpu, seqs_cpu, tokens_in=cpu_tokens, concat=concat)
        lg = logits.float().cpu().numpy()[rows]
        max_err = max(max_err, assert_close(lg, out["logits"], w.dtype, f"step {s + 1} logits"))
        assert_close(hidden.float().cpu().numpy()[rows], out["h"], w.dtype, f"step {s + 1} hidden")
        gt = t_out.cpu().numpy()
        ref_ids = check_tokens(gt[rows], out["logits"], f"step {s + 1} tokens")
        drafted_gpu[:, s] = gt
        drafted_ref[:, s] = ref_ids
        same = bool(np.all(gt[rows] == ref_ids))
        if same and len(rows) == B:
            tok_dev = None                       # continue from the device-resident greedy tokens
        else:
            forced = gt.copy()
            forced[rows] = ref_ids               # teacher-force the oracle's ids
            tok_dev = to_dev(forced.astype(np.int32), w.dtype)
        cpu_tokens = [int(t) for t in ref_ids]
    return drafted_gpu, drafted_ref, max_err
