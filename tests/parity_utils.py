"""Helpers of the GPU parity tests: drive the CUDA library and the CPU oracle on the same seeded
inputs and compare them under the stated tolerances.

Tolerances (written here once, used by every parity test):
  * token ids, arg-max, accepted lengths: bit-exact wherever the oracle's top-2 logit margin
    exceeds 1e-2; below that margin either of the oracle's two best ids is accepted and the chain
    continues teacher-forced with the oracle's token;
  * bf16 storage: |gpu - ref| <= 2e-2 + 1e-2 |ref| on logits and hidden states;
  * fp32 storage: |gpu - ref| <= 1e-5 + 1e-5 |ref|.

Which oracle.  At the small sizes the reference is the oracle as defined (nothing rounded).  At the
full model sizes the bf16 storage of the K/V cache and of the activations alone moves the logits
(standard deviation ~2.7 under the synthetic weights) by up to ~9e-2, above the bf16 tolerance,
whatever computes them; there the reference is the oracle in its "bf16" storage mode, which rounds
at the same places the library stores bf16 values, and the unrounded oracle is used for a second
statement: the library's distance to the exact result is explained by those roundings
(explained_by_storage).
"""
from __future__ import annotations

import numpy as np
import torch

import oracle as O
from paper_2505_24544_b200 import workloads as WL

MARGIN = 1e-2


def tolerances(dtype: str):
    return (2e-2, 1e-2) if dtype == "bf16" else (1e-5, 1e-5)


def oracle_head(w: WL.Workload, weights_np, storage=None, rope_theta=0.0) -> O.OracleHead:
    cfg = O.HeadConfig(w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.mlp_dim, w.vocab, rms_eps=w.rms_eps, storage=storage,
                       rope_theta=rope_theta)
    return O.OracleHead(cfg, weights_np)


def explained_by_storage(gpu: np.ndarray, stored: np.ndarray, exact: np.ndarray, what: str, slack: float = 1.5):
    """The library is no farther from the exact (unrounded fp64) result than the bf16 storage
    roundings explain: rms and max distance within `slack` of the storage-mode oracle's own."""
    gpu, stored, exact = (np.asarray(a, dtype=np.float64) for a in (gpu, stored, exact))
    e_gpu, e_st = gpu - exact, stored - exact
    rms_gpu, rms_st = float(np.sqrt(np.mean(e_gpu ** 2))), float(np.sqrt(np.mean(e_st ** 2)))
    assert rms_gpu <= slack * rms_st + 1e-3, f"{what}: rms distance to the exact result {rms_gpu:.3e}, storage roundings explain {rms_st:.3e}"
    assert np.abs(e_gpu).max() <= slack * np.abs(e_st).max() + 5e-3, (
        f"{what}: max distance to the exact result {np.abs(e_gpu).max():.3e}, storage roundings explain {np.abs(e_st).max():.3e}")
    return rms_gpu, rms_st


def record_distance(what: str, **numbers):
    """Prints a measured distance (visible with pytest -s / -rP) and, when BEAGLE_PARITY_REPORT names a file, appends it
    there as one JSON line, so that a GPU run leaves the figures the design notes quote."""
    import json
    import os
    line = {"what": what, **{k: (float(v) if isinstance(v, (float, np.floating)) else v) for k, v in numbers.items()}}
    print("[parity]", json.dumps(line))
    path = os.environ.get("BEAGLE_PARITY_REPORT")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(line) + "\n")


def first_hop_end_to_end(gpu, cpu_storage: O.OracleHead, w: WL.Workload, slots, first_tokens: np.ndarray, contexts: dict, what: str,
                         scale: float):
    """End to end on the first draft hop (no predicted state is read yet), in the launch configuration of `slots`:
    the library's logits of the rows in `contexts` (batch row -> that sequence's true states)
      * against the storage-mode oracle, within `scale` x the bf16 tolerance;
      * against the UNROUNDED oracle: no farther than the storage roundings explain (explained_by_storage), the measured
        distances recorded, and the greedy token equal to the unrounded oracle's wherever its top-2 margin exceeds what
        bf16 storage alone can swap (at these sizes that is more than the 1e-2 of the small-size rule: the storage-mode
        oracle itself picks another token than the unrounded one on the Llama-2-7B shaped first hop, margin 3e-2);
      * bit for bit equal to a second run from the same state (same split schedule, no atomics in the sums).
    Leaves the slots as it found them (draft tails dropped)."""
    exact = cpu_storage.with_storage(None)
    tok_dev = to_dev(np.asarray(first_tokens, dtype=np.int32), w.dtype)
    tok1, logits1, _ = gpu.draft_step(slots, tokens_in=tok_dev, want_logits=True)
    gpu.rollback(slots)
    tok2, logits2, _ = gpu.draft_step(slots, tokens_in=tok_dev, want_logits=True)
    gpu.rollback(slots)
    torch.cuda.synchronize()
    assert torch.equal(logits1, logits2) and torch.equal(tok1, tok2), f"{what}: two runs from the same state differ"
    lg_all = logits1.float().cpu().numpy().astype(np.float64)
    toks = tok1.cpu().numpy()
    for b, ctx in contexts.items():
        seq_s, seq_e = O.OracleSequence(cpu_storage), O.OracleSequence(exact)
        O.prefill_kv(cpu_storage, seq_s, ctx)
        O.prefill_kv(exact, seq_e, ctx)
        ref = O.draft_step(cpu_storage, [seq_s], tokens_in=[int(first_tokens[b])])["logits"][0]
        ref_exact = O.draft_step(exact, [seq_e], tokens_in=[int(first_tokens[b])])["logits"][0]
        lg = lg_all[b]
        name = f"{what} row {b} (n = {ctx.shape[0]})"
        err_st = assert_close(lg, ref, w.dtype, f"{name}: end-to-end logits vs storage-mode oracle", scale=scale)
        rms_gpu, rms_st = explained_by_storage(lg, ref, ref_exact, f"{name}: end-to-end logits")
        atol, rtol = tolerances(w.dtype)
        e = np.abs(lg - ref_exact)
        top = np.partition(ref_exact, -2)[-2:]
        record_distance(name, gpu_vs_exact_rms=rms_gpu, gpu_vs_exact_max=float(e.max()),
                        gpu_beyond_tol=int(np.count_nonzero(e > atol + rtol * np.abs(ref_exact))), of=int(e.size),
                        storage_vs_exact_rms=rms_st, storage_vs_exact_max=float(np.abs(ref - ref_exact).max()),
                        gpu_vs_storage_max=err_st, exact_top2_margin=float(top[1] - top[0]),
                        token_equals_exact=bool(int(toks[b]) == int(np.argmax(ref_exact))),
                        token_equals_storage_oracle=bool(int(toks[b]) == int(np.argmax(ref))))
        # Token rule against the UNROUNDED oracle.  bf16 storage alone moves a logit by up to d_store (an oracle-only figure);
        # the library may be 1.5 x that + 5e-3 away (explained_by_storage), so two logits whose exact values differ by less
        # than twice that can legitimately swap.  Wherever the exact top-2 margin exceeds that the token must be the exact
        # oracle's; inside it the chosen token's exact logit must lie within the same distance of the exact maximum.
        d_store = float(np.abs(ref - ref_exact).max())
        swap = 2.0 * (1.5 * d_store + 5e-3)
        t = int(toks[b])
        assert ref_exact[t] >= ref_exact.max() - swap, (
            f"{name}: greedy token {t} has exact logit {ref_exact[t]:.4f}, exact maximum {ref_exact.max():.4f}, storage noise allows {swap:.3e}")
        if top[1] - top[0] > swap:
            assert t == int(np.argmax(ref_exact)), f"{name}: greedy token {t} != unrounded oracle's {int(np.argmax(ref_exact))} at margin {top[1] - top[0]:.3e}"


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
        # a different id is admissible only in a near tie, and only if the oracle itself puts it within the margin of its maximum
        # (with three or more logits inside the margin the runner-up is not the only valid answer)
        assert margin <= MARGIN and 0 <= gt[r] < flat.shape[1] and top[1] - flat[r][gt[r]] <= MARGIN, (
            f"{what}: row {r}: gpu id {gt[r]} (oracle logit {flat[r][min(max(int(gt[r]), 0), flat.shape[1] - 1)]:.6f}), oracle id {ref_ids[r]} "
            f"(logit {top[1]:.6f}), oracle top-2 margin {margin:.3e}")
    return ref_ids.reshape(ref_logits.shape[:-1])


def run_chain_parity(head_gpu, head_cpu: O.OracleHead, w: WL.Workload, slots, seqs_cpu, first_tokens: np.ndarray,
                     depth: int, concat: bool = True, check_rows=None, exact=None):
    """Drafts ``depth`` tokens on both sides from the current cache state and compares every step.
    ``check_rows``: batch rows that also exist on the oracle side (all by default); seqs_cpu lists
    the oracle sequences of exactly those rows.  ``exact`` = (unrounded oracle head, its sequences
    for the same rows): every step is also run there, with the same tokens, for the
    explained-by-storage statement."""
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
        if exact is not None:
            out_exact = O.draft_step(exact[0], exact[1], tokens_in=cpu_tokens, concat=concat)
            explained_by_storage(lg, out["logits"], out_exact["logits"], f"step {s + 1} logits")
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


# ---- per-stage parity: every kernel against the definition applied to that kernel's own inputs -------------------------

def _np(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


def serve_stage_parity(head_gpu, head_cpu: O.OracleHead, w: WL.Workload, slots, tokens: np.ndarray, kv_len, attn_rows,
                       tokens_gpu: np.ndarray, logits_gpu=None):
    """After one beagle_draft_step over `slots`: reads every intermediate vector of that step from the
    workspace and compares each stage's output with the oracle's stage function fed with the
    library's own inputs of that stage (so one stage's rounding noise is not carried into the next).
    `kv_len[b]`: states visible to row b during the step; `attn_rows`: rows whose attention is
    recomputed by the oracle from the library's cache."""
    from paper_2505_24544_b200 import binding as B
    n = len(slots)
    buf = {name: _np(B.beagle_workspace_buffer(head_gpu.ctx, name, n)) for name in ("x", "xn", "q", "o", "y", "yn", "act", "h")}
    dt = w.dtype
    np.testing.assert_array_equal(buf["x"], O.embed_tokens(head_cpu, tokens))                 # a gather: exact
    xn_ref, q_ref = O.query_projection(head_cpu, buf["x"])
    assert_close(buf["xn"], xn_ref, dt, "stage xn")
    assert_close(buf["q"], q_ref, dt, "stage q")
    kc, vc = B.kv_cache_views(head_gpu.ctx)
    for b in attn_rows:
        k = _np(kc[slots[b], :, :kv_len[b], :]).transpose(1, 0, 2)                            # [nv, Hkv, dh]
        v = _np(vc[slots[b], :, :kv_len[b], :]).transpose(1, 0, 2)
        o_ref = O.attention_rows(head_cpu, buf["q"][b:b + 1], [(k, v)])
        assert_close(buf["o"][b:b + 1], o_ref, dt, f"stage attention row {b}")
    assert_close(buf["y"], O.output_projection(head_cpu, buf["o"], buf["x"]), dt, "stage y")
    yn_ref, act_ref, h_ref = O.mlp_block(head_cpu, buf["y"])
    assert_close(buf["yn"], yn_ref, dt, "stage yn")
    assert_close(buf["act"], act_ref, dt, "stage act")
    assert_close(buf["h"], h_ref, dt, "stage h (gate/up + down from the library's y)")
    assert_close(buf["h"], O.down_projection(head_cpu, buf["act"], buf["y"]), dt, "stage h (down projection of the library's act)")
    z_ref = O.lm_head(head_cpu, buf["h"])
    if logits_gpu is not None:
        err = np.abs(_np(logits_gpu) - z_ref)
        assert np.all(err <= 1e-3 + 1e-4 * np.abs(z_ref)), f"stage logits: max abs err {err.max():.3e}"     # fp32 from exact bf16 products
    check_tokens(tokens_gpu, z_ref, "stage greedy token")
    return buf


def cache_rows_parity(head_gpu, head_cpu: O.OracleHead, w: WL.Workload, slot: int, pos0: int, states: np.ndarray, what: str):
    """K/V cache rows [pos0, pos0 + len(states)) of `slot` against the oracle's projection of `states`."""
    from paper_2505_24544_b200 import binding as B
    kc, vc = B.kv_cache_views(head_gpu.ctx)
    k_ref, v_ref = O.project_kv(head_cpu, states)
    n = states.shape[0]
    assert_close(_np(kc[slot, :, pos0:pos0 + n, :]).transpose(1, 0, 2), k_ref, w.dtype, f"{what} K rows")
    assert_close(_np(vc[slot, :, pos0:pos0 + n, :]).transpose(1, 0, 2), v_ref, w.dtype, f"{what} V rows")


def block_stage_parity(head_gpu, head_cpu: O.OracleHead, w: WL.Workload, tokens: np.ndarray, hidden: np.ndarray, block: int,
                       offset: int, sim_steps: int, seq: int, positions, hidden_out=None, argmax_gpu=None, logits_gpu=None):
    """After one beagle_block_forward(batch, S): the same per-stage comparison on sampled 1-based
    positions of sequence `seq`.  `hidden_out`: the caller's h tensor when one was passed."""
    from paper_2505_24544_b200 import binding as B
    batch, S = tokens.shape
    idx = np.asarray([seq * S + p - 1 for p in positions])
    rows = torch.from_numpy(idx).cuda()
    names = ["x", "xn", "q", "o", "y", "yn", "act", "kt", "vt"] + (["kp", "vp"] if sim_steps > 1 else []) + ([] if hidden_out is not None else ["h"])
    full = {name: B.beagle_block_workspace_buffer(head_gpu.ctx, name, batch, S) for name in names}
    buf = {name: _np(t[rows]) for name, t in full.items() if name not in ("kt", "vt", "kp", "vp")}
    buf["h"] = _np(hidden_out.reshape(batch * S, -1)[rows]) if hidden_out is not None else buf["h"]
    dt = w.dtype
    c = head_cpu.cfg
    np.testing.assert_array_equal(buf["x"], O.embed_tokens(head_cpu, tokens.reshape(-1)[idx]))
    xn_ref, q_ref = O.query_projection(head_cpu, buf["x"])
    assert_close(buf["xn"], xn_ref, dt, "block stage xn")
    assert_close(buf["q"], q_ref, dt, "block stage q")
    k_ref, v_ref = O.project_kv(head_cpu, hidden[seq][np.asarray(positions) - 1])
    assert_close(_np(full["kt"][rows]).reshape(len(idx), c.n_kv_heads, c.head_dim), k_ref, dt, "block stage Kt")
    assert_close(_np(full["vt"][rows]).reshape(len(idx), c.n_kv_heads, c.head_dim), v_ref, dt, "block stage Vt")
    base = seq * S
    for i, p in enumerate(positions):
        n = O.visible_true_count(p, block, offset)
        extra = min(p - n, sim_steps) - 1
        k = _np(full["kt"][base:base + n]).reshape(n, c.n_kv_heads, c.head_dim)
        v = _np(full["vt"][base:base + n]).reshape(n, c.n_kv_heads, c.head_dim)
        if extra > 0:
            k = np.concatenate([k, _np(full["kp"][base + n:base + n + extra]).reshape(extra, c.n_kv_heads, c.head_dim)])
            v = np.concatenate([v, _np(full["vp"][base + n:base + n + extra]).reshape(extra, c.n_kv_heads, c.head_dim)])
        o_ref = O.attention_rows(head_cpu, buf["q"][i:i + 1], [(k, v)])
        assert_close(buf["o"][i:i + 1], o_ref, dt, f"block stage attention p={p}")
    assert_close(buf["y"], O.output_projection(head_cpu, buf["o"], buf["x"]), dt, "block stage y")
    yn_ref, act_ref, h_ref = O.mlp_block(head_cpu, buf["y"])
    assert_close(buf["yn"], yn_ref, dt, "block stage yn")
    assert_close(buf["act"], act_ref, dt, "block stage act")
    assert_close(buf["h"], h_ref, dt, "block stage h")
    z_ref = O.lm_head(head_cpu, buf["h"])
    if logits_gpu is not None:
        err = np.abs(_np(logits_gpu.reshape(batch * S, -1)[rows]) - z_ref)
        assert np.all(err <= 1e-3 + 1e-4 * np.abs(z_ref)), f"block stage logits: max abs err {err.max():.3e}"
    if argmax_gpu is not None:
        check_tokens(argmax_gpu.reshape(-1)[rows].cpu().numpy(), z_ref, "block stage arg-max")
