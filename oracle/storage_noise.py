#!/usr/bin/env python
"""How far the bf16 storage of intermediates alone moves the draft head's outputs, per workload.

TEST INFRASTRUCTURE (CPU only; calls nothing but the oracle and the seeded input generators).

The bf16 workloads keep the K/V cache and the activations between two operations in bf16.  This
script measures, with the oracle alone, what that storage costs: it runs the first draft hop of
C2, C3 and of three sequences of C4 (shortest, longest, one more), and the first window slot of
sampled C5 positions, twice -- once with nothing rounded, once in the oracle's "bf16" storage mode
-- and prints the distance between the two: rms, max, and how many outputs lie beyond the bf16
tolerance 2e-2 + 1e-2 |ref|.  A third run rounds only the K/V cache rows (keys and values made by
the storage-mode head, everything after them exact), to separate the cache's share.

Those distances bound what ANY implementation that stores bf16 can achieve against the unrounded
definition; the GPU parity tests at the full sizes compare their own distance with them.

    python oracle/storage_noise.py [--workloads c2 c3 c4 c5] [--json out.json]
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle as O  # noqa: E402
from paper_2505_24544_b200 import workloads as WL  # noqa: E402

ATOL, RTOL = 2e-2, 1e-2


def distance(a: np.ndarray, exact: np.ndarray) -> dict:
    """rms / max distance of `a` to `exact` and the count of entries beyond the bf16 tolerance."""
    e = np.abs(np.asarray(a, dtype=np.float64) - exact)
    return {"rms": float(np.sqrt(np.mean(e ** 2))), "max": float(e.max()),
            "beyond_tol": int(np.count_nonzero(e > ATOL + RTOL * np.abs(exact))), "of": int(e.size)}


def first_hop(w: WL.Workload, head_exact: O.OracleHead, ctx: np.ndarray, token: int) -> dict:
    """First draft step after a context of true states: exact, storage mode, and cache-only rounding."""
    head_st = head_exact.with_storage("bf16")
    seq_e, seq_s = O.OracleSequence(head_exact), O.OracleSequence(head_st)
    O.prefill_kv(head_exact, seq_e, ctx)
    O.prefill_kv(head_st, seq_s, ctx)
    z_exact = O.draft_step(head_exact, [seq_e], tokens_in=[token])["logits"][0]
    z_store = O.draft_step(head_st, [seq_s], tokens_in=[token])["logits"][0]
    # cache-only rounding: the storage-mode head's K/V rows, read by the exact head
    seq_c = O.OracleSequence(head_exact)
    seq_c.k_true, seq_c.v_true = seq_s.k_true, seq_s.v_true
    z_cache = O.draft_step(head_exact, [seq_c], tokens_in=[token])["logits"][0]
    top = np.partition(z_exact, -2)[-2:]
    return {"n_ctx": int(ctx.shape[0]), "logit_std": float(z_exact.std()), "top2_margin_exact": float(top[1] - top[0]),
            "same_argmax": bool(int(np.argmax(z_exact)) == int(np.argmax(z_store))),
            "all_roundings": distance(z_store, z_exact), "cache_only": distance(z_cache, z_exact)}


def make_head(w: WL.Workload) -> O.OracleHead:
    cfg = O.HeadConfig(w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.mlp_dim, w.vocab, rms_eps=w.rms_eps)
    return O.OracleHead(cfg, WL.make_weights(w))


def run_c2():
    w = WL.WORKLOADS["c2_llama2_7b_b1"]
    head = make_head(w)
    rng = WL.data_rng(w)
    ctx = WL.make_hidden(w, rng, w.ctx_max)
    first = WL.make_tokens(w, rng, (1,))
    return {"c2_llama2_7b_b1 first hop": first_hop(w, head, ctx, int(first[0]))}, head


def run_c3_c4():
    w4 = WL.WORKLOADS["c4_llama3_8b_b32"]
    w3 = WL.WORKLOADS["c3_llama3_8b_b1"]
    head = make_head(w4)                     # C3 and C4 share the head (the batch-32 seed), as in the GPU tests
    out = {}
    rng = WL.data_rng(w4, 7)
    lengths = WL.make_context_lengths(w4, rng).astype(int)
    sample = sorted({int(np.argmin(lengths)), int(np.argmax(lengths)), 5, 17})
    kept = {}
    for b, n in enumerate(lengths):
        h = WL.make_hidden(w4, rng, int(n))
        if b in sample:
            kept[b] = h
    first = WL.make_tokens(w4, rng, (w4.batch,))
    for b in sample:
        out[f"c4_llama3_8b_b32 seq {b} first hop"] = first_hop(w4, head, kept[b], int(first[b]))
    rng3 = WL.data_rng(w3)
    ctx3 = WL.make_hidden(w3, rng3, w3.ctx_max)
    first3 = WL.make_tokens(w3, rng3, (1,))
    out["c3_llama3_8b_b1 first hop"] = first_hop(w3, head, ctx3, int(first3[0]))
    return out


def run_c5(head):
    w = WL.WORKLOADS["c5_block_llama2_7b"]
    if head is None:
        head = make_head(w.scaled(seed=WL.WORKLOADS["c2_llama2_7b_b1"].seed))
    out = {}
    S = w.ctx_max
    positions = sorted(set([1, 2, 3, 4, 5, 6, 7, 8, 61, 62, 63, 64, 65, 66, 67, 68, 1021, 1022, 1023, 1024, 1025, 1026, 1027, 1028,
                            S - 3, S - 2, S - 1, S]))
    for sim_steps in (1, 4):
        rng = WL.data_rng(w, 10 + sim_steps)
        tokens = WL.make_tokens(w, rng, (w.batch, S))
        hidden = np.stack([WL.make_hidden(w, rng, S) for _ in range(w.batch)])
        ex = O.block_forward(head, tokens[3], hidden[3], w.block, 0, sim_steps, positions=positions)
        st = O.block_forward(head.with_storage("bf16"), tokens[3], hidden[3], w.block, 0, sim_steps, positions=positions)
        slot = np.array([p - O.visible_true_count(p, w.block, 0) for p in positions])
        for name, rows in (("window slot 1", slot == 1), ("window slots 2..4", slot > 1)):
            if not rows.any():
                continue
            d = {"hidden": distance(st["hidden"][rows], ex["hidden"][rows]), "hidden_std": float(ex["hidden"][rows].std())}
            out[f"c5_block_llama2_7b sim_steps {sim_steps}, {name} ({int(rows.sum())} positions of one sequence)"] = d
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workloads", nargs="*", default=["c2", "c3", "c4", "c5"])
    ap.add_argument("--json", default=None)
    args = ap.parse_args()
    res, t0 = {}, time.perf_counter()
    head2 = None
    if "c2" in args.workloads:
        r, head2 = run_c2()
        res.update(r)
    if "c5" in args.workloads:
        res.update(run_c5(head2))
    del head2
    if "c3" in args.workloads or "c4" in args.workloads:
        res.update(run_c3_c4())
    print(f"# bf16 tolerance: {ATOL} + {RTOL}|ref|; distances are storage-mode oracle vs unrounded oracle ({time.perf_counter() - t0:.0f} s)")
    print("| case | rms | max | beyond tolerance | cache rounding only: rms / max / beyond |")
    print("|---|---|---|---|---|")
    for name, r in res.items():
        if "all_roundings" in r:
            a, c = r["all_roundings"], r["cache_only"]
            print(f"| {name} (n = {r['n_ctx']}, logit std {r['logit_std']:.2f}) | {a['rms']:.2e} | {a['max']:.2e} | {a['beyond_tol']} / {a['of']} | "
                  f"{c['rms']:.2e} / {c['max']:.2e} / {c['beyond_tol']} |")
        else:
            a = r["hidden"]
            print(f"| {name} (hidden std {r['hidden_std']:.2f}) | {a['rms']:.2e} | {a['max']:.2e} | {a['beyond_tol']} / {a['of']} | |")
    if args.json:
        with open(args.json, "w") as f:
            json.dump(res, f, indent=1)


if __name__ == "__main__":
    main()
