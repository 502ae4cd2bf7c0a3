#!/usr/bin/env python
"""Benchmark of the Beagle draft-head hot path on B200.

A "step" is one speculative-decoding iteration over the whole batch of the serving workload:
append K/V of the true states accepted by the previous verification (beagle_prefill_kv), draft
gamma tokens (beagle_draft_step x gamma, concat on, tokens fed device-to-device) and run the
greedy acceptance (beagle_verify_greedy) against a seeded synthetic target stream that agrees with
the draft at ~70 % per position.  value = drafted tokens per second = batch * gamma * steps / time.

One JSON line is printed by rank 0.  Besides the headline (batched serving, batch 32) the line
carries the batch-1 workloads, the block-attention forward, the roofline of the dominant kernel
(from per-stage CUDA events), the end-to-end figure with host buffers and the CPU oracle baseline.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2505_24544_b200 import workloads as WL  # noqa: E402

METRIC = "draft_tokens_per_s"
UNIT = "draft tokens/s"
HEADLINE = "c4_llama3_8b_b32"
STEP_TEXT = ("one SD iteration, enqueued call by call: prefill_kv(accepted states) + gamma x draft_step(concat) + verify_greedy; "
             "the draft chain alone under CUDA-graph replay is reported as draft_chain")
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# ------------------------------------------------------------------------------------------------ helpers

def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


def load_ncu_traffic():
    """Per-launch DRAM bytes of the profiled kernels, from the committed ncu summaries."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f)
    return {}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed regions run."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,utilization.gpu,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="beagle_clocks_", suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.out,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        rows = []
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) == 8:
                        rows.append(parts)
            os.unlink(self.path)
        except Exception:
            pass
        if not rows:
            return res
        def num(s):
            try:
                return float(s)
            except ValueError:
                return None
        busy = [r for r in rows if (num(r[3]) or 0) >= 50] or rows
        clocks = sorted(c for c in (num(r[0]) for r in busy) if c is not None)
        res["samples"] = len(busy)
        if clocks:
            res["sm_mhz"] = clocks[len(clocks) // 2]
        mx = [num(r[1]) for r in rows if num(r[1]) is not None]
        res["sm_max_mhz"] = max(mx) if mx else None
        pw = [num(r[2]) for r in busy if num(r[2]) is not None]
        res["power_w_max"] = max(pw) if pw else None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for i, n in enumerate(names):
            if any(r[4 + i].lower().startswith("active") for r in busy):
                res["reasons"].append(n)
        return res


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",")
    if local < len(vis) and vis[local].strip().isdigit():
        return int(vis[local])
    return local


def dist_info():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(ms: float, world: int, device=None, backend_is_gloo: bool = False) -> float:
    """The slowest rank's time (MAX all-reduce); identity on one rank."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device="cpu" if backend_is_gloo else device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ------------------------------------------------------------------------------------------------ serving scenario

class ServeScenario:
    """Pre-generated, device-resident inputs of `iters` speculative-decoding iterations."""

    def __init__(self, head, w: WL.Workload, iters: int, device):
        import torch
        self.torch = torch
        self.head, self.w, self.iters, self.device = head, w, iters, device
        self.slots = list(range(w.batch))
        rng = WL.data_rng(w, 7)
        self.lengths = WL.make_context_lengths(w, rng)
        g = torch.Generator(device=device)
        g.manual_seed(w.seed)
        dt = head.dtype
        # context states ~ N(0,1), generated on the device (values are bf16/fp32 representable by construction)
        self.ctx_hidden = torch.randn(int(self.lengths.sum()), w.hidden, generator=g, device=device, dtype=torch.float32).to(dt)
        self.new_hidden = torch.randn(iters, w.batch * (w.gamma + 1), w.hidden, generator=g, device=device, dtype=torch.float32).to(dt)
        self.first_tokens = torch.from_numpy(WL.make_tokens(w, rng, (iters, w.batch))).to(device)
        self.draft = torch.zeros(iters, w.batch, w.gamma, dtype=torch.int32, device=device)
        self.accept = torch.zeros(iters, w.batch, dtype=torch.int32, device=device)
        self.out_tokens = torch.zeros(iters, w.batch, w.gamma + 1, dtype=torch.int32, device=device)
        self.target_ids = torch.zeros(iters, w.batch, w.gamma + 1, dtype=torch.int32, device=device)
        self.new_len = [[1] * w.batch for _ in range(iters)]      # rows appended at the START of iteration it
        self.rng = rng

    def reset(self):
        from paper_2505_24544_b200 import binding as B
        for s in self.slots:
            B.beagle_reset_slot(self.head.ctx, s)
        self.head.prefill_kv(self.slots, [int(n) for n in self.lengths], self.ctx_hidden)

    def iteration(self, it: int, new_len=None, hidden=None, first=None, target=None):
        """Enqueues one SD iteration; nothing here synchronises."""
        from paper_2505_24544_b200 import binding as B
        w, head = self.w, self.head
        nl = self.new_len[it] if new_len is None else new_len
        hid = self.new_hidden[it] if hidden is None else hidden
        if it > 0:
            B.beagle_prefill_kv(head.ctx, self.slots, nl, hid)
        first = self.first_tokens[it] if first is None else first
        for s in range(w.gamma):
            B.beagle_draft_step(head.ctx, self.slots, first if s == 0 else None, True, self.draft[it, :, s])
        B.beagle_verify_greedy(head.ctx, self.draft[it], None, self.target_ids[it] if target is None else target,
                               self.accept[it], self.out_tokens[it])

    def rehearse(self):
        """Runs every iteration once (untimed) to learn the draft tokens, builds the ~70 %-agreement
        target stream from them and records how many true states each iteration appends."""
        torch = self.torch
        self.reset()
        for it in range(self.iters):
            w = self.w
            from paper_2505_24544_b200 import binding as B
            if it > 0:
                B.beagle_prefill_kv(self.head.ctx, self.slots, self.new_len[it], self.new_hidden[it])
            for s in range(w.gamma):
                B.beagle_draft_step(self.head.ctx, self.slots, self.first_tokens[it] if s == 0 else None, True, self.draft[it, :, s])
            torch.cuda.synchronize()
            draft = self.draft[it].cpu().numpy()
            target = WL.make_target_stream(w, self.rng, draft)
            self.target_ids[it].copy_(torch.from_numpy(target))
            a = 0
            acc = np.zeros(w.batch, dtype=np.int64)
            for b in range(w.batch):
                a = 0
                while a < w.gamma and draft[b, a] == target[b, a]:
                    a += 1
                acc[b] = a
            if it + 1 < self.iters:
                self.new_len[it + 1] = [int(a) + 1 for a in acc]
        self.mean_tau = float(np.mean([np.mean(n) for n in self.new_len[1:]])) if self.iters > 1 else None


def time_serve(scn: ServeScenario, steps: int, warmup: int, world: int):
    """Device-resident timing: W untimed + K timed iterations, CUDA events, barrier on both sides."""
    import torch
    scn.reset()
    for it in range(warmup):
        scn.iteration(it)
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    l0 = scn.head.launch_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for it in range(warmup, warmup + steps):
        scn.iteration(it)
    e1.record()
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    return e0.elapsed_time(e1), scn.head.launch_count - l0


def bench_draft_chain(scn: ServeScenario, reps: int = 30, warmup: int = 3):
    """The gamma chained draft steps alone (token fed device to device, concatenation on), captured once as a CUDA graph and
    replayed: median device time over `reps` replays, each bracketed by its own event pair, and the same chain enqueued call
    by call for comparison.  Every replay repeats the same work (same cache rows read and rewritten).  Weights exceed L2; the
    K/V cache of a batch-1 workload (17 MB) stays L2-resident between replays, as it does between the steps of a real chain."""
    import torch
    from paper_2505_24544_b200 import binding as B
    w, head = scn.w, scn.head
    scn.reset()
    draft = torch.zeros(w.batch, w.gamma, dtype=torch.int32, device=scn.device)

    def chain():
        for s in range(w.gamma):
            B.beagle_draft_step(head.ctx, scn.slots, scn.first_tokens[0] if s == 0 else None, True, draft[:, s])

    def timed(fn):
        ts = []
        for i in range(warmup + reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            if i >= warmup:
                ts.append(e0.elapsed_time(e1))
        return float(np.median(ts)), float(np.min(ts))

    def eager():
        chain()
        head.rollback(scn.slots)

    eager_ms, _ = timed(eager)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        chain()
    head.rollback(scn.slots)
    graph_ms, graph_min = timed(g.replay)
    del g
    toks = w.batch * w.gamma
    mean_ctx = float(np.mean(scn.lengths)) + (w.gamma - 1) / 2.0
    # step 1 has no draft state to append, so it does not stream W_k / W_v
    gb = (sum(step_bytes(w, float(np.mean(scn.lengths)) + s) for s in range(w.gamma))
          - elt(w) * 2 * w.hidden * w.n_kv_heads * w.head_dim) / 1e9
    return {"value": toks / (graph_ms * 1e-3), "unit": UNIT, "ms_per_chain": graph_ms, "min_ms": graph_min, "reps": reps,
            "timing": "median over CUDA-graph replays of gamma draft steps (argmax and draft-state append included), one event pair each",
            "enqueued_call_by_call": {"value": toks / (eager_ms * 1e-3), "ms_per_chain": eager_ms},
            "algorithmic_gb_per_chain": gb, "achieved_gbs": gb / (graph_ms * 1e-3), "mean_ctx": mean_ctx}


def profile_serve(scn: ServeScenario, steps: int, warmup: int):
    """Same iterations with every stage bracketed by CUDA events inside the library."""
    import torch
    from paper_2505_24544_b200 import binding as B
    scn.reset()
    for it in range(warmup):
        scn.iteration(it)
    torch.cuda.synchronize()
    B.beagle_profile_enable(scn.head.ctx, True)
    for it in range(warmup, warmup + steps):
        scn.iteration(it)
    torch.cuda.synchronize()
    stages = B.beagle_profile_read(scn.head.ctx)
    B.beagle_profile_enable(scn.head.ctx, False)
    return stages


def time_serve_e2e(scn: ServeScenario, steps: int, warmup: int, world: int):
    """End to end through the binding with HOST buffers: every iteration copies its new true
    states, first tokens and target ids from pinned host memory and reads accept lengths and
    emitted tokens back; the host's bookkeeping uses the values it read."""
    import torch
    w = scn.w
    dev = scn.device
    rows = w.batch * (w.gamma + 1)
    host_hidden = scn.new_hidden.cpu().pin_memory()
    host_first = scn.first_tokens.cpu().pin_memory()
    host_target = scn.target_ids.cpu().pin_memory()
    stage_h = torch.empty(rows, w.hidden, dtype=scn.head.dtype).pin_memory()
    dev_h = torch.empty(rows, w.hidden, dtype=scn.head.dtype, device=dev)
    dev_first = torch.empty(w.batch, dtype=torch.int32, device=dev)
    dev_target = torch.empty(w.batch, w.gamma + 1, dtype=torch.int32, device=dev)
    host_acc = torch.empty(w.batch, dtype=torch.int32).pin_memory()
    host_out = torch.empty(w.batch, w.gamma + 1, dtype=torch.int32).pin_memory()
    scn.reset()
    new_len = [1] * w.batch
    h2d = d2h = 0
    seq_row0 = np.arange(w.batch, dtype=np.int64) * (w.gamma + 1)      # first row of every sequence in host_hidden[it]

    def one(it, count):
        nonlocal new_len, h2d, d2h
        if it > 0:
            # pack the accepted rows of every sequence into the pinned staging buffer with one gather
            counts = np.asarray(new_len, dtype=np.int64)
            r = int(counts.sum())
            first_row = np.cumsum(counts) - counts
            idx = np.repeat(seq_row0 - first_row, counts) + np.arange(r)
            torch.index_select(host_hidden[it], 0, torch.from_numpy(idx), out=stage_h[:r])
            dev_h[:r].copy_(stage_h[:r], non_blocking=True)
            if count:
                h2d += r * w.hidden * stage_h.element_size()
        dev_first.copy_(host_first[it], non_blocking=True)
        dev_target.copy_(host_target[it], non_blocking=True)
        if count:
            h2d += dev_first.numel() * 4 + dev_target.numel() * 4
        scn.iteration(it, new_len=new_len, hidden=dev_h, first=dev_first, target=dev_target)
        host_acc.copy_(scn.accept[it], non_blocking=True)
        host_out.copy_(scn.out_tokens[it], non_blocking=True)
        torch.cuda.current_stream().synchronize()
        if count:
            d2h += (host_acc.numel() + host_out.numel()) * 4
        new_len = [int(a) + 1 for a in host_acc.tolist()]

    for it in range(warmup):
        one(it, False)
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for it in range(warmup, warmup + steps):
        one(it, True)
    e1.record()
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    return e0.elapsed_time(e1), h2d / steps, d2h / steps


# ------------------------------------------------------------------------------------------------ byte / flop accounting

def elt(w):
    return 2 if w.dtype == "bf16" else 4


def workload_config(w: WL.Workload, parallelism: str) -> dict:
    """The `config` object of a bench line: the workload and nothing that depends on the run, so that both arms print the same."""
    e, d, qd, kd, m, V = elt(w), w.hidden, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim, w.mlp_dim, w.vocab
    weights_gb = e * (2 * d * qd + 2 * d * kd + 3 * d * m + V * d) / 1e9
    return {"workload": w.name, "batch": w.batch, "gamma": w.gamma, "ctx": [w.ctx_min, w.ctx_max],
            "hidden": w.hidden, "heads": [w.n_q_heads, w.n_kv_heads, w.head_dim], "mlp": w.mlp_dim, "vocab": w.vocab,
            "step": STEP_TEXT,
            "l2": "inputs larger than L2: every draft step streams the head's %.2f GB of weights and the batch's K/V cache" % weights_gb,
            "parallelism": parallelism}


def step_bytes(w: WL.Workload, mean_ctx: float):
    """Algorithmic HBM bytes of one draft step of the whole batch (weights once + K/V per sequence)."""
    e, d, qd, kd, m, V = elt(w), w.hidden, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim, w.mlp_dim, w.vocab
    weights = e * (2 * d * qd + 2 * d * kd + 3 * d * m + V * d)
    kv = w.batch * 2 * kd * mean_ctx * e
    return weights + kv


def stage_bytes(w: WL.Workload, stage: str, mean_ctx: float):
    e, d, qd, kd, m, V, B = elt(w), w.hidden, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim, w.mlp_dim, w.vocab, w.batch
    return {
        "lm_head": e * (V * d + B * d),
        "gate_up": e * (2 * m * d + B * d + B * m),
        "down_proj": e * (d * m + B * m + 2 * B * d),
        "q_proj": e * (qd * d + B * d + B * qd),
        "o_proj": e * (d * qd + B * qd + 2 * B * d),
        "kv_append": e * (2 * kd * d + B * d + 2 * B * kd),
        "qkv_proj": e * (qd * d + B * d + B * qd + 2 * kd * d + B * d + 2 * B * kd),
        "attn_decode": e * (B * 2 * kd * mean_ctx + 2 * B * qd),
    }.get(stage)


# ------------------------------------------------------------------------------------------------ CPU oracle legs

def oracle_head_for(w: WL.Workload):
    import oracle as O
    weights = WL.make_weights(w)
    head = O.OracleHead(O.HeadConfig(w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.mlp_dim, w.vocab, rms_eps=w.rms_eps), weights)
    del weights
    return head


def blas_threads() -> int:
    threads = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        nt = [p.get("num_threads") for p in threadpool_info() if p.get("user_api") == "blas"]
        if nt:
            threads = max(nt)
    except Exception:
        pass
    return threads


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except Exception:
        pass
    return "unknown"


def oracle_sample(w: WL.Workload, n_seq: int, iters: int, warm: int = 0, head=None, threads=None):
    """Times the CPU oracle, as it stands, on `n_seq` sequences of the workload for `iters` SD
    iterations (context prefill untimed; `threads`: limit of the BLAS pool, None = all cores).
    Returns (draft tokens/s, seconds, threads used)."""
    import contextlib

    import oracle as O
    if head is None:
        head = oracle_head_for(w)
    rng = WL.data_rng(w, 7)
    lengths = WL.make_context_lengths(w, rng)[:n_seq]
    seqs = []
    for n in lengths:
        s = O.OracleSequence(head)
        O.prefill_kv(head, s, WL.make_hidden(w, rng, int(n)))
        seqs.append(s)
    new_len = [1] * n_seq
    first = WL.make_tokens(w, rng, (n_seq,))
    limit = contextlib.nullcontext()
    if threads is not None:
        from threadpoolctl import threadpool_limits
        limit = threadpool_limits(limits=threads)
    with limit:
        used = blas_threads() if threads is None else threads
        t0 = time.perf_counter()
        for it in range(-warm, iters):
            if it == 0:
                t0 = time.perf_counter()
            if it != -warm:
                for b, s in enumerate(seqs):
                    O.prefill_kv(head, s, WL.make_hidden(w, rng, new_len[b]))
            drafted = np.zeros((n_seq, w.gamma), dtype=np.int64)
            for st in range(w.gamma):
                out = O.draft_step(head, seqs, tokens_in=list(first) if st == 0 else None, concat=True)
                drafted[:, st] = out["argmax"]
            target = WL.make_target_stream(w, rng, drafted)
            acc, out_tok = O.verify_greedy(drafted, target_ids=target)
            new_len = [int(a) + 1 for a in acc]
            first = np.array([out_tok[b, acc[b]] for b in range(n_seq)])
        dt = time.perf_counter() - t0
    return n_seq * w.gamma * iters / dt, dt, used


def cpu_baseline_legs(head_llama3):
    """The oracle as it stands on the machine's host cores, single-threaded and with all cores, on every serving workload:
    C1..C3 one or more full SD iterations of the whole workload, C4 on a stated subset of its sequences.  `head_llama3`:
    an oracle head of the Llama-3-8B shape (C3 and C4 share it; the weights' seed does not matter for a timing)."""
    out = {"nproc": os.cpu_count(), "cpu_model": cpu_model(), "workloads": {}}
    plan = [("c1_tiny_fp32", 1, 8, None), ("c2_llama2_7b_b1", 1, 1, None), ("c3_llama3_8b_b1", 1, 1, head_llama3), (HEADLINE, 4, 1, head_llama3)]
    for name, n_seq, iters, head in plan:
        w = WL.WORKLOADS[name]
        if head is None:
            head = oracle_head_for(w)
        n_seq = min(n_seq, w.batch)
        v_all, s_all, t_all = oracle_sample(w, n_seq, iters, head=head)
        v_one, s_one, _ = oracle_sample(w, n_seq, iters, head=head, threads=1)
        out["workloads"][name] = {"all_cores": {"value": v_all, "seconds": s_all, "threads": t_all},
                                  "single_thread": {"value": v_one, "seconds": s_one, "threads": 1}, "unit": UNIT,
                                  "sample": f"{n_seq} of {w.batch} sequence(s) x {iters} SD iteration(s) of {w.gamma} draft tokens, context prefill untimed"}
        del head
    return out


def run_reference(args):
    """`--impl reference`: the CPU oracle, unmodified, on the host cores (rank 0 only)."""
    rank, world, _ = dist_info()
    if rank != 0:
        return
    w = WL.WORKLOADS[args.workload]
    n_seq = min(8, w.batch)
    steps = max(1, min(args.steps, 4))
    warm = 1 if args.warmup > 0 else 0
    t0 = time.perf_counter()
    val, sec, threads = oracle_sample(w, n_seq, steps, warm)
    sample = f"{n_seq} of {w.batch} sequences x {steps} SD iteration(s) of {w.gamma} draft tokens, context prefill untimed"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": 1e3 * sec / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, "single"),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample, "nproc": os.cpu_count(),
                         "cpu_model": cpu_model()},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "wall_s": time.perf_counter() - t0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------ block forward

def bench_block(head, w: WL.Workload, steps: int, warmup: int, peaks):
    import torch
    from paper_2505_24544_b200 import binding as B
    dev = head.device
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed)
    S = w.ctx_max
    tokens = torch.randint(0, w.vocab, (w.batch, S), generator=g, device=dev, dtype=torch.int32)
    hidden = torch.randn(w.batch, S, w.hidden, generator=g, device=dev, dtype=torch.float32).to(head.dtype)
    argmax = torch.empty(w.batch, S, dtype=torch.int32, device=dev)

    def run():
        B.beagle_block_forward(head.ctx, tokens, hidden, w.block, 0, 1, None, argmax, None)

    for _ in range(warmup):
        run()
    torch.cuda.synchronize()
    l0 = head.launch_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    launches = (head.launch_count - l0) // steps
    B.beagle_profile_enable(head.ctx, True)
    run()
    torch.cuda.synchronize()
    stages = B.beagle_profile_read(head.ctx)
    B.beagle_profile_enable(head.ctx, False)
    M = w.batch * S
    d, qd, kd, m, V = w.hidden, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim, w.mlp_dim, w.vocab
    flops = {"blk_lm_head": 2.0 * M * V * d, "blk_gate_up": 4.0 * M * m * d, "blk_down": 2.0 * M * m * d,
             "blk_qkv": 2.0 * M * d * (qd + 2 * kd), "blk_o_proj": 2.0 * M * d * qd}
    vis = sum(WL_vis(p, w.block) for p in range(1, S + 1)) * w.batch
    flops["blk_attn"] = 4.0 * w.head_dim * w.n_q_heads * vis
    total = sum(flops.values())
    st = {k: {"ms": v[0], "tflops": (flops[k] / (v[0] * 1e-3) / 1e12) if k in flops and v[0] > 0 else None} for k, v in stages.items()}
    lm = st.get("blk_lm_head", {})
    peak = peaks["bf16_tflops"]               # the stage timer brackets this GEMM alone: the burst figure is its denominator
    peak_sustained = peaks["bf16_tflops_sustained"]
    # loss forward (Eq. 4, hard labels): the same forward with the cross-entropy epilogue instead of the arg-max one
    labels = torch.randint(0, w.vocab, (w.batch, S), generator=g, device=dev, dtype=torch.int32)
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    for _ in range(2):
        B.beagle_block_loss(head.ctx, tokens, hidden, w.block, 0, 1, "early", None, labels, loss, None)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        B.beagle_block_loss(head.ctx, tokens, hidden, w.block, 0, 1, "early", None, labels, loss, None)
    e1.record()
    torch.cuda.synchronize()
    loss_ms = e0.elapsed_time(e1) / steps
    # one training step (forward + backward, Eq. 4 with hard labels plus the state regression, coefficient 10):
    # gradients of the head's own parameters (the embedding and the LM head belong to the target model)
    own = ("g_q", "w_q", "w_k", "w_v", "w_o", "g_mlp", "w_gate", "w_up", "w_down")
    grads = {n: torch.empty(head.weight_shapes[n], dtype=torch.float32, device=dev) for n in own}
    losses = torch.empty(3, dtype=torch.float32, device=dev)

    def train_step():
        B.beagle_block_grad(head.ctx, tokens, hidden, w.block, 0, 1, "early", None, labels, 10.0, grads, losses)

    for _ in range(2):
        train_step()
    torch.cuda.synchronize()
    l0 = head.launch_count
    e0.record()
    for _ in range(steps):
        train_step()
    e1.record()
    torch.cuda.synchronize()
    train_ms = e0.elapsed_time(e1) / steps
    train_launches = (head.launch_count - l0) // steps
    B.beagle_profile_enable(head.ctx, True)
    train_step()
    torch.cuda.synchronize()
    tstages = {k: {"ms": v[0], "n": v[1]} for k, v in B.beagle_profile_read(head.ctx).items()}
    B.beagle_profile_enable(head.ctx, False)
    # forward once, re-materialised logits once, then two products per linear layer (dX and dW; no dX for K/V inputs, no dW for the LM head)
    train_flop = total + flops["blk_lm_head"] + flops["blk_lm_head"] + 2 * (flops["blk_gate_up"] + flops["blk_down"] + flops["blk_o_proj"]) \
        + 2.0 * M * d * (qd + 2 * kd) + 2.0 * M * d * qd + 2.5 * flops["blk_attn"]
    return {
        "loss_forward": {"ms": loss_ms, "tflops": total / (loss_ms * 1e-3) / 1e12, "loss": float(loss.item()), "stage": "early, hard labels"},
        "train_step": {"ms": train_ms, "tflop": train_flop / 1e12, "tflops": train_flop / (train_ms * 1e-3) / 1e12, "gpu_launches": train_launches,
                       "positions_per_s": M / (train_ms * 1e-3), "losses": [float(x) for x in losses.tolist()], "stages": tstages,
                       "what": "forward + backward, early stage, hard labels, vloss 10, gradients of the head's own parameters"},
        "workload": w.name, "positions_per_s": M / (ms * 1e-3), "ms_per_forward": ms, "tflop_per_forward": total / 1e12,
        "tflops": total / (ms * 1e-3) / 1e12, "gpu_launches": launches, "stages": st,
        "roofline": {"bound": "tensor", "kernel": "blk_lm_head", "achieved": lm.get("tflops"), "peak": peak, "unit": "TFLOP/s",
                     "frac": (lm.get("tflops") / peak) if lm.get("tflops") else None, "traffic": None,
                     "peak_source": peaks["source"] + " (burst)",
                     "peak_sustained": peak_sustained, "frac_of_sustained": (lm.get("tflops") / peak_sustained) if lm.get("tflops") else None,
                     "whole_forward_frac_of_sustained": total / (ms * 1e-3) / 1e12 / peak_sustained},
    }


def bench_verify_sample(head, w: WL.Workload, steps: int, warmup: int, peaks):
    """Acceptance under sampling on the workload's shape: batch x (gamma+1) bf16 target rows and
    gamma x batch fp32 draft rows of V logits; HBM-bound (every logit is read once, two rows per
    sequence a second time)."""
    import torch
    dev = head.device
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed + 1)
    B, gamma, V = w.batch, w.gamma, w.vocab
    zq = torch.randn(gamma, B, V, generator=g, device=dev, dtype=torch.float32) * 2
    zp = (zq.transpose(0, 1) * 0.7 + torch.randn(B, gamma, V, generator=g, device=dev) * 1.4)
    zp = torch.cat([zp, torch.randn(B, 1, V, generator=g, device=dev) * 2], dim=1).to(torch.bfloat16).contiguous()
    draft = torch.distributions.Categorical(logits=zq).sample().transpose(0, 1).to(torch.int32).contiguous()
    ua = torch.rand(B, gamma, generator=g, device=dev)
    ur = torch.rand(B, generator=g, device=dev)
    for _ in range(warmup):
        acc, _ = head.verify_sample(draft, zq, zp, ua, ur)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        acc, _ = head.verify_sample(draft, zq, zp, ua, ur)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    by = B * (gamma + 1) * V * 2 + gamma * B * V * 4 + 2 * B * V * (2 + 4)
    return {"us_per_call": 1e3 * ms, "algorithmic_mb": by / 1e6, "gbs": by / (ms * 1e-3) / 1e9,
            "frac_of_hbm_peak": by / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "mean_accept_len": float(acc.float().mean()),
            "note": "156 MB of logits is close to L2 size: repeated calls partly hit L2"}


def bench_prefill(scn, peaks, reps: int = 5, warmup: int = 2):
    """K/V projection of a whole context into the cache (beagle_prefill_kv over every sequence's true states, packed):
    the one tensor-bound step of the serving path.  Median over `reps` calls, one event pair each; the states (> 1 GB at
    batch 32) exceed L2."""
    import torch
    from paper_2505_24544_b200 import binding as B
    w, head = scn.w, scn.head
    lengths = [int(n) for n in scn.lengths]
    rows = int(sum(lengths))
    ts = []
    l0 = 0
    for i in range(warmup + reps):
        for s in scn.slots:
            B.beagle_reset_slot(head.ctx, s)
        torch.cuda.synchronize()
        l0 = head.launch_count
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        head.prefill_kv(scn.slots, lengths, scn.ctx_hidden)
        e1.record()
        torch.cuda.synchronize()
        if i >= warmup:
            ts.append(e0.elapsed_time(e1))
    ms = float(np.median(ts))
    kd = w.n_kv_heads * w.head_dim
    flop = 2.0 * rows * w.hidden * 2 * kd
    by = elt(w) * (rows * w.hidden + 2 * kd * w.hidden + 2 * rows * kd)
    tf = flop / (ms * 1e-3) / 1e12
    return {"rows": rows, "sequences": len(lengths), "ms": ms, "min_ms": float(np.min(ts)), "states_per_s": rows / (ms * 1e-3),
            "tflop": flop / 1e12, "tflops": tf, "frac_of_bf16_burst_peak": tf / peaks["bf16_tflops"],
            "algorithmic_gb": by / 1e9, "gbs": by / (ms * 1e-3) / 1e9, "gpu_launches": head.launch_count - l0,
            "timing": "median of %d calls, one CUDA-event pair each" % reps}


def bench_verify_greedy_logits(head, w: WL.Workload, peaks, reps: int = 20, warmup: int = 3):
    """Greedy verification from the target's logits (fp32 [batch, gamma + 1, V]): arg-max of every row + the acceptance
    walk, one launch.  HBM-bound: every logit is read once.  The calls rotate over enough distinct logit buffers to
    exceed L2 several times, so every call reads from HBM."""
    import torch
    dev = head.device
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed + 2)
    Bn, gamma, V = w.batch, w.gamma, w.vocab
    by = Bn * (gamma + 1) * V * 4
    nbuf = max(3, int(np.ceil(512e6 / by)) + 1)
    bufs = [torch.randn(Bn, gamma + 1, V, generator=g, device=dev, dtype=torch.float32) for _ in range(nbuf)]
    draft = torch.stack([b[:, :gamma].argmax(dim=-1) for b in bufs]).to(torch.int32)
    flip = torch.rand(draft.shape, generator=g, device=dev) > 0.7           # ~70 % agreement per position
    draft = torch.where(flip, (draft + 1) % V, draft).contiguous()
    from paper_2505_24544_b200 import binding as B
    acc = torch.empty(nbuf, Bn, dtype=torch.int32, device=dev)
    out = torch.empty(nbuf, Bn, gamma + 1, dtype=torch.int32, device=dev)

    def calls():
        for i in range(reps):
            B.beagle_verify_greedy(head.ctx, draft[i % nbuf], bufs[i % nbuf], None, acc[i % nbuf], out[i % nbuf])

    # the kernel lasts a few microseconds at batch 1, less than the host needs to enqueue it: the calls are captured once
    # into a CUDA graph and the replay is timed (one launch per call either way)
    l0 = head.launch_count
    calls()
    launches = head.launch_count - l0
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        calls()
    ts = []
    for i in range(warmup + 5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        if i >= warmup:
            ts.append(e0.elapsed_time(e1) / reps)
    del graph
    ms = float(np.median(ts))
    acc = acc[0]
    return {"us_per_call": 1e3 * ms, "algorithmic_mb": by / 1e6, "gbs": by / (ms * 1e-3) / 1e9,
            "frac_of_hbm_peak": by / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "launches_per_call": launches / reps,
            "timing": "median of 5 CUDA-graph replays of %d calls" % reps,
            "mean_accept_len": float(acc.float().mean()), "rotating_buffers": nbuf,
            "shape": [Bn, gamma + 1, V], "dtype": "f32"}


def bench_draft_tree(head, w: WL.Workload, scn, steps: int, warmup: int, peaks):
    """Dynamic draft tree at the paper's setting (depth 1 + 6, top-10, 60 candidates) on one sequence
    of the batch-1 workload: 7 forwards of 1 / 10 rows, each streaming the head's weights once."""
    import torch
    from paper_2505_24544_b200 import binding as B
    depth, topk, n_cand = 6, 10, 60
    scn.reset()
    root = scn.first_tokens[0, :1].contiguous()
    tok = torch.empty(n_cand, dtype=torch.int32, device=head.device)
    par = torch.empty_like(tok)
    sc = torch.empty(n_cand, dtype=torch.float32, device=head.device)
    for _ in range(warmup):
        B.beagle_draft_tree(head.ctx, 0, root, depth, topk, n_cand, tok, par, sc)
    torch.cuda.synchronize()
    l0 = head.launch_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        B.beagle_draft_tree(head.ctx, 0, root, depth, topk, n_cand, tok, par, sc)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    e, d, qd, kd, m, V = elt(w), w.hidden, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim, w.mlp_dim, w.vocab
    weights = e * (2 * d * qd + 2 * d * kd + 3 * d * m + V * d)
    gb = (depth + 1) * weights / 1e9
    return {"ms_per_tree": ms, "candidates_per_s": n_cand / (ms * 1e-3), "depth": depth, "topk": topk, "candidates": n_cand,
            "algorithmic_gb_per_tree": gb, "achieved_gbs": gb / (ms * 1e-3), "frac_of_hbm_peak": gb / (ms * 1e-3) / peaks["hbm_gbs"],
            "gpu_launches": (head.launch_count - l0) // steps}


def WL_vis(p: int, block: int, offset: int = 0) -> int:
    """Visible true keys of position p under the inverse block mask (flop accounting only)."""
    return p - 1 if p <= offset else offset + block * ((p - 1 - offset) // block)


# ------------------------------------------------------------------------------------------------ main

def serve_result(scn, w, ms, steps, world):
    total_tokens = world * w.batch * w.gamma * steps
    return total_tokens / (ms * 1e-3)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=[k for k in WL.WORKLOADS if not k.startswith("c5")])
    ap.add_argument("--only-headline", action="store_true", help="skip the batch-1, block-forward and CPU legs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fp8-lm-head", action="store_true", help="diagnostic: the serve scenario with the optional FP8 LM head (not the headline arithmetic)")
    ap.add_argument("--only-block", action="store_true", help="diagnostic: time only the block-attention forward (C5 shape)")
    ap.add_argument("--block-batch", type=int, default=0, help="sequences of the block forward (default: the workload's 8)")
    ap.add_argument("--only-legs", action="store_true", help="diagnostic: only the prefill, verification and draft-tree legs of the headline workload")
    ap.add_argument("--legs-batch", type=int, default=0, help="with --only-legs: cut the workload down to this many sequences (profiler captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    from paper_2505_24544_b200 import build as _build
    _build.build()
    from paper_2505_24544_b200 import binding as B
    from paper_2505_24544_b200.binding import BeagleHead

    rank, world, local = dist_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=device)
    peaks = load_peaks()
    traffic = load_ncu_traffic()
    t_wall = time.perf_counter()

    if args.only_block:
        w5 = WL.WORKLOADS["c5_block_llama2_7b"]
        if args.block_batch > 0:
            w5 = w5.scaled(batch=args.block_batch)
        head5 = BeagleHead.from_workload(w5, WL.make_weights(w5), device=device, max_slots=1, max_ctx=64, max_draft=1)
        res = bench_block(head5, w5, steps=max(1, args.steps), warmup=args.warmup, peaks=peaks)
        if rank == 0:
            print(json.dumps({"metric": "block_positions_per_s", "value": res["positions_per_s"], "unit": "positions/s", "n_gpus": world,
                              "steps": args.steps, "warmup": args.warmup, "ms_per_step": res["ms_per_forward"], "higher_is_better": True,
                              "dtype": "bf16", "data": "synthetic", "config": {"workload": w5.name, "batch": w5.batch, "S": w5.ctx_max},
                              "block_forward": res}), flush=True)
        return

    w = WL.WORKLOADS[args.workload]
    if args.only_legs and args.legs_batch > 0:
        w = w.scaled(batch=min(w.batch, args.legs_batch))
    iters = args.steps + args.warmup
    extra = iters * (w.gamma + 1) + 64
    max_draft = 64          # chain depth <= 8; the draft tree (depth 6, top-10) keeps 51 draft states
    weights = WL.make_weights(w)
    head = BeagleHead.from_workload(w, weights, device=device, max_slots=w.batch, max_ctx=w.ctx_max + extra, max_draft=max_draft,
                                    fp8_lm_head=args.fp8_lm_head)
    del weights

    sampler = ClockSampler(physical_gpu_index(local))
    scn = ServeScenario(head, w, iters, device)
    if args.only_legs:
        out = {"prefill": {w.name: bench_prefill(scn, peaks)}, "verify_greedy_logits": {w.name: bench_verify_greedy_logits(head, w, peaks)},
               "verify_sample": bench_verify_sample(head, w, steps=20, warmup=3, peaks=peaks)}
        w3 = WL.WORKLOADS["c3_llama3_8b_b1"]
        if w.name == HEADLINE and args.legs_batch == 0:
            scn3 = ServeScenario(head, w3, iters, device)
            out["prefill"][w3.name] = bench_prefill(scn3, peaks)
            out["draft_tree"] = bench_draft_tree(head, w3, scn3, steps=5, warmup=3, peaks=peaks)
            out["verify_greedy_logits"][w3.name] = bench_verify_greedy_logits(head, w3, peaks)
        if rank == 0:
            print(json.dumps(out), flush=True)
        return
    scn.rehearse()
    sampler.start()
    ms, launches = time_serve(scn, args.steps, args.warmup, world)
    ms = max_over_ranks(ms, world, device)
    value = serve_result(scn, w, ms, args.steps, world)
    stages = profile_serve(scn, args.steps, args.warmup)
    e2e_ms, h2d, d2h = time_serve_e2e(scn, args.steps, args.warmup, world)
    e2e_ms = max_over_ranks(e2e_ms, world, device)
    e2e_value = serve_result(scn, w, e2e_ms, args.steps, world)
    mean_ctx = float(scn.lengths.mean()) + (args.warmup + args.steps / 2) * (scn.mean_tau or 1.0)

    stage_out = {}
    for name, (sms, cnt) in stages.items():
        per = sms / cnt
        by = stage_bytes(w, name, mean_ctx)
        if args.fp8_lm_head and name == "lm_head":
            by = w.vocab * w.hidden + w.batch * w.hidden          # one byte per element
        stage_out[name] = {"us_per_launch": 1e3 * per, "launches": cnt, "share": sms / max(1e-9, sum(v[0] for v in stages.values())),
                           "gbs": (by / (per * 1e-3) / 1e9) if by else None}
    dom = max((k for k in stage_out if stage_out[k]["gbs"]), key=lambda k: stage_out[k]["share"])
    achieved = stage_out[dom]["gbs"]
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": traffic.get(f"{dom}@{w.name}"),
                "algorithmic_bytes_per_launch": stage_bytes(w, dom, mean_ctx), "peak_source": peaks["source"],
                "attn_decode_gbs": stage_out.get("attn_decode", {}).get("gbs"),
                "attn_decode_frac": (stage_out["attn_decode"]["gbs"] / peaks["hbm_gbs"]) if stage_out.get("attn_decode", {}).get("gbs") else None}
    if args.fp8_lm_head:
        roofline["traffic"] = None
        roofline["algorithmic_bytes_per_launch"] = (w.vocab * w.hidden + w.batch * w.hidden) if dom == "lm_head" else roofline["algorithmic_bytes_per_launch"]
    step_gb = (step_bytes(w, mean_ctx) - (w.vocab * w.hidden if args.fp8_lm_head else 0)) * w.gamma / 1e9

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": ("bf16" if w.dtype == "bf16" else "f32") + ("+e4m3 LM head (diagnostic run, not the headline)" if args.fp8_lm_head else ""),
        "data": "synthetic",
        "config": workload_config(w, "replicas" if world > 1 else "single"),
        "run": {"mean_tau": scn.mean_tau,
                "weights": "row-major as the caller gave them + tile-major copies of the eight projection matrices, made once at load "
                           "(beagle_pack_weights, %.2f GB), which the draft steps of this batch size stream"
                           % ((head.ctx.packed_buf.numel() if head.ctx.packed_buf is not None else 0) / 1e9)},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": launches,
        "roofline": roofline,
        "step_hbm": {"algorithmic_gb_per_step": step_gb, "achieved_gbs": step_gb / (ms / args.steps * 1e-3),
                     "frac_of_peak": step_gb / (ms / args.steps * 1e-3) / peaks["hbm_gbs"]},
        "stages": stage_out,
    }

    if not args.only_headline and world == 1:
        # batch-1 serving on the same head (Llama-3-8B shape) and on the Llama-2-7B shaped head
        others = {}
        line["verify_sample"] = bench_verify_sample(head, w, steps=max(3, min(20, args.steps)), warmup=3, peaks=peaks)
        line["prefill"] = {w.name: bench_prefill(scn, peaks)}
        line["verify_greedy_logits"] = {w.name: bench_verify_greedy_logits(head, w, peaks)}
        chains = {w.name: bench_draft_chain(scn)}
        if w.name == HEADLINE:
            w3 = WL.WORKLOADS["c3_llama3_8b_b1"]
            scn3 = ServeScenario(head, w3, iters, device)
            scn3.rehearse()
            ms3, l3 = time_serve(scn3, args.steps, args.warmup, 1)
            st3 = profile_serve(scn3, args.steps, args.warmup)
            others[w3.name] = summarize_b1(w3, scn3, ms3, l3, st3, args, peaks)
            chains[w3.name] = bench_draft_chain(scn3)
            line["prefill"][w3.name] = bench_prefill(scn3, peaks)
            line["verify_greedy_logits"][w3.name] = bench_verify_greedy_logits(head, w3, peaks)
            line["draft_tree"] = bench_draft_tree(head, w3, scn3, steps=max(3, min(20, args.steps)), warmup=3, peaks=peaks)
            del scn3
            # the same batch-32 scenario with the optional FP8 (E4M3) copy of the LM head (NOT the headline: another arithmetic type
            # for the largest weight stream; greedy verification stays lossless, only the acceptance rate could change)
            w8 = dict(head.ctx.weights)
            w8["w_lm_fp8"], w8["w_lm_scale"] = B.beagle_quantize_rows_e4m3(w8["w_lm"])
            head8 = BeagleHead(hidden=w.hidden, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim, mlp_dim=w.mlp_dim,
                               vocab=w.vocab, dtype=w.dtype, weights=w8, max_slots=w.batch, max_ctx=w.ctx_max + extra, max_draft=max_draft,
                               rms_eps=w.rms_eps)
            scn8 = ServeScenario(head8, w, iters, device)
            scn8.rehearse()
            ms8, l8 = time_serve(scn8, args.steps, args.warmup, 1)
            st8 = profile_serve(scn8, args.steps, args.warmup)
            lm8 = st8.get("lm_head")
            line["fp8_lm_head"] = {"value": serve_result(scn8, w, ms8, args.steps, 1), "unit": UNIT, "ms_per_step": ms8 / args.steps,
                                   "gpu_launches": l8, "dtype": "bf16, LM head weights and its input states in FP8 E4M3 with row scales",
                                   "lm_head_us": (1e3 * lm8[0] / lm8[1]) if lm8 else None,
                                   "lm_head_gbs": ((w.vocab * w.hidden + w.batch * w.hidden) / (lm8[0] / lm8[1] * 1e-3) / 1e9) if lm8 else None,
                                   "speedup_over_bf16": (ms / args.steps) / (ms8 / args.steps)}
            del scn8
            head8.ctx.close()
            del head8, w8
        del scn
        head.ctx.close()
        del head
        torch.cuda.empty_cache()
        w2 = WL.WORKLOADS["c2_llama2_7b_b1"]
        w5 = WL.WORKLOADS["c5_block_llama2_7b"]
        weights2 = WL.make_weights(w2)
        head2 = BeagleHead.from_workload(w2, weights2, device=device, max_slots=1, max_ctx=w2.ctx_max + extra, max_draft=max_draft)
        del weights2
        scn2 = ServeScenario(head2, w2, iters, device)
        scn2.rehearse()
        ms2, l2 = time_serve(scn2, args.steps, args.warmup, 1)
        st2 = profile_serve(scn2, args.steps, args.warmup)
        others[w2.name] = summarize_b1(w2, scn2, ms2, l2, st2, args, peaks)
        chains[w2.name] = bench_draft_chain(scn2)
        for c in chains.values():
            c["frac_of_hbm_peak"] = c["achieved_gbs"] / peaks["hbm_gbs"]
        line["batch1"] = others
        line["draft_chain"] = chains
        del scn2
        line["block_forward"] = bench_block(head2, w5, steps=max(2, min(5, args.steps)), warmup=3, peaks=peaks)
        head2.ctx.close()
        del head2
        torch.cuda.empty_cache()
    line["clocks"] = sampler.stop()

    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.only_headline:
        n_seq, n_it = min(8, w.batch), 4                 # a few seconds of numpy on the machine's cores
        head_cpu = oracle_head_for(w)
        val, sec, threads = oracle_sample(w, n_seq, n_it, head=head_cpu)
        line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": sec,
                                "sample": f"{n_seq} of {w.batch} sequences x {n_it} SD iterations of {w.gamma} draft tokens, context prefill untimed"}
        if w.name == HEADLINE:
            line["cpu_baseline"].update(cpu_baseline_legs(head_cpu))
        del head_cpu
    line["wall_s"] = time.perf_counter() - t_wall
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


def summarize_b1(w, scn, ms, launches, stages, args, peaks):
    mean_ctx = float(scn.lengths.mean()) + (args.warmup + args.steps / 2) * (scn.mean_tau or 1.0)
    gb = step_bytes(w, mean_ctx) * w.gamma / 1e9
    per_step = ms / args.steps
    out = {"value": w.batch * w.gamma * args.steps / (ms * 1e-3), "unit": UNIT, "ms_per_step": per_step, "gpu_launches": launches,
           "mean_tau": scn.mean_tau, "algorithmic_gb_per_step": gb, "achieved_gbs": gb / (per_step * 1e-3),
           "frac_of_hbm_peak": gb / (per_step * 1e-3) / peaks["hbm_gbs"], "stages": {}}
    tot = sum(v[0] for v in stages.values())
    for name, (sms, cnt) in stages.items():
        by = stage_bytes(w, name, mean_ctx)
        per = sms / cnt
        out["stages"][name] = {"us_per_launch": 1e3 * per, "share": sms / tot, "gbs": (by / (per * 1e-3) / 1e9) if by else None}
    return out


if __name__ == "__main__":
    main()
