"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU checker.

This module holds no arithmetic of the method: it only draws random numbers,
rounds them to the storage type and names the shapes of the five workloads.
The stand-ins replace the paper's trained heads (Vicuna-7B / LLaMA-2-7B /
LLaMA-3 shapes) and its evaluation suites, which are not available: weights and
embeddings ~ N(0, 0.02), norm gains 1 + N(0, 0.02), target hidden states
~ N(0, 1), token ids uniform over the vocabulary, context lengths as listed.
All values are float32 arrays whose entries are exactly representable in the
storage type (bf16 or fp32), so both sides of a parity check read the same
numbers.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    mlp_dim: int
    vocab: int
    dtype: str              # "fp32" | "bf16" : storage of weights, states and cache
    batch: int
    ctx_min: int            # true states per sequence, uniform in [ctx_min, ctx_max]
    ctx_max: int
    gamma: int              # chain draft depth
    seed: int
    block: int = 0          # block-attention window (block-forward workloads only)
    agree: float = 0.7      # per-position agreement of the synthetic target stream
    rms_eps: float = 1e-5

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS: Dict[str, Workload] = {
    # tiny fp32 head, 64 target states, batch 1, depth 4
    "c1_tiny_fp32": Workload("c1_tiny_fp32", 256, 4, 4, 64, 688, 1024, "fp32", 1, 64, 64, 4, 1001),
    # Llama-2-7B shaped head (MHA), 1024 states, batch 1, depth 6
    "c2_llama2_7b_b1": Workload("c2_llama2_7b_b1", 4096, 32, 32, 128, 11008, 32000, "bf16", 1, 1024, 1024, 6, 1002),
    # Llama-3-8B shaped head (GQA 32/8), 4096 states, batch 1, depth 8
    "c3_llama3_8b_b1": Workload("c3_llama3_8b_b1", 4096, 32, 8, 128, 14336, 128256, "bf16", 1, 4096, 4096, 8, 1003),
    # batched serving, Llama-3-8B shape, 32 sequences, ragged contexts in [512, 8192], depth 6
    "c4_llama3_8b_b32": Workload("c4_llama3_8b_b32", 4096, 32, 8, 128, 14336, 128256, "bf16", 32, 512, 8192, 6, 1004),
    # block-attention forward, Llama-2-7B shape, 8 sequences x 2048 positions, window 4
    "c5_block_llama2_7b": Workload("c5_block_llama2_7b", 4096, 32, 32, 128, 11008, 32000, "bf16", 8, 2048, 2048, 4, 1005, block=4),
}


def round_to_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float32 array to the storage type (round-to-nearest-even for
    bf16) and return it as float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "fp32":
        return a
    if dtype != "bf16":
        raise ValueError(dtype)
    u = a.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def _normal(rng: np.random.Generator, shape, std: float, dtype: str, mean: float = 0.0) -> np.ndarray:
    a = rng.standard_normal(size=shape, dtype=np.float32)
    a *= np.float32(std)
    if mean:
        a += np.float32(mean)
    return round_to_storage(a, dtype)


def make_weights(w: Workload, seed: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Random-init parameters of the draft head, [out, in] row-major."""
    rng = np.random.Generator(np.random.PCG64(w.seed if seed is None else seed))
    d, qd, kd, m, V = w.hidden, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim, w.mlp_dim, w.vocab
    return {
        "embed": _normal(rng, (V, d), 0.02, w.dtype),
        "g_q": _normal(rng, (d,), 0.02, w.dtype, mean=1.0),
        "w_q": _normal(rng, (qd, d), 0.02, w.dtype),
        "w_k": _normal(rng, (kd, d), 0.02, w.dtype),
        "w_v": _normal(rng, (kd, d), 0.02, w.dtype),
        "w_o": _normal(rng, (d, qd), 0.02, w.dtype),
        "g_mlp": _normal(rng, (d,), 0.02, w.dtype, mean=1.0),
        "w_gate": _normal(rng, (m, d), 0.02, w.dtype),
        "w_up": _normal(rng, (m, d), 0.02, w.dtype),
        "w_down": _normal(rng, (d, m), 0.02, w.dtype),
        "w_lm": _normal(rng, (V, d), 0.02, w.dtype),
    }


def data_rng(w: Workload, stream: int = 1) -> np.random.Generator:
    """Generator for per-run data (states, tokens, lengths), separate from the weights' stream."""
    return np.random.Generator(np.random.PCG64([w.seed, stream]))


def make_context_lengths(w: Workload, rng: np.random.Generator) -> np.ndarray:
    """True-state count per sequence, uniform in [ctx_min, ctx_max]."""
    return rng.integers(w.ctx_min, w.ctx_max + 1, size=w.batch).astype(np.int32)


def make_hidden(w: Workload, rng: np.random.Generator, rows: int) -> np.ndarray:
    """Target-model hidden states ~ N(0, 1), [rows, hidden]."""
    return _normal(rng, (rows, w.hidden), 1.0, w.dtype)


def make_tokens(w: Workload, rng: np.random.Generator, shape) -> np.ndarray:
    return rng.integers(0, w.vocab, size=shape).astype(np.int32)


def make_target_stream(w: Workload, rng: np.random.Generator, draft_tokens: np.ndarray) -> np.ndarray:
    """Synthetic target top-1 ids [B, gamma+1]: each position copies the draft
    token with probability ``w.agree``, otherwise takes a different id; the
    bonus position is uniform."""
    draft = np.asarray(draft_tokens, dtype=np.int64)
    B, gamma = draft.shape
    keep = rng.random(size=(B, gamma)) < w.agree
    shift = rng.integers(1, w.vocab, size=(B, gamma))
    ids = np.where(keep, draft, (draft + shift) % w.vocab)
    bonus = rng.integers(0, w.vocab, size=(B, 1))
    return np.concatenate([ids, bonus], axis=1).astype(np.int32)


def make_target_logits(w: Workload, rng: np.random.Generator, rows: int,
                       planted: Optional[np.ndarray] = None, boost: float = 10.0) -> np.ndarray:
    """Random target logits [rows, vocab] ~ N(0, 1) in float32; ``planted[r] >= 0``
    raises that id's logit by ``boost`` so that it becomes the row's top-1."""
    z = rng.standard_normal(size=(rows, w.vocab), dtype=np.float32)
    if planted is not None:
        for r, t in enumerate(np.asarray(planted).reshape(-1)):
            if t >= 0:
                z[r, int(t)] += np.float32(boost)
    return z
