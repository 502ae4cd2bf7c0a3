"""Plain fp64 CPU statement of the Beagle draft head (cross-attention speculative decoding).

TEST INFRASTRUCTURE ONLY -- slow, obvious, independent of the CUDA library.
Every floating-point operation runs in numpy float64; the only library
primitives are matrix products, exp, sqrt and argmax.  Inputs arrive already
rounded to whatever storage type the caller studies (bf16 values are exactly
representable in float64).  By default the oracle rounds nothing in between;
two options do round, each where its paragraph below says: the "bf16" storage
mode (stored intermediates) and the FP8 LM head (quantised operands).

Notation follows the paper (Section 3 "Preliminaries", Section 4.1
"Cross-Attention Draft Modeling", Section 4.2 "Two-Stage Block-Attention
Training"):

  * positions are 1-based; ``h_j`` is the higher-level state at position j
    (it predicts token j+1); the query at position p is built from ``e(t_p)``;
  * Eq. 1:  y_p = CrossAttn(h_{1:p-1}, e(t_p)) + e(t_p);  h_p = MLP(y_p) + y_p;
  * Eq. 2:  Q = W_Q^T e(t_p), K_j = W_K^T h_j, V_j = W_V^T h_j, softmax over
    the visible keys of <Q, K_j>/sqrt(d_h), o = sum_j s_j V_j, y = W_O^T[o^1..o^H];
  * the cross mask hides every key j >= p (the diagonal too);
  * logits z_p = e^{-1}(h_p) is a plain linear map to the vocabulary.

Arrays are 0-based: ``tokens[p-1]`` is t_p and ``hidden[j-1]`` is h_j.
Weights use the [out, in] row-major layout, i.e. the stored matrix is the
paper's W^T; per-head matrices are consecutive row blocks of w_q / w_k / w_v
and consecutive column blocks of w_o.

Readings taken where the paper is silent (all are the caller's config flags or
stated in the function that uses them):
  * the mask is applied before the softmax (rows over visible keys sum to one);
  * RMSNorm (gain g, eps) on the query input and on the MLP input, residuals
    add the un-normalised vectors, no norm on key/value inputs, none before the
    LM head;
  * the MLP is SiLU-gated without biases: W_down( SiLU(W_gate n) * (W_up n) );
  * grouped-query attention: query head h reads key/value head h // (Hq/Hkv);
  * a query with no visible key gets o = 0;
  * argmax ties go to the lowest index, NaN never wins.

Positional option.  Eq. 2 has no positional term and the five workloads use
none.  With ``HeadConfig.rope_theta > 0`` the queries and keys carry a rotary
position embedding in the LLaMA convention ("rotate half"): within every head,
components i and i + d_h/2 are rotated by the angle pos * theta^(-2i/d_h),
pos = position - 1 (the query at position p uses p - 1; the key made from the
state at position j uses j - 1, true or predicted), so a score depends on
p - j only.  Values are not rotated.

Storage mode.  By default nothing is rounded.  With ``HeadConfig.storage = "bf16"`` the
values that a bf16 deployment keeps in memory between two operations -- the
normalised query input, Q, the K/V cache rows, the attention output o, y, the
normalised MLP input, the MLP hidden vector and the block output h -- are
rounded to bf16 (round to nearest, ties to even) exactly where they would be
stored; everything in between stays float64 and the logits are not rounded.
This is the reading "weights, states and cache in bf16" of the bf16 workloads:
at the full model sizes the rounding of the cache alone moves logits of
standard deviation ~2.7 by up to ~5e-2, so a comparison that wants to see
kernel errors rather than storage noise has to round at the same places.

FP8 option (not in the paper): lm_head_fp8 is the LM head with weights and incoming
states quantised row-wise to FP8 E4M3; round_e4m3 follows the published format.

Speculative-sampling verification (verify_sample) follows Section 3 literally;
the random numbers it needs are inputs.

Training step (block_loss_grad): the losses of Section 4.2 (Eq. 4, Eq. 7), the
hidden-state regression term of Appendix B (smooth-L1, as in the EAGLE papers
it cites) and their gradient in every parameter, by the chain rule written out
operation by operation.  Under simulation the predicted states are constants of
the differentiation (the function's docstring states this reading).  Pinned by
central differences of block_loss and by automatic differentiation of a torch
restatement.

Pins (tests/test_oracle_*.py, all CPU): hand-worked tiny head, softmax row
sums, single-key / identical-key special cases, GQA==MHA with repeated heads,
mask brute force against the literal window rule, block forward == step-by-step
drafting, greedy losslessness, the tail-sum closed form for the expected
acceptance length, and a library cross-check (torch scaled-dot-product
attention, F.silu, F.linear).  The paper prints no numeric example of the
layer; its tokens/s and acceptance-length tables need trained weights and
public evaluation suites, so those figures are "parity unpinned".
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Iterable, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


@dataclass(frozen=True)
class HeadConfig:
    hidden: int          # d
    n_q_heads: int       # Hq
    n_kv_heads: int      # Hkv (Hq % Hkv == 0)
    head_dim: int        # d_h
    mlp_dim: int         # m
    vocab: int           # V
    rms_eps: float = 1e-5
    norm_q: bool = True
    norm_mlp: bool = True
    storage: Optional[str] = None   # None: never round; "bf16": round stored intermediates (module docstring)
    rope_theta: float = 0.0         # 0: no positional term (Eq. 2 as printed); > 0: rotary embedding base (module docstring)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


_WEIGHT_SHAPES = {
    "embed": lambda c: (c.vocab, c.hidden),
    "g_q": lambda c: (c.hidden,),
    "w_q": lambda c: (c.n_q_heads * c.head_dim, c.hidden),
    "w_k": lambda c: (c.n_kv_heads * c.head_dim, c.hidden),
    "w_v": lambda c: (c.n_kv_heads * c.head_dim, c.hidden),
    "w_o": lambda c: (c.hidden, c.n_q_heads * c.head_dim),
    "g_mlp": lambda c: (c.hidden,),
    "w_gate": lambda c: (c.mlp_dim, c.hidden),
    "w_up": lambda c: (c.mlp_dim, c.hidden),
    "w_down": lambda c: (c.hidden, c.mlp_dim),
    "w_lm": lambda c: (c.vocab, c.hidden),
}


class OracleHead:
    """The draft head's parameters, widened to float64."""

    def __init__(self, cfg: HeadConfig, weights: Dict[str, np.ndarray]):
        if cfg.n_q_heads % cfg.n_kv_heads != 0:
            raise ValueError("n_q_heads must be a multiple of n_kv_heads")
        self.cfg = cfg
        for name, shape_of in _WEIGHT_SHAPES.items():
            w = np.asarray(weights[name], dtype=F64)
            if w.shape != shape_of(cfg):
                raise ValueError(f"{name}: shape {w.shape}, expected {shape_of(cfg)}")
            setattr(self, name, w)


    def with_storage(self, storage: Optional[str]) -> "OracleHead":
        """The same parameters (shared arrays) under another storage mode."""
        import copy
        from dataclasses import replace
        other = copy.copy(self)
        other.cfg = replace(self.cfg, storage=storage)
        return other


# --------------------------------------------------------------------------- primitives

def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bfloat16 (8 significand bits, ties to
    even), returned as float64.  The 64-bit pattern is rounded directly at the
    bf16 significand width, so there is no double rounding through float32.
    For finite inputs inside the bf16 normal range (all values met here)."""
    a = np.ascontiguousarray(a, dtype=F64)
    u = a.view(np.uint64)
    drop = np.uint64(52 - 7)                      # float64 keeps 52 fraction bits, bf16 keeps 7
    lsb = (u >> drop) & np.uint64(1)
    r = (u + ((np.uint64(1) << (drop - np.uint64(1))) - np.uint64(1)) + lsb) & ~((np.uint64(1) << drop) - np.uint64(1))
    return r.view(F64).reshape(a.shape)


def round_e4m3(a: np.ndarray) -> np.ndarray:
    """Round to the nearest FP8 E4M3 value (the OCP 8-bit format "e4m3fn": 4 exponent bits with bias 7, 3 fraction
    bits, no infinities, largest magnitude 448, subnormal step 2^-9), ties to even, magnitudes above 448 saturate
    to 448.  Returned as float64 (every E4M3 value is exactly representable)."""
    a = np.asarray(a, dtype=F64)
    mag = np.abs(a)
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(mag > 0, mag, 1.0)))
    e = np.maximum(e, -6.0)                               # below 2^-6 the spacing stays that of the subnormals
    step = np.exp2(e - 3.0)                               # 3 fraction bits
    q = np.rint(mag / step) * step                        # numpy rounds halves to even
    return np.sign(a) * np.minimum(q, 448.0)


def quantize_rows_e4m3(x: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Row-wise FP8 quantisation as the optional FP8 LM head uses it: scale_r = max|x_r| / 448 (1 for a zero row),
    q_r = round_e4m3(x_r / scale_r), so that x_r ~ scale_r * q_r.  The scale and the quotient are formed in IEEE
    float32: the code is an integer decision, and float32 is the precision in which FP8 scaling is stated wherever
    it is deployed (a float64 quotient that lies within 2^-24 of a rounding boundary would decide differently).
    Returns (q as float64 values, scale as float64)."""
    x32 = np.asarray(x, dtype=np.float32)
    amax = np.max(np.abs(x32), axis=-1, keepdims=True)
    scale = np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)
    q = round_e4m3((x32 / scale).astype(np.float32).astype(F64))
    return q, scale[..., 0].astype(F64)


def lm_head_fp8(head: "OracleHead", h: np.ndarray) -> np.ndarray:
    """Logits with the LM head's weights and the incoming states both quantised row-wise to FP8 E4M3:
    z[b, v] = scale_h[b] * scale_w[v] * sum_i q_h[b, i] q_w[v, i]."""
    qh, sh = quantize_rows_e4m3(np.asarray(h, dtype=F64))
    qw, sw = quantize_rows_e4m3(head.w_lm)
    return (qh @ qw.T) * sh[:, None] * sw[None, :]


def _stored(cfg: "HeadConfig", a: np.ndarray) -> np.ndarray:
    """A value as it is kept in memory under the configuration's storage mode."""
    if cfg.storage is None:
        return a
    if cfg.storage == "bf16":
        return round_bf16(a)
    raise ValueError(f"unknown storage mode {cfg.storage!r}")


def rms_norm(v: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """RMSNorm over the last axis: g * v / sqrt(mean(v^2) + eps)."""
    v = np.asarray(v, dtype=F64)
    ms = np.mean(v * v, axis=-1, keepdims=True)
    return g * (v / np.sqrt(ms + eps))


def silu(u: np.ndarray) -> np.ndarray:
    """SiLU(u) = u / (1 + exp(-u))."""
    u = np.asarray(u, dtype=F64)
    return u / (1.0 + np.exp(-u))


def rope_rotate(x: np.ndarray, pos: np.ndarray, theta: float, inverse: bool = False) -> np.ndarray:
    """Rotary position embedding, "rotate half": x [rows, H, d_h], pos [rows] (0-based); component i < d_h/2
    of every head pairs with component i + d_h/2 and the pair is rotated by pos * theta^(-2i/d_h)
    (by the opposite angle when ``inverse``: the transpose of the rotation)."""
    x = np.asarray(x, dtype=F64)
    half = x.shape[-1] // 2
    freq = F64(theta) ** (-2.0 * np.arange(half, dtype=F64) / x.shape[-1])
    ang = np.asarray(pos, dtype=F64)[:, None] * freq[None, :]
    if inverse:
        ang = -ang
    cs, sn = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cs - x2 * sn, x2 * cs + x1 * sn], axis=-1)


def argmax_lowest(z: np.ndarray) -> np.ndarray:
    """Arg-max over the last axis; ties go to the lowest index, NaN never wins
    (a row of NaNs gives 0)."""
    z = np.asarray(z, dtype=F64)
    z = np.where(np.isnan(z), -np.inf, z)
    return np.argmax(z, axis=-1).astype(np.int64)


def visible_true_count(p: int, block: int, offset: int) -> int:
    """Number of true states the query at (1-based) position p may read under
    the inverse block mask of Section 4.2 combined with the strict cross mask
    of Section 4.1.

    Positions p <= offset lie before the first window and are plain strict
    causal: keys 1..p-1.  Windows of size ``block`` tile the positions from
    ``offset`` on; a window that starts at n holds the queries n+1..n+block,
    and hides the keys n+1..n+block from all of them, so each of those queries
    reads keys 1..n.
    """
    if block < 1 or offset < 0 or p < 1:
        raise ValueError("bad mask arguments")
    if p <= offset:
        return p - 1
    return offset + block * ((p - 1 - offset) // block)


# --------------------------------------------------------------------------- Eq. 2

def project_kv(head: OracleHead, states: np.ndarray, pos: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """K_j = W_K^T h_j, V_j = W_V^T h_j for every row of ``states`` [n, d].
    Returns K, V of shape [n, Hkv, d_h]  (Eq. 2, first line).  ``pos`` [n]: 0-based positions of the
    states, needed (and used) only with the rotary option: K is rotated, V is not."""
    c = head.cfg
    s = np.asarray(states, dtype=F64).reshape(-1, c.hidden)
    k = _stored(c, s @ head.w_k.T).reshape(-1, c.n_kv_heads, c.head_dim)
    v = _stored(c, s @ head.w_v.T).reshape(-1, c.n_kv_heads, c.head_dim)
    if c.rope_theta > 0:
        if pos is None:
            raise ValueError("the rotary option needs the states' positions")
        k = _stored(c, rope_rotate(k, pos, c.rope_theta))
    return k, v


def attention_weights(head: OracleHead, q: np.ndarray, k_vis: np.ndarray) -> np.ndarray:
    """Softmax over the visible keys of <Q^h, K_j^h> / sqrt(d_h)  (Eq. 2, second
    line; only visible keys enter the softmax).  q: [Hq, d_h]; k_vis:
    [nv, Hkv, d_h]; returns [Hq, nv]."""
    c = head.cfg
    nv = k_vis.shape[0]
    w = np.zeros((c.n_q_heads, nv), dtype=F64)
    if nv == 0:
        return w
    for h in range(c.n_q_heads):
        kh = h // c.group
        a = (k_vis[:, kh, :] @ q[h]) / np.sqrt(F64(c.head_dim))
        a = a - np.max(a)
        e = np.exp(a)
        w[h] = e / np.sum(e)
    return w


def cross_attention(head: OracleHead, q: np.ndarray, k_vis: np.ndarray,
                    v_vis: np.ndarray) -> np.ndarray:
    """o^h = sum_j s^h_j V^h_j over the visible keys (Eq. 2, third line),
    heads concatenated to [Hq*d_h].  No visible key: o = 0."""
    c = head.cfg
    w = attention_weights(head, q, k_vis)
    o = np.zeros((c.n_q_heads, c.head_dim), dtype=F64)
    for h in range(c.n_q_heads):
        kh = h // c.group
        if k_vis.shape[0]:
            o[h] = w[h] @ v_vis[:, kh, :]
    return o.reshape(-1)


# --------------------------------------------------------------------------- Eq. 1

def embed_tokens(head: OracleHead, tokens: Sequence[int]) -> np.ndarray:
    """x = e(t_p): rows of the embedding table."""
    tok = np.asarray(tokens, dtype=np.int64).reshape(-1)
    if np.any(tok < 0) or np.any(tok >= head.cfg.vocab):
        raise ValueError("token id out of range")
    return head.embed[tok]


def query_projection(head: OracleHead, x: np.ndarray, pos: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """(xq, Q): xq = RMSNorm(x; g_q) (or x when the flag is off), Q = W_Q^T xq  (Eq. 2, first line);
    with the rotary option Q is rotated by the queries' 0-based positions ``pos``."""
    c = head.cfg
    xq = _stored(c, rms_norm(x, head.g_q, c.rms_eps)) if c.norm_q else np.asarray(x, dtype=F64)
    q = _stored(c, xq @ head.w_q.T)
    if c.rope_theta > 0:
        if pos is None:
            raise ValueError("the rotary option needs the queries' positions")
        q = _stored(c, rope_rotate(q.reshape(-1, c.n_q_heads, c.head_dim), pos, c.rope_theta).reshape(q.shape))
    return xq, q


def attention_rows(head: OracleHead, q: np.ndarray,
                   kv_vis: Sequence[Tuple[np.ndarray, np.ndarray]]) -> np.ndarray:
    """o for independent query rows: row r reads kv_vis[r] = (K, V) of its visible states."""
    c = head.cfg
    o = np.zeros((q.shape[0], c.n_q_heads * c.head_dim), dtype=F64)
    for r in range(q.shape[0]):
        k_vis, v_vis = kv_vis[r]
        o[r] = cross_attention(head, q[r].reshape(c.n_q_heads, c.head_dim), k_vis, v_vis)
    return _stored(c, o)


def output_projection(head: OracleHead, o: np.ndarray, x: np.ndarray) -> np.ndarray:
    """y = W_O^T [o^1..o^H] + e(t_p)  (Eq. 2 last line and the residual of Eq. 1)."""
    return _stored(head.cfg, o @ head.w_o.T + x)


def down_projection(head: OracleHead, act: np.ndarray, y: np.ndarray) -> np.ndarray:
    """h = W_down act + y: the MLP's last matrix and the residual of Eq. 1."""
    return _stored(head.cfg, np.asarray(act, dtype=F64) @ head.w_down.T + y)


def mlp_block(head: OracleHead, y: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """(yn, act, h): yn = RMSNorm(y; g_mlp), act = SiLU(W_gate yn) * (W_up yn), h = W_down act + y  (Eq. 1)."""
    c = head.cfg
    yn = _stored(c, rms_norm(y, head.g_mlp, c.rms_eps)) if c.norm_mlp else np.asarray(y, dtype=F64)
    act = _stored(c, silu(yn @ head.w_gate.T) * (yn @ head.w_up.T))
    return yn, act, down_projection(head, act, y)


def lm_head(head: OracleHead, h: np.ndarray) -> np.ndarray:
    """z = e^{-1}(h): the linear map to the vocabulary."""
    return np.asarray(h, dtype=F64) @ head.w_lm.T


def draft_block(head: OracleHead, tokens: Sequence[int],
                kv_vis: Sequence[Tuple[np.ndarray, np.ndarray]], pos: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """The draft Transformer block (Eq. 1) and the LM head for a set of
    independent query rows.  Row r has token ``tokens[r]`` and reads the
    visible keys/values ``kv_vis[r] = (K [nv,Hkv,d_h], V [nv,Hkv,d_h])``.

    Returns x (embeddings), q, o, y, h (the block output, also the state that
    is re-used as key/value input when drafting continues), logits z and the
    greedy token argmax z.
    """
    x = embed_tokens(head, tokens)                              # e(t_p)
    xq, q = query_projection(head, x, pos)                      # Q = W_Q^T e(t_p)   (pos: rotary option only)
    o = attention_rows(head, q, kv_vis)
    y = output_projection(head, o, x)                           # y = W_O^T[o] + e(t_p)
    yn, act, h = mlp_block(head, y)                             # h = MLP(y) + y
    z = lm_head(head, h)                                        # z = e^{-1}(h)
    return {"x": x, "xn": xq, "q": q, "o": o, "y": y, "yn": yn, "act": act, "h": h, "logits": z, "argmax": argmax_lowest(z)}


# --------------------------------------------------------------------------- serve-time drafting

class OracleSequence:
    """Key/value cache of one sequence: a prefix made from true (target)
    states and a tail made from the draft's own states (Section 4.1, last
    paragraphs: reuse cached K_j,V_j, append the new state's K,V when the next
    state is queried, reset to true states at the end of the SD iteration)."""

    def __init__(self, head: OracleHead):
        c = head.cfg
        self.k_true = np.zeros((0, c.n_kv_heads, c.head_dim), dtype=F64)
        self.v_true = np.zeros((0, c.n_kv_heads, c.head_dim), dtype=F64)
        self.k_draft: List[np.ndarray] = []
        self.v_draft: List[np.ndarray] = []
        self.pending_h: Optional[np.ndarray] = None   # previous step's h, not yet appended
        self.pending_token: Optional[int] = None      # previous step's greedy token
        self.steps = 0                                # draft steps since the cache was last reset to true states

    @property
    def n_true(self) -> int:
        return self.k_true.shape[0]

    @property
    def n_draft(self) -> int:
        return len(self.k_draft)


def rollback(seq: OracleSequence) -> None:
    """Reset the cache to true states only."""
    seq.k_draft, seq.v_draft = [], []
    seq.pending_h, seq.pending_token = None, None
    seq.steps = 0


def prefill_kv(head: OracleHead, seq: OracleSequence, hidden_rows: np.ndarray) -> None:
    """Drop the draft tail, then append K/V of new true states [r, d]."""
    rollback(seq)
    rows = np.asarray(hidden_rows, dtype=F64).reshape(-1, head.cfg.hidden)
    if rows.shape[0] == 0:
        return
    k, v = project_kv(head, rows, np.arange(seq.n_true, seq.n_true + rows.shape[0]))
    seq.k_true = np.concatenate([seq.k_true, k], axis=0)
    seq.v_true = np.concatenate([seq.v_true, v], axis=0)


def draft_step(head: OracleHead, seqs: Sequence[OracleSequence],
               tokens_in: Optional[Sequence[int]] = None, concat: bool = True) -> Dict[str, np.ndarray]:
    """One drafted token for each sequence.

    ``tokens_in`` None: each sequence continues from its previous step's greedy
    token.  ``concat`` true: the previous step's state h is projected and
    appended to the cache tail before attending (the paper's default); false:
    only true states are read and the previous state is discarded.
    """
    toks: List[int] = []
    kv: List[Tuple[np.ndarray, np.ndarray]] = []
    qpos: List[int] = []
    for b, seq in enumerate(seqs):
        if tokens_in is None:
            if seq.pending_token is None:
                raise ValueError("no previous draft token for this sequence")
            toks.append(int(seq.pending_token))
        else:
            toks.append(int(tokens_in[b]))
        # the s-th step since the reset queries position n + s (0-based n + s - 1); the previous step's state sits one before it
        if seq.pending_h is not None and concat:
            k, v = project_kv(head, seq.pending_h[None, :], np.array([seq.n_true + seq.steps - 1]))
            seq.k_draft.append(k[0])
            seq.v_draft.append(v[0])
        seq.pending_h = None
        qpos.append(seq.n_true + seq.steps)
        seq.steps += 1
        if seq.k_draft:
            k_vis = np.concatenate([seq.k_true, np.stack(seq.k_draft)], axis=0)
            v_vis = np.concatenate([seq.v_true, np.stack(seq.v_draft)], axis=0)
        else:
            k_vis, v_vis = seq.k_true, seq.v_true
        kv.append((k_vis, v_vis))
    out = draft_block(head, toks, kv, np.asarray(qpos))
    for b, seq in enumerate(seqs):
        seq.pending_h = out["h"][b].copy()
        seq.pending_token = int(out["argmax"][b])
    return out


# --------------------------------------------------------------------------- block-attention forward

def block_forward(head: OracleHead, tokens: Sequence[int], hidden: np.ndarray, block: int,
                  offset: int, sim_steps: int = 1,
                  positions: Optional[Iterable[int]] = None) -> Dict[str, np.ndarray]:
    """Block-attention forward over one sequence of S tokens and S true states
    (Section 4.2 and its mask figure).

    Simulation step 1 is the early-stage inverse block mask: the query at
    position p reads the true states 1..n, n = visible_true_count(p).  At
    simulation step i > 1 the state predicted at step i-1 for window slot i-1
    (position n+i-1) has been written into the key/value memory at that
    position, and the queries of the same window with slot >= i are recomputed
    with true states 1..n plus predicted states n+1..n+i-1.  No new queries are
    made: every query is the data token's embedding.  The reported output of a
    position is that of its last recomputation (step min(slot, sim_steps)).

    ``positions``: optional subset of 1-based positions to report (their
    window predecessors are computed as needed).  Returns arrays over the
    reported positions in ascending order: 'positions', 'hidden', 'logits',
    'argmax'.
    """
    c = head.cfg
    tok = np.asarray(tokens, dtype=np.int64).reshape(-1)
    S = tok.shape[0]
    hid = np.asarray(hidden, dtype=F64).reshape(S, c.hidden)
    if not (1 <= sim_steps <= block):
        raise ValueError("sim_steps must be in [1, block]")
    if not (0 <= offset < max(S, 1)):
        raise ValueError("offset must be in [0, S)")
    want = sorted(set(range(1, S + 1) if positions is None else (int(p) for p in positions)))
    if want and (want[0] < 1 or want[-1] > S):
        raise ValueError("position out of range")

    def slot_of(p: int) -> int:
        return p - visible_true_count(p, block, offset)   # 1 for p <= offset

    # closure: a reported position needs the predicted states of the earlier slots of its window
    need = set()
    for p in want:
        n, i = visible_true_count(p, block, offset), slot_of(p)
        for r in range(1, min(i, sim_steps)):
            need.add(n + r)
        need.add(p)
    active = sorted(need)

    k_true, v_true = project_kv(head, hid, np.arange(S))         # K_j, V_j of every true state
    k_pred: Dict[int, np.ndarray] = {}                           # position -> [Hkv, d_h]
    v_pred: Dict[int, np.ndarray] = {}
    result: Dict[int, Tuple[np.ndarray, np.ndarray, int]] = {}

    for step in range(1, sim_steps + 1):
        rows = [p for p in active if slot_of(p) >= step]
        if not rows:
            break
        kv = []
        for p in rows:
            n = visible_true_count(p, block, offset)
            ks = [k_true[:n]] + [k_pred[n + r][None] for r in range(1, step)]
            vs = [v_true[:n]] + [v_pred[n + r][None] for r in range(1, step)]
            kv.append((np.concatenate(ks, axis=0), np.concatenate(vs, axis=0)))
        out = draft_block(head, tok[[p - 1 for p in rows]], kv, np.asarray([p - 1 for p in rows]))
        for r, p in enumerate(rows):
            result[p] = (out["h"][r], out["logits"][r], int(out["argmax"][r]))
            if slot_of(p) == step and step < sim_steps:
                k, v = project_kv(head, out["h"][r][None, :], np.array([p - 1]))    # saved predicted state
                k_pred[p], v_pred[p] = k[0], v[0]

    pos = np.asarray(want, dtype=np.int64)
    return {
        "positions": pos,
        "hidden": np.stack([result[p][0] for p in want]) if want else np.zeros((0, c.hidden)),
        "logits": np.stack([result[p][1] for p in want]) if want else np.zeros((0, c.vocab)),
        "argmax": np.asarray([result[p][2] for p in want], dtype=np.int64),
    }


# --------------------------------------------------------------------------- greedy verification

def verify_greedy(draft_tokens: np.ndarray, target_logits: Optional[np.ndarray] = None,
                  target_ids: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Greedy draft/verify acceptance (Section 3): with target top-1 tokens
    g_1..g_{gamma+1} and drafts t_1..t_gamma, accept the longest prefix with
    t_r == g_r; emit g_1..g_{a+1} (the accepted drafts equal the target's
    tokens, plus the one extra target token).  Returns accept_len [B] and
    out_tokens [B, gamma+1] padded with -1; tau = accept_len + 1.
    """
    draft = np.asarray(draft_tokens, dtype=np.int64)
    B, gamma = draft.shape
    if (target_logits is None) == (target_ids is None):
        raise ValueError("give exactly one of target_logits / target_ids")
    if target_ids is None:
        g = argmax_lowest(np.asarray(target_logits, dtype=F64).reshape(B, gamma + 1, -1))
    else:
        g = np.asarray(target_ids, dtype=np.int64).reshape(B, gamma + 1)
    accept = np.zeros(B, dtype=np.int64)
    out = np.full((B, gamma + 1), -1, dtype=np.int64)
    for b in range(B):
        a = 0
        while a < gamma and draft[b, a] == g[b, a]:
            a += 1
        accept[b] = a
        out[b, : a + 1] = g[b, : a + 1]
    return accept, out


# --------------------------------------------------------------------------- speculative-sampling verification

def softmax_rows(logits: np.ndarray, temperature: float = 1.0) -> np.ndarray:
    """softmax(z / temperature) over the last axis, with max-subtraction."""
    z = np.asarray(logits, dtype=F64) / F64(temperature)
    z = z - np.max(z, axis=-1, keepdims=True)
    e = np.exp(z)
    return e / np.sum(e, axis=-1, keepdims=True)


def residual_distribution(p: np.ndarray, q: Optional[np.ndarray]) -> np.ndarray:
    """The distribution the extra token is drawn from (Section 3): normalised
    max(0, p - q) at a rejection; p itself after gamma acceptances, where no
    draft distribution exists.  If p == q everywhere (no mass left, a case that
    cannot follow a rejection) it falls back to p."""
    p = np.asarray(p, dtype=F64)
    if q is None:
        return p / np.sum(p)
    w = np.maximum(0.0, p - np.asarray(q, dtype=F64))
    s = np.sum(w)
    return w / s if s > 0.0 else p / np.sum(p)


def inverse_cdf(dist: np.ndarray, r: float) -> Tuple[int, float]:
    """Token drawn from ``dist`` with the uniform r in [0, 1): the smallest v
    whose cumulative mass exceeds r.  Also returns how far r lies from the
    nearest cumulative boundary (the decision margin of this draw)."""
    c = np.cumsum(np.asarray(dist, dtype=F64))
    c[-1] = max(c[-1], 1.0)
    v = int(np.searchsorted(c, r, side="right"))
    v = min(v, len(c) - 1)
    lo = c[v - 1] if v > 0 else 0.0
    return v, float(min(r - lo, c[v] - r))


def verify_sample(draft_tokens: np.ndarray, draft_logits: np.ndarray, target_logits: np.ndarray,
                  u_accept: np.ndarray, u_resample: np.ndarray,
                  temperature: float = 1.0) -> Dict[str, np.ndarray]:
    """Lossless draft/verify acceptance under sampling (Section 3).

    For one SD iteration of B sequences: drafts t_1..t_gamma [B, gamma], the
    draft's logits at those positions [gamma, B, V] (one block per draft step),
    the target's logits at positions 1..gamma+1 [B, gamma+1, V], and the random
    numbers the method draws, passed in: u_accept [B, gamma] and u_resample [B],
    uniform in [0, 1).  With p_i = softmax(target_i / T), q_i = softmax(draft_i / T):
    draft i is accepted iff u_accept[i] < min(1, p_i(t_i) / q_i(t_i)); at the first
    rejection j (or j = gamma + 1) one token is drawn by inverse CDF with
    u_resample from the normalised max(0, p_j - q_j) (from p_{gamma+1} when
    nothing was rejected).

    Returns accept_len [B]; out_tokens [B, gamma+1] = the accepted drafts, the
    extra token, then -1; and the decision margins accept_margin [B] (smallest
    |u - ratio| over the tests made) and resample_margin [B] (distance of
    u_resample to the nearest CDF boundary), which tell a checker where another
    floating-point precision may legitimately decide otherwise.
    """
    draft = np.asarray(draft_tokens, dtype=np.int64)
    B, gamma = draft.shape
    pl = np.asarray(target_logits, dtype=F64).reshape(B, gamma + 1, -1)
    ql = np.asarray(draft_logits, dtype=F64).reshape(gamma, B, pl.shape[-1])
    ua = np.asarray(u_accept, dtype=F64).reshape(B, gamma)
    ur = np.asarray(u_resample, dtype=F64).reshape(B)
    accept = np.zeros(B, dtype=np.int64)
    out = np.full((B, gamma + 1), -1, dtype=np.int64)
    am = np.full(B, np.inf)
    rm = np.zeros(B)
    for b in range(B):
        p = softmax_rows(pl[b], temperature)                         # [gamma+1, V]
        q = softmax_rows(ql[:, b, :], temperature) if gamma else np.zeros((0, p.shape[1]))
        a = 0
        while a < gamma:
            t = int(draft[b, a])
            ratio = min(1.0, p[a, t] / q[a, t]) if q[a, t] > 0.0 else 1.0
            am[b] = min(am[b], abs(ua[b, a] - ratio) if ratio < 1.0 else np.inf)
            if not (ua[b, a] < ratio):
                break
            a += 1
        accept[b] = a
        out[b, :a] = draft[b, :a]
        dist = residual_distribution(p[a], q[a] if a < gamma else None)
        out[b, a], rm[b] = inverse_cdf(dist, ur[b])
    return {"accept_len": accept, "out_tokens": out, "accept_margin": am, "resample_margin": rm}


# --------------------------------------------------------------------------- block-attention training losses (forward)

def cross_entropy_rows(draft_logits: np.ndarray, target_logits: Optional[np.ndarray] = None,
                       target_ids: Optional[np.ndarray] = None) -> np.ndarray:
    """-E_{t ~ p}[log q(t)] per row, q = softmax(draft_logits); p = softmax(target_logits),
    or the point mass at target_ids (exactly one of the two is given)."""
    z = np.asarray(draft_logits, dtype=F64)
    m = np.max(z, axis=-1, keepdims=True)
    logq = z - (m + np.log(np.sum(np.exp(z - m), axis=-1, keepdims=True)))
    if (target_logits is None) == (target_ids is None):
        raise ValueError("give exactly one of target_logits / target_ids")
    if target_ids is not None:
        ids = np.asarray(target_ids, dtype=np.int64).reshape(-1)
        return -logq[np.arange(logq.shape[0]), ids]
    return -np.sum(softmax_rows(target_logits) * logq, axis=-1)


def loss_weights(S: int, block: int, offset: int, sim_steps: int, stage: str) -> Tuple[np.ndarray, int]:
    """Weight of every (1-based) position's loss term and the number of windows N.

    Positions p <= offset lie in no window and carry no term.  In a window starting at n the
    query at p = n + i is the i-step-ahead prediction.  'early' (Eq. 4): every window position
    counts once.  'late' (Eq. 7 with l = i and beta*_{i,i} = k - i + 1): the slot-i prediction made
    at simulation step i counts k - i + 1 times for i <= sim_steps and not at all beyond.
    """
    if stage not in ("early", "late"):
        raise ValueError(stage)
    w = np.zeros(S, dtype=F64)
    for p in range(offset + 1, S + 1):
        i = p - visible_true_count(p, block, offset)
        if stage == "early":
            w[p - 1] = 1.0
        elif i <= sim_steps:
            w[p - 1] = block - i + 1
    n_windows = -(-(S - offset) // block)
    return w, n_windows


def block_loss(head: OracleHead, tokens: np.ndarray, hidden: np.ndarray, block: int, offset: int, stage: str,
               sim_steps: int = 1, target_logits: Optional[np.ndarray] = None,
               target_ids: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Early-stage (Eq. 4) or late-stage (Eq. 7) loss of a batch of sequences, forward only.

    tokens [B, S], hidden [B, S, d]; the target model's distribution at position p (it predicts
    token p+1, like the draft state at p, Eq. 1) is softmax(target_logits[b, p-1]) or the point
    mass at target_ids[b, p-1].  Early stage: sim_steps must be 1.  Returns 'ce' [B, S] (every
    position's cross-entropy from the block forward), 'weights' [S], 'n_windows' and
    'loss' = sum_b sum_p weights[p] ce[b, p] / (B * n_windows).
    """
    tok = np.asarray(tokens, dtype=np.int64)
    B, S = tok.shape
    if stage == "early" and sim_steps != 1:
        raise ValueError("the early-stage loss uses the plain inverse block mask (sim_steps = 1)")
    w, n_windows = loss_weights(S, block, offset, sim_steps, stage)
    ce = np.zeros((B, S), dtype=F64)
    for b in range(B):
        out = block_forward(head, tok[b], np.asarray(hidden)[b], block, offset, sim_steps)
        ce[b] = cross_entropy_rows(out["logits"],
                                   None if target_logits is None else np.asarray(target_logits)[b],
                                   None if target_ids is None else np.asarray(target_ids)[b])
    return {"ce": ce, "weights": w, "n_windows": n_windows, "loss": float(np.sum(ce * w[None, :]) / (B * n_windows))}


# --------------------------------------------------------------------------- block-attention training step: loss and gradients

def smooth_l1(r: np.ndarray) -> np.ndarray:
    """Smooth-L1 (Huber, threshold 1) element-wise: r^2 / 2 for |r| < 1, |r| - 1/2 otherwise.  The
    hidden-state regression term that Appendix B adds to both training stages is the one of the
    EAGLE papers, which is this function averaged over elements."""
    r = np.asarray(r, dtype=F64)
    a = np.abs(r)
    return np.where(a < 1.0, 0.5 * r * r, a - 0.5)


def rms_norm_backward(v: np.ndarray, g: np.ndarray, eps: float, dn: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """(dv, dg) of n = g * v * r, r = (mean(v^2) + eps)^(-1/2), row by row."""
    v = np.asarray(v, dtype=F64)
    r = 1.0 / np.sqrt(np.mean(v * v, axis=-1, keepdims=True) + eps)
    gd = g * dn
    dv = r * gd - v * (r ** 3) * np.mean(v * gd, axis=-1, keepdims=True)
    return dv, np.sum(dn * v * r, axis=0)


def block_loss_grad(head: OracleHead, tokens: np.ndarray, hidden: np.ndarray, block: int, offset: int, stage: str,
                    sim_steps: int = 1, target_logits: Optional[np.ndarray] = None,
                    target_ids: Optional[np.ndarray] = None, vloss_coef: float = 0.0) -> Dict[str, object]:
    """One training step's loss and its gradient with respect to every parameter of the head.

    total = L + vloss_coef * vloss, L the early (Eq. 4) or late (Eq. 7) loss of ``block_loss``;
    vloss = mean over the positions that carry a loss term (weight > 0) and over the d components of
    smooth_l1(h_hat_p - h_p): the draft state at p regresses on the target's true state at p, whose
    place it takes as a key/value input when drafting continues (Section 4.1).

    Gradient flow under simulation (the paper does not spell it out): the states predicted at
    earlier simulation steps enter the final step as key/value INPUTS, exactly as the true states
    they replace do, and are constants of the differentiation; W_K and W_V receive the gradient of
    projecting them.  With sim_steps = 1 there is no predicted state and nothing is cut.

    Returns 'loss' (the L term), 'vloss', 'total', and 'grads': name -> array shaped like the
    parameter (embed, g_q, w_q, w_k, w_v, w_o, g_mlp, w_gate, w_up, w_down, w_lm).
    """
    c = head.cfg
    tok = np.asarray(tokens, dtype=np.int64)
    B, S = tok.shape
    hid_all = np.asarray(hidden, dtype=F64).reshape(B, S, c.hidden)
    if stage == "early" and sim_steps != 1:
        raise ValueError("the early-stage loss uses the plain inverse block mask (sim_steps = 1)")
    w, n_windows = loss_weights(S, block, offset, sim_steps, stage)
    n_reg = B * int(np.count_nonzero(w))
    grads = {name: np.zeros(shape_of(c), dtype=F64) for name, shape_of in _WEIGHT_SHAPES.items()}
    loss = 0.0
    vloss = 0.0
    inv_sqrt = 1.0 / np.sqrt(F64(c.head_dim))
    G = c.group
    for b in range(B):
        hid = hid_all[b]
        # the states that earlier simulation steps wrote in place: constants of this step
        h_pred = block_forward(head, tok[b], hid, block, offset, sim_steps)["hidden"] if sim_steps > 1 else None
        k_true, v_true = project_kv(head, hid, np.arange(S))
        if h_pred is not None:
            k_pred, v_pred = project_kv(head, h_pred, np.arange(S))
        kv, src = [], []                                    # per position: visible (K, V) and where each row came from
        for p in range(1, S + 1):
            n = visible_true_count(p, block, offset)
            extra = list(range(n, n + min(p - n, sim_steps) - 1))        # 0-based rows of predicted states
            if extra:
                kv.append((np.concatenate([k_true[:n], k_pred[extra]]), np.concatenate([v_true[:n], v_pred[extra]])))
            else:
                kv.append((k_true[:n], v_true[:n]))
            src.append((n, extra))
        f = draft_block(head, tok[b], kv, np.arange(S))
        x, xn, q, o, y, yn, h, z = f["x"], f["xn"], f["q"], f["o"], f["y"], f["yn"], f["h"], f["logits"]
        gate, up = yn @ head.w_gate.T, yn @ head.w_up.T
        sig = 1.0 / (1.0 + np.exp(-gate))
        act = gate * sig * up
        # loss terms
        qd = softmax_rows(z)
        if target_ids is not None:
            pd = np.zeros_like(qd)
            pd[np.arange(S), np.asarray(target_ids, dtype=np.int64)[b]] = 1.0
        else:
            pd = softmax_rows(np.asarray(target_logits, dtype=F64)[b])
        ce = cross_entropy_rows(z, None if target_logits is None else np.asarray(target_logits)[b],
                                None if target_ids is None else np.asarray(target_ids)[b])
        coef = w / (B * n_windows)
        loss += float(np.sum(coef * ce))
        dz = coef[:, None] * (qd - pd)
        reg = (w > 0).astype(F64)[:, None]
        resid = h - hid
        dh = dz @ head.w_lm
        if n_reg > 0:
            vloss += float(np.sum(reg * smooth_l1(resid)) / (n_reg * c.hidden))
            dh = dh + vloss_coef * reg * np.clip(resid, -1.0, 1.0) / (n_reg * c.hidden)
        grads["w_lm"] += dz.T @ h
        # h = y + W_down act
        grads["w_down"] += dh.T @ act
        dact = dh @ head.w_down
        dgate = dact * up * (sig * (1.0 + gate * (1.0 - sig)))
        dup = dact * gate * sig
        grads["w_gate"] += dgate.T @ yn
        grads["w_up"] += dup.T @ yn
        dyn = dgate @ head.w_gate + dup @ head.w_up
        if c.norm_mlp:
            dy_n, dg = rms_norm_backward(y, head.g_mlp, c.rms_eps, dyn)
            grads["g_mlp"] += dg
        else:
            dy_n = dyn
        dy = dh + dy_n
        # y = W_O o + x
        grads["w_o"] += dy.T @ o
        do = (dy @ head.w_o).reshape(S, c.n_q_heads, c.head_dim)
        dq = np.zeros((S, c.n_q_heads, c.head_dim), dtype=F64)
        dk_true = np.zeros_like(k_true); dv_true = np.zeros_like(v_true)
        dk_pred = np.zeros_like(k_true); dv_pred = np.zeros_like(v_true)
        qh = q.reshape(S, c.n_q_heads, c.head_dim)
        for r in range(S):
            k_vis, v_vis = kv[r]
            nv = k_vis.shape[0]
            if nv == 0:
                continue
            wts = attention_weights(head, qh[r], k_vis)                  # [Hq, nv]
            dk_vis = np.zeros_like(k_vis); dv_vis = np.zeros_like(v_vis)
            for hh in range(c.n_q_heads):
                kh = hh // G
                dp = v_vis[:, kh, :] @ do[r, hh]
                ds = wts[hh] * (dp - np.dot(wts[hh], dp))
                dq[r, hh] = (ds @ k_vis[:, kh, :]) * inv_sqrt
                dk_vis[:, kh, :] += np.outer(ds, qh[r, hh]) * inv_sqrt
                dv_vis[:, kh, :] += np.outer(wts[hh], do[r, hh])
            n, extra = src[r]
            dk_true[:n] += dk_vis[:n]; dv_true[:n] += dv_vis[:n]
            for t, row in enumerate(extra):
                dk_pred[row] += dk_vis[n + t]; dv_pred[row] += dv_vis[n + t]
        if c.rope_theta > 0:        # back through the rotations (orthogonal: the transpose is the opposite angle)
            dq = rope_rotate(dq, np.arange(S), c.rope_theta, inverse=True)
            dk_true = rope_rotate(dk_true, np.arange(S), c.rope_theta, inverse=True)
            dk_pred = rope_rotate(dk_pred, np.arange(S), c.rope_theta, inverse=True)
        kd = c.n_kv_heads * c.head_dim
        grads["w_k"] += dk_true.reshape(S, kd).T @ hid
        grads["w_v"] += dv_true.reshape(S, kd).T @ hid
        if h_pred is not None:
            grads["w_k"] += dk_pred.reshape(S, kd).T @ h_pred
            grads["w_v"] += dv_pred.reshape(S, kd).T @ h_pred
        dq2 = dq.reshape(S, -1)
        grads["w_q"] += dq2.T @ xn
        dxn = dq2 @ head.w_q
        if c.norm_q:
            dx_n, dg = rms_norm_backward(x, head.g_q, c.rms_eps, dxn)
            grads["g_q"] += dg
        else:
            dx_n = dxn
        dx = dy + dx_n
        np.add.at(grads["embed"], tok[b], dx)
    return {"loss": loss, "vloss": vloss, "total": loss + vloss_coef * vloss, "grads": grads}


# --------------------------------------------------------------------------- dynamic draft tree (EAGLE-2's method, which the paper adopts)

def log_softmax_rows(logits: np.ndarray) -> np.ndarray:
    z = np.asarray(logits, dtype=F64)
    m = np.max(z, axis=-1, keepdims=True)
    return z - (m + np.log(np.sum(np.exp(z - m), axis=-1, keepdims=True)))


def top_k_lowest(values: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest values, largest first; equal values in index order."""
    v = np.asarray(values, dtype=F64)
    order = np.lexsort((np.arange(v.shape[0]), -v))
    return order[:k]


def draft_tree(head: OracleHead, seq: OracleSequence, root_token: int, depth: int, topk: int,
               n_candidates: int) -> Dict[str, np.ndarray]:
    """Dynamic draft tree over the true states cached in ``seq`` (the experimental setup's
    "dynamic draft attention tree": depth = 1 + ``depth`` forwards, ``topk`` children per node,
    ``n_candidates`` nodes handed to verification).

    The root token is forwarded first; its ``topk`` most likely next tokens become the first
    frontier, each scored by its log-probability.  ``depth`` times: every frontier node is forwarded
    -- its query is its token's embedding, and it reads the true states plus the draft states of
    the root and of its own ancestors (concatenation of newly generated states, Section 4.1) --
    and proposes its ``topk`` children with score = own score + log-probability; the ``topk`` best
    of all children form the next frontier.  Finally the ``n_candidates`` best nodes overall are
    kept (a parent never scores below its child, so they form a tree).  Ties go to the smaller
    token id / the earlier node.

    Returns tokens [N], parents [N] (index into the returned arrays, -1 = child of the root),
    scores [N], depths [N] (1 = child of the root), in creation order, and for every frontier
    forward the rows it ran: 'forward_nodes' (list of arrays of node ids, in all-node numbering)
    with 'all_tokens', 'all_parents', 'all_scores' of every node ever created.  'cut_margin' is the
    smallest score gap across any of the selections made (k-th against (k+1)-th child, frontier,
    final n-th against (n+1)-th): below it another floating-point precision may select otherwise.
    """
    c = head.cfg
    k_true, v_true = seq.k_true, seq.v_true
    margin = [np.inf]

    def cut(values, k):
        v = np.sort(np.asarray(values, dtype=F64))[::-1]
        if k < len(v):
            margin[0] = min(margin[0], float(v[k - 1] - v[k]))

    n_true = k_true.shape[0]

    def forward(tokens, state_lists):
        # a row that reads a draft states after the true ones is the token at 0-based position n_true + a
        kv = []
        for states in state_lists:
            if states:
                k, v = project_kv(head, np.stack(states), n_true + np.arange(len(states)))
                kv.append((np.concatenate([k_true, k]), np.concatenate([v_true, v])))
            else:
                kv.append((k_true, v_true))
        return draft_block(head, tokens, kv, np.asarray([n_true + len(st) for st in state_lists]))

    out = forward([int(root_token)], [[]])
    h_root = out["h"][0]
    logq = log_softmax_rows(out["logits"][0])
    cut(logq, topk)
    first = top_k_lowest(logq, topk)
    tok = [int(t) for t in first]
    par = [-1] * topk
    sc = [float(logq[t]) for t in first]
    dep = [1] * topk
    state_of: Dict[int, np.ndarray] = {}            # node id -> its draft state h (only forwarded nodes)
    frontier = list(range(topk))
    forwards = []
    for _ in range(depth):
        lists = []
        for f in frontier:
            chain = []
            a = par[f]
            while a >= 0:
                chain.append(state_of[a])
                a = par[a]
            lists.append([h_root] + chain[::-1])
        out = forward([tok[f] for f in frontier], lists)
        forwards.append(np.asarray(frontier))
        lq = log_softmax_rows(out["logits"])
        base = len(tok)
        for r, f in enumerate(frontier):
            state_of[f] = out["h"][r]
            cut(lq[r], topk)
            for t in top_k_lowest(lq[r], topk):
                tok.append(int(t)); par.append(f); sc.append(sc[f] + float(lq[r, t])); dep.append(dep[f] + 1)
        new = np.arange(base, len(tok))
        cut(np.asarray(sc)[new], topk)
        frontier = [int(new[i]) for i in top_k_lowest(np.asarray(sc)[new], topk)]
    cut(sc, min(n_candidates, len(tok)))
    keep = np.sort(top_k_lowest(np.asarray(sc), min(n_candidates, len(tok))))
    remap = {int(n): i for i, n in enumerate(keep)}
    return {
        "tokens": np.asarray([tok[n] for n in keep], dtype=np.int64),
        "parents": np.asarray([remap[par[n]] if par[n] >= 0 else -1 for n in keep], dtype=np.int64),
        "scores": np.asarray([sc[n] for n in keep], dtype=F64),
        "depths": np.asarray([dep[n] for n in keep], dtype=np.int64),
        "all_tokens": np.asarray(tok, dtype=np.int64), "all_parents": np.asarray(par, dtype=np.int64),
        "all_scores": np.asarray(sc, dtype=F64), "forward_nodes": forwards, "kept_nodes": keep, "cut_margin": margin[0],
    }


def verify_tree_greedy(tokens: np.ndarray, parents: np.ndarray, target_root_id: int,
                       target_ids: np.ndarray) -> Tuple[int, np.ndarray, np.ndarray]:
    """Greedy acceptance on a draft tree (Section 3 applied along the tree's paths): starting at
    the root, follow the child whose token equals the target's top-1 token at the current node
    (``target_root_id`` at the root, ``target_ids[n]`` after node n); stop when no child matches
    and emit the target's token there.  Returns (accept_len, emitted tokens, accepted node ids)."""
    tokens = np.asarray(tokens, dtype=np.int64)
    parents = np.asarray(parents, dtype=np.int64)
    cur, want = -1, int(target_root_id)
    path, out = [], []
    while True:
        nxt = [n for n in range(len(tokens)) if parents[n] == cur and tokens[n] == want]
        if not nxt:
            break
        cur = nxt[0]
        path.append(cur)
        out.append(want)
        want = int(np.asarray(target_ids)[cur])
    out.append(want)
    return len(path), np.asarray(out, dtype=np.int64), np.asarray(path, dtype=np.int64)
