"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each one names the passage it
leans on; together they are chosen so that a dropped term, a wrong sign or
index, or a transposed operand in the oracle fails at least one of them.
"""
import math
import os

import numpy as np
import pytest

import oracle as O
from paper_2505_24544_b200 import workloads as WL

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_head(seed=0, d=32, hq=4, hkv=2, dh=8, m=48, V=50, std=0.3, **kw):
    rng = np.random.default_rng(seed)
    cfg = O.HeadConfig(d, hq, hkv, dh, m, V, **kw)
    w = {
        "embed": rng.normal(0, 1.0, (V, d)),
        "g_q": 1 + rng.normal(0, 0.1, d),
        "w_q": rng.normal(0, std, (hq * dh, d)),
        "w_k": rng.normal(0, std, (hkv * dh, d)),
        "w_v": rng.normal(0, std, (hkv * dh, d)),
        "w_o": rng.normal(0, std, (d, hq * dh)),
        "g_mlp": 1 + rng.normal(0, 0.1, d),
        "w_gate": rng.normal(0, std, (m, d)),
        "w_up": rng.normal(0, std, (m, d)),
        "w_down": rng.normal(0, std, (d, m)),
        "w_lm": rng.normal(0, std, (V, d)),
    }
    return O.OracleHead(cfg, w), w, rng


# ----------------------------------------------------------------------------- hand-worked case

def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals])
    return out


def tiny_head():
    ln3, ln7, s2 = math.log(3.0), math.log(7.0), math.sqrt(2.0)
    cfg = O.HeadConfig(hidden=2, n_q_heads=2, n_kv_heads=1, head_dim=2, mlp_dim=2, vocab=3, rms_eps=0.0)
    w = {
        "embed": [[1, 1], [1, -1], [s2, 0]],
        "g_q": [2, 0.5],
        "w_q": [[1, 4], [ln3 / (2 * s2), 0], [s2 * ln7 / 2, 0], [1, 4]],
        "w_k": [[0, 1], [2, 0]],
        "w_v": [[1, 2], [3, 4]],
        "w_o": [[1, -1, 0, 0], [0, 0, -1, 1]],
        "g_mlp": [0.5, 2],
        "w_gate": [[0, ln3 / 2], [2 * ln3, 0]],
        "w_up": [[2, 1], [4, 0]],
        "w_down": [[1, 1], [2, -2]],
        "w_lm": [[1, 0], [0, 1], [1, 1]],
    }
    return O.OracleHead(cfg, {k: np.array(v, dtype=float) for k, v in w.items()})


def test_hand_worked_draft_step_matches_golden():
    """Eq. 1-2 and the LM head on the pencil-and-paper instance (serve-time path)."""
    g = read_golden("tiny_head.txt")
    head = tiny_head()
    seq = O.OracleSequence(head)
    O.prefill_kv(head, seq, np.array([[1.0, 0.0], [0.0, 1.0]]))
    out = O.draft_step(head, [seq], tokens_in=[1])
    q = out["q"][0].reshape(2, 2)
    w = O.attention_weights(head, q, seq.k_true)
    np.testing.assert_allclose(w[0], g["attn_head1"], atol=1e-15)
    np.testing.assert_allclose(w[1], g["attn_head2"], atol=1e-15)
    np.testing.assert_allclose(out["o"][0], g["o"], atol=1e-14)
    np.testing.assert_allclose(out["y"][0], g["y"], atol=1e-14)
    np.testing.assert_allclose(out["h"][0], g["h"], atol=1e-14)
    np.testing.assert_allclose(out["logits"][0], g["z"], atol=1e-14)
    assert int(out["argmax"][0]) == int(g["argmax"][0])


def test_hand_worked_block_forward_hides_diagonal():
    """Same instance through the block path: the query at position 3 must not
    read h_3 (Mask_{i,j} = 0 for j >= i, Section 4.1)."""
    g = read_golden("tiny_head.txt")
    head = tiny_head()
    hidden = np.array([[1.0, 0.0], [0.0, 1.0], [5.0, 5.0]])
    out = O.block_forward(head, tokens=[0, 2, 1], hidden=hidden, block=1, offset=0, sim_steps=1, positions=[3])
    np.testing.assert_allclose(out["hidden"][0], g["h"], atol=1e-14)
    np.testing.assert_allclose(out["logits"][0], g["z"], atol=1e-14)
    assert int(out["argmax"][0]) == 2


# ----------------------------------------------------------------------------- softmax invariants

def test_attention_rows_sum_to_one_and_shift_invariance():
    """Rows of s_{i,j} over the visible keys are probability vectors; adding
    one vector to every key shifts every score of a head by the same amount and
    so leaves the softmax unchanged (Eq. 2, second line)."""
    head, _, rng = small_head(1)
    c = head.cfg
    q = rng.normal(0, 2.0, (c.n_q_heads, c.head_dim))
    k = rng.normal(0, 2.0, (37, c.n_kv_heads, c.head_dim))
    w = O.attention_weights(head, q, k)
    assert w.shape == (c.n_q_heads, 37)
    assert np.all(w >= 0)
    np.testing.assert_allclose(w.sum(axis=1), 1.0, atol=1e-12)
    shift = rng.normal(0, 3.0, (1, c.n_kv_heads, c.head_dim))
    np.testing.assert_allclose(O.attention_weights(head, q, k + shift), w, atol=1e-12)
    # the scale 1/sqrt(d_h): a single dominating score ratio, checked against the scalar formula
    q1 = np.zeros_like(q); q1[0, 0] = 1.0
    k2 = np.zeros((2, c.n_kv_heads, c.head_dim)); k2[0, 0, 0] = 3.0
    w2 = O.attention_weights(head, q1, k2)
    expect = 1.0 / (1.0 + math.exp(-3.0 / math.sqrt(c.head_dim)))
    assert abs(w2[0, 0] - expect) < 1e-15


def test_single_key_and_identical_keys():
    """One visible key: o = V_1.  Identical keys: o = mean of the values."""
    head, _, rng = small_head(2)
    c = head.cfg
    q = rng.normal(size=(c.n_q_heads, c.head_dim))
    k = rng.normal(size=(1, c.n_kv_heads, c.head_dim))
    v = rng.normal(size=(1, c.n_kv_heads, c.head_dim))
    o = O.cross_attention(head, q, k, v).reshape(c.n_q_heads, c.head_dim)
    for h in range(c.n_q_heads):
        np.testing.assert_allclose(o[h], v[0, h // c.group], atol=1e-15)
    k5 = np.repeat(k, 5, axis=0)
    v5 = rng.normal(size=(5, c.n_kv_heads, c.head_dim))
    o5 = O.cross_attention(head, q, k5, v5).reshape(c.n_q_heads, c.head_dim)
    for h in range(c.n_q_heads):
        np.testing.assert_allclose(o5[h], v5[:, h // c.group].mean(axis=0), atol=1e-14)


def test_no_visible_key_gives_embedding_path_only():
    """Position 1 has no key: o = 0, y = e(t)."""
    head, w, rng = small_head(3)
    seq = O.OracleSequence(head)
    out = O.draft_step(head, [seq], tokens_in=[7])
    np.testing.assert_array_equal(out["o"][0], 0.0)
    np.testing.assert_allclose(out["y"][0], w["embed"][7], atol=0)


def test_zero_output_projections_reduce_to_embedding_times_lm_head():
    """W_O = 0 and W_down = 0 remove both sub-layers: z = W_lm e(t) (Eq. 1 residual paths)."""
    head, w, rng = small_head(4)
    w = dict(w); w["w_o"] = np.zeros_like(w["w_o"]); w["w_down"] = np.zeros_like(w["w_down"])
    head0 = O.OracleHead(head.cfg, w)
    seq = O.OracleSequence(head0)
    O.prefill_kv(head0, seq, rng.normal(size=(9, head.cfg.hidden)))
    out = O.draft_step(head0, [seq], tokens_in=[11])
    np.testing.assert_allclose(out["logits"][0], w["w_lm"] @ w["embed"][11], atol=1e-13)


def test_gqa_equals_mha_with_repeated_kv_heads():
    """Grouped-query attention equals multi-head attention whose key/value
    head weights are each repeated Hq/Hkv times."""
    head, w, rng = small_head(5, hq=6, hkv=2, dh=4)
    c = head.cfg
    rep = lambda a: np.repeat(a.reshape(c.n_kv_heads, c.head_dim, c.hidden), c.group, axis=0).reshape(-1, c.hidden)
    w_mha = dict(w); w_mha["w_k"] = rep(w["w_k"]); w_mha["w_v"] = rep(w["w_v"])
    head_mha = O.OracleHead(O.HeadConfig(c.hidden, c.n_q_heads, c.n_q_heads, c.head_dim, c.mlp_dim, c.vocab), w_mha)
    states = rng.normal(size=(13, c.hidden))
    outs = []
    for hd in (head, head_mha):
        seq = O.OracleSequence(hd)
        O.prefill_kv(hd, seq, states)
        outs.append(O.draft_step(hd, [seq], tokens_in=[3]))
    np.testing.assert_allclose(outs[0]["logits"], outs[1]["logits"], atol=1e-12)
    np.testing.assert_allclose(outs[0]["o"], outs[1]["o"], atol=1e-13)


def test_norm_flags_and_rmsnorm_definition():
    """RMSNorm(v) has unit mean square when g = 1, eps = 0; flags switch it off."""
    rng = np.random.default_rng(6)
    v = rng.normal(size=(5, 17)) * 3.0
    n = O.rms_norm(v, np.ones(17), 0.0)
    np.testing.assert_allclose((n * n).mean(axis=1), 1.0, atol=1e-13)
    np.testing.assert_allclose(n * np.sqrt((v * v).mean(axis=1, keepdims=True)), v, atol=1e-12)
    # eps enters under the root: v = 0 stays 0 and a constant vector c gives c/sqrt(c^2+eps)
    assert abs(O.rms_norm(np.full(4, 2.0), np.ones(4), 5.0)[0] - 2.0 / 3.0) < 1e-15
    head, w, _ = small_head(7, norm_q=False, norm_mlp=False)
    w1 = dict(w); w1["g_q"] = w["g_q"] * 9.0; w1["g_mlp"] = w["g_mlp"] * -2.0
    a = O.draft_block(head, [1], [(np.zeros((0, 2, 8)), np.zeros((0, 2, 8)))])
    b = O.draft_block(O.OracleHead(head.cfg, w1), [1], [(np.zeros((0, 2, 8)), np.zeros((0, 2, 8)))])
    np.testing.assert_array_equal(a["logits"], b["logits"])


def test_silu_values():
    """SiLU(u) = u * sigmoid(u): SiLU(0) = 0, SiLU(ln 3) = 3/4 ln 3, SiLU(-ln 3) = -1/4 ln 3."""
    l3 = math.log(3.0)
    np.testing.assert_allclose(O.silu(np.array([0.0, l3, -l3])), [0.0, 0.75 * l3, -0.25 * l3], atol=1e-15)


# ----------------------------------------------------------------------------- the mask

def literal_visible_keys(S, block, offset):
    """The mask built literally from the text: key j is visible to query i iff
    j < i (Section 4.1) and not (i and j lie in the same window) (Section 4.2,
    a window starting at n holds positions n+1..n+block; windows tile from
    ``offset``)."""
    def window(p):
        return None if p <= offset else (p - 1 - offset) // block
    vis = {}
    for i in range(1, S + 1):
        vis[i] = [j for j in range(1, S + 1)
                  if j < i and not (window(i) is not None and window(i) == window(j))]
    return vis


def test_mask_brute_force():
    for S in (1, 2, 7, 16):
        for block in (1, 2, 3, 4, 5):
            for offset in range(0, S):
                vis = literal_visible_keys(S, block, offset)
                for p in range(1, S + 1):
                    n = O.visible_true_count(p, block, offset)
                    assert vis[p] == list(range(1, n + 1)), (S, block, offset, p)


def test_block_of_one_is_strict_causal():
    for p in range(1, 20):
        for offset in (0, 3, 11):
            assert O.visible_true_count(p, 1, offset) == p - 1


# ----------------------------------------------------------------------------- block forward == sequential drafting

def sequential_reference(head, tokens, hidden, block, offset, sim_steps):
    """Step-by-step serve-time drafting that the block forward has to reproduce
    (the mask figure's caption: the unrolled states simulate inference): from
    every window start n, prefill the n true states and draft the window's
    tokens one at a time, feeding the DATA tokens."""
    S = len(tokens)
    hid_out = np.zeros((S, head.cfg.hidden)); logits = np.zeros((S, head.cfg.vocab))
    p = 1
    while p <= S:
        n = O.visible_true_count(p, block, offset)
        width = 1 if p <= offset else min(block, S - n)
        seq = O.OracleSequence(head)
        O.prefill_kv(head, seq, hidden[:n])
        for i in range(1, width + 1):
            out = O.draft_step(head, [seq], tokens_in=[tokens[n + i - 1]], concat=(i <= sim_steps))
            hid_out[n + i - 1] = out["h"][0]; logits[n + i - 1] = out["logits"][0]
        p = n + width + 1
    return hid_out, logits


@pytest.mark.parametrize("block,offset,sim_steps", [(4, 0, 1), (4, 0, 4), (4, 3, 1), (4, 3, 4), (3, 2, 2), (5, 1, 3), (1, 0, 1)])
def test_block_forward_equals_sequential_drafting(block, offset, sim_steps):
    head, _, rng = small_head(10 + block)
    S = 19
    tokens = rng.integers(0, head.cfg.vocab, S)
    hidden = rng.normal(size=(S, head.cfg.hidden))
    out = O.block_forward(head, tokens, hidden, block, offset, sim_steps)
    ref_h, ref_z = sequential_reference(head, tokens, hidden, block, offset, sim_steps)
    np.testing.assert_allclose(out["hidden"], ref_h, atol=1e-10)
    np.testing.assert_allclose(out["logits"], ref_z, atol=1e-10)
    # a subset of positions reports the same rows
    sub = O.block_forward(head, tokens, hidden, block, offset, sim_steps, positions=[S, 6, 1])
    np.testing.assert_allclose(sub["logits"], out["logits"][[0, 5, S - 1]], atol=1e-12)


def test_simulation_changes_only_later_slots():
    """Slot-1 queries never read a predicted state, so their outputs do not
    depend on sim_steps; later slots do change."""
    head, _, rng = small_head(21)
    S, k = 16, 4
    tokens = rng.integers(0, head.cfg.vocab, S); hidden = rng.normal(size=(S, head.cfg.hidden))
    a = O.block_forward(head, tokens, hidden, k, 0, 1)["logits"]
    b = O.block_forward(head, tokens, hidden, k, 0, k)["logits"]
    np.testing.assert_allclose(a[0::k], b[0::k], atol=1e-12)
    assert np.max(np.abs(a[5] - b[5])) > 1e-6      # slot 2 of window 2 reads a predicted state


# ----------------------------------------------------------------------------- cache semantics

def test_cache_reset_drops_draft_tail_and_order_is_irrelevant():
    """The cache is reset to true states at the end of an iteration; with no
    positional term the order of visible keys cannot matter (Eq. 2)."""
    head, _, rng = small_head(30)
    d = head.cfg.hidden
    states = rng.normal(size=(10, d))
    seq = O.OracleSequence(head)
    O.prefill_kv(head, seq, states)
    first = O.draft_step(head, [seq], tokens_in=[4])
    O.draft_step(head, [seq])                     # continues from its own token, appends a draft state
    assert seq.n_draft == 1
    O.prefill_kv(head, seq, np.zeros((0, d)))     # reset only
    assert seq.n_draft == 0 and seq.n_true == 10
    again = O.draft_step(head, [seq], tokens_in=[4])
    np.testing.assert_array_equal(first["logits"], again["logits"])
    perm = rng.permutation(10)
    seq2 = O.OracleSequence(head)
    O.prefill_kv(head, seq2, states[perm])
    other = O.draft_step(head, [seq2], tokens_in=[4])
    np.testing.assert_allclose(other["logits"], first["logits"], atol=1e-12)


def test_sequences_are_independent_and_chain_feeds_own_token():
    head, _, rng = small_head(31)
    d = head.cfg.hidden
    sa, sb = rng.normal(size=(6, d)), rng.normal(size=(9, d))
    seqs = [O.OracleSequence(head), O.OracleSequence(head)]
    O.prefill_kv(head, seqs[0], sa); O.prefill_kv(head, seqs[1], sb)
    both1 = O.draft_step(head, seqs, tokens_in=[1, 2])
    both2 = O.draft_step(head, seqs)
    alone = O.OracleSequence(head)
    O.prefill_kv(head, alone, sb)
    one1 = O.draft_step(head, [alone], tokens_in=[2])
    one2 = O.draft_step(head, [alone], tokens_in=[int(one1["argmax"][0])])
    np.testing.assert_allclose(both1["logits"][1], one1["logits"][0], atol=1e-12)
    np.testing.assert_allclose(both2["logits"][1], one2["logits"][0], atol=1e-12)
    # concat off ignores the draft's own state
    seqs2 = [O.OracleSequence(head)]
    O.prefill_kv(head, seqs2[0], sb)
    O.draft_step(head, seqs2, tokens_in=[2], concat=False)
    off2 = O.draft_step(head, seqs2, concat=False)
    plain = O.OracleSequence(head); O.prefill_kv(head, plain, sb)
    ref = O.draft_step(head, [plain], tokens_in=[int(one1["argmax"][0])])
    np.testing.assert_allclose(off2["logits"], ref["logits"], atol=1e-12)
    assert np.max(np.abs(off2["logits"] - one2["logits"])) > 1e-9


# ----------------------------------------------------------------------------- verification

def test_greedy_verify_is_lossless_and_bounded():
    """Accepted drafts equal the target's top-1 tokens, one more target token is
    always emitted, and 1 <= tau <= gamma + 1 (Section 3)."""
    rng = np.random.default_rng(40)
    B, gamma, V = 200, 6, 11
    logits = rng.normal(size=(B, gamma + 1, V))
    g = np.argmax(logits, axis=-1)
    draft = np.where(rng.random((B, gamma)) < 0.6, g[:, :gamma], rng.integers(0, V, (B, gamma)))
    acc, out = O.verify_greedy(draft, target_logits=logits)
    acc2, out2 = O.verify_greedy(draft, target_ids=g)
    np.testing.assert_array_equal(acc, acc2); np.testing.assert_array_equal(out, out2)
    for b in range(B):
        a = int(acc[b])
        assert 0 <= a <= gamma
        np.testing.assert_array_equal(out[b, : a + 1], g[b, : a + 1])
        assert np.all(out[b, a + 1:] == -1)
        np.testing.assert_array_equal(draft[b, :a], g[b, :a])
        if a < gamma:
            assert draft[b, a] != g[b, a]
    # the extremes
    acc, out = O.verify_greedy(g[:, :gamma], target_ids=g)
    assert np.all(acc == gamma) and np.all(out == g)
    acc, out = O.verify_greedy((g[:, :gamma] + 1) % V, target_ids=g)
    assert np.all(acc == 0) and np.all(out[:, 0] == g[:, 0]) and np.all(out[:, 1:] == -1)


def test_argmax_ties_and_nan():
    z = np.array([[1.0, 3.0, 3.0, 2.0], [np.nan, -5.0, np.nan, -7.0], [np.nan] * 4])
    np.testing.assert_array_equal(O.argmax_lowest(z), [1, 1, 0])


@pytest.mark.parametrize("gamma,expect", [(8, 3.1988), (6, 3.0588)])
def test_expected_tau_matches_tail_sum_closed_form(gamma, expect):
    """Appendix tail-sum: E[L] = sum_i prod_{j<=i} alpha^(j).  With a constant
    rate alpha the iteration emits E[tau] = 1 + sum_{i=1}^{gamma} alpha^i tokens."""
    alpha = 0.7
    closed = 1.0 + sum(alpha ** i for i in range(1, gamma + 1))
    assert abs(closed - expect) < 5e-5
    w = WL.WORKLOADS["c3_llama3_8b_b1"].scaled(batch=200_000, gamma=gamma)
    rng = np.random.default_rng(41)
    draft = rng.integers(0, w.vocab, (w.batch, gamma))
    target = WL.make_target_stream(w, rng, draft)
    acc, _ = O.verify_greedy(draft, target_ids=target)
    tau = acc + 1
    sigma = tau.std() / math.sqrt(w.batch)
    assert abs(tau.mean() - closed) < 3.5 * sigma


# ----------------------------------------------------------------------------- library cross-check

def test_against_torch_library_routines():
    """The block reduces to library routines: F.linear, F.rms_norm-free formula,
    scaled_dot_product_attention with a boolean mask, F.silu."""
    torch = pytest.importorskip("torch")
    F = torch.nn.functional
    head, w, rng = small_head(50, d=48, hq=6, hkv=3, dh=8, m=40, V=31)
    c = head.cfg
    S, k, offset = 13, 3, 2
    tokens = rng.integers(0, c.vocab, S); hidden = rng.normal(size=(S, c.hidden))
    ours = O.block_forward(head, tokens, hidden, k, offset, 1)
    T = {n: torch.tensor(np.asarray(v), dtype=torch.float64) for n, v in w.items()}
    x = T["embed"][torch.tensor(tokens)]
    rms = lambda v, g: v * torch.rsqrt(v.pow(2).mean(-1, keepdim=True) + c.rms_eps) * g
    q = F.linear(rms(x, T["g_q"]), T["w_q"]).view(S, c.n_q_heads, c.head_dim).transpose(0, 1)
    hs = torch.tensor(hidden)
    kk = F.linear(hs, T["w_k"]).view(S, c.n_kv_heads, c.head_dim).transpose(0, 1).repeat_interleave(c.group, 0)
    vv = F.linear(hs, T["w_v"]).view(S, c.n_kv_heads, c.head_dim).transpose(0, 1).repeat_interleave(c.group, 0)
    mask = torch.zeros(S, S, dtype=torch.bool)
    vis = literal_visible_keys(S, k, offset)
    for i in range(1, S + 1):
        for j in vis[i]:
            mask[i - 1, j - 1] = True
    keep = mask.any(-1)
    mask_safe = mask.clone(); mask_safe[~keep, 0] = True           # SDPA needs a non-empty row
    o = F.scaled_dot_product_attention(q[None], kk[None], vv[None], attn_mask=mask_safe[None, None])[0]
    o = o.transpose(0, 1).reshape(S, -1) * keep[:, None]
    y = F.linear(o, T["w_o"]) + x
    yn = rms(y, T["g_mlp"])
    h = F.linear(F.silu(F.linear(yn, T["w_gate"])) * F.linear(yn, T["w_up"]), T["w_down"]) + y
    z = F.linear(h, T["w_lm"])
    np.testing.assert_allclose(ours["hidden"], h.numpy(), atol=1e-11)
    np.testing.assert_allclose(ours["logits"], z.numpy(), atol=1e-11)
    np.testing.assert_array_equal(ours["argmax"], z.argmax(-1).numpy())


# ----------------------------------------------------------------------------- speculative-sampling verification

def _logits_of(dist):
    return np.log(np.asarray(dist, dtype=float))


def test_verify_sample_first_token_follows_the_target_distribution():
    """Losslessness (Section 3): whatever q is, the first emitted token is distributed as p_1.
    Integrated over a midpoint grid of the three uniforms (draft draw, acceptance test, resample);
    p and q are dyadic so that every threshold falls on a grid line and the integral is exact."""
    p = np.array([3, 1, 1, 3]) / 8.0
    q = np.array([1, 4, 2, 1]) / 8.0            # ratios min(1, p/q) = 1, 1/4, 1/2, 1; residual (1/2, 0, 0, 1/2)
    n = 16
    mid = (np.arange(n) + 0.5) / n
    cq = np.cumsum(q)
    hist = np.zeros(4)
    ua, ur = np.meshgrid(mid, mid, indexing="ij")
    B = ua.size
    for ud in mid:                                               # the draft token itself is drawn from q
        t = int(np.searchsorted(cq, ud, side="right"))
        res = O.verify_sample(np.full((B, 1), t), np.broadcast_to(_logits_of(q), (1, B, 4)),
                              np.broadcast_to(_logits_of(np.stack([p, p])), (B, 2, 4)), ua.reshape(B, 1), ur.reshape(B))
        hist += np.bincount(res["out_tokens"][:, 0], minlength=4)
        assert np.all(res["accept_len"] <= 1) and np.all(res["out_tokens"][res["accept_len"] == 1, 0] == t)
    np.testing.assert_allclose(hist / hist.sum(), p, atol=1e-12)


def test_verify_sample_special_cases():
    V = 5
    rng = np.random.default_rng(71)
    z = rng.normal(size=(3, V))
    draft = np.array([[1, 4]])
    u = rng.random((1, 2))
    # q == p: every draft is accepted, the extra token comes from p_{gamma+1} by inverse CDF
    r = O.verify_sample(draft, z[:2][:, None, :], z[None], u, np.array([0.999999]))
    assert r["accept_len"][0] == 2 and r["out_tokens"][0].tolist() == [1, 4, V - 1]
    r = O.verify_sample(draft, z[:2][:, None, :], z[None], u, np.array([0.0]))
    assert r["out_tokens"][0].tolist() == [1, 4, 0]
    # the target gives the first draft (almost) no mass: rejected at once, and the residual never returns it
    zt = z.copy(); zt[0, 1] = -80.0
    for ur in (0.0, 0.3, 0.7, 0.999):
        r = O.verify_sample(draft, z[:2][:, None, :], zt[None], np.array([[1e-9, 0.5]]), np.array([ur]))
        assert r["accept_len"][0] == 0 and r["out_tokens"][0, 0] != 1 and r["out_tokens"][0, 1:].tolist() == [-1, -1]
    # residual distribution by hand: p = (.5,.5,0), q = (.75,.25,0) -> max(0,p-q) = (0,.25,0) -> token 1 always
    np.testing.assert_allclose(O.residual_distribution([0.5, 0.5, 0.0], [0.75, 0.25, 0.0]), [0, 1, 0])
    np.testing.assert_allclose(O.residual_distribution([0.2, 0.8], None), [0.2, 0.8])
    assert O.inverse_cdf(np.array([0.25, 0.5, 0.25]), 0.25)[0] == 1 and O.inverse_cdf(np.array([0.25, 0.5, 0.25]), 0.2499)[0] == 0
    # temperature: T -> small makes both sides one-hot, so the rule reduces to greedy matching
    zq = np.array([[0.0, 3.0, 1.0]]); zp = np.array([[0.0, 1.0, 3.0], [2.0, 0.0, 0.0]])
    r = O.verify_sample(np.array([[1]]), zq[:, None, :], zp[None], np.array([[0.5]]), np.array([0.5]), temperature=0.01)
    assert r["accept_len"][0] == 0 and r["out_tokens"][0, 0] == 2            # target's top-1 replaces the rejected draft
    np.testing.assert_allclose(O.softmax_rows(np.array([[0.0, np.log(3.0)]])), [[0.25, 0.75]])
    np.testing.assert_allclose(O.softmax_rows(np.array([[0.0, np.log(3.0)]]), temperature=0.5), [[0.1, 0.9]])


def test_verify_sample_acceptance_rate_matches_closed_form():
    """With drafts drawn from q, a position is accepted with probability sum_v min(p(v), q(v))."""
    rng = np.random.default_rng(72)
    V, gamma, B = 6, 3, 60000
    zp, zq = rng.normal(size=(gamma + 1, V)), rng.normal(size=(gamma, V))
    p, q = O.softmax_rows(zp), O.softmax_rows(zq)
    draft = np.stack([rng.choice(V, size=B, p=q[i]) for i in range(gamma)], axis=1)
    r = O.verify_sample(draft, np.broadcast_to(zq[:, None, :], (gamma, B, V)), np.broadcast_to(zp[None], (B, gamma + 1, V)),
                        rng.random((B, gamma)), rng.random(B))
    alpha = np.minimum(p[:gamma], q).sum(axis=1)
    expect = alpha[0] + alpha[0] * alpha[1] + alpha[0] * alpha[1] * alpha[2]      # E[accept_len], tail-sum
    assert abs(r["accept_len"].mean() - expect) < 4 * np.sqrt(gamma) / np.sqrt(B) + 1e-3
    assert np.all((r["out_tokens"] >= 0).sum(axis=1) == r["accept_len"] + 1)
    # the extra token after full acceptance follows p_{gamma+1}
    full = r["accept_len"] == gamma
    h = np.bincount(r["out_tokens"][full, gamma], minlength=V) / full.sum()
    np.testing.assert_allclose(h, p[gamma], atol=4 / np.sqrt(full.sum()))


# ----------------------------------------------------------------------------- training losses (forward)

def test_cross_entropy_closed_forms():
    V = 7
    # uniform draft: CE = log V whatever the target; equal distributions: CE = entropy
    np.testing.assert_allclose(O.cross_entropy_rows(np.zeros((2, V)), target_ids=[3, 0]), np.log(V))
    p = np.array([0.5, 0.25, 0.125, 0.125])
    np.testing.assert_allclose(O.cross_entropy_rows(np.log(p)[None], target_logits=np.log(p)[None] + 5.0), [1.75 * np.log(2)])
    # hand case: q = (1/4, 3/4), p = (1/2, 1/2): -(log 1/4 + log 3/4) / 2
    np.testing.assert_allclose(O.cross_entropy_rows(np.array([[0.0, np.log(3.0)]]), target_logits=np.zeros((1, 2))),
                               [-(np.log(0.25) + np.log(0.75)) / 2])
    # a (nearly) one-hot soft target equals the hard label
    z = np.random.default_rng(80).normal(size=(3, V))
    hot = np.full((3, V), -60.0); hot[[0, 1, 2], [4, 0, 6]] = 60.0
    np.testing.assert_allclose(O.cross_entropy_rows(z, target_logits=hot), O.cross_entropy_rows(z, target_ids=[4, 0, 6]), rtol=1e-12)
    # Gibbs: CE(p, q) >= entropy(p)
    t = np.random.default_rng(81).normal(size=(3, V))
    pt = O.softmax_rows(t)
    assert np.all(O.cross_entropy_rows(z, target_logits=t) >= -np.sum(pt * np.log(pt), axis=-1) - 1e-12)


def test_loss_weights_follow_eq4_and_eq7():
    # S = 11, k = 4, offset 2: windows start at 2, 6, 10 -> N = 3; slots of positions 3..11: 1 2 3 4 1 2 3 4 1
    w, n = O.loss_weights(11, 4, 2, 1, "early")
    assert n == 3 and w.tolist() == [0, 0] + [1] * 9
    w, n = O.loss_weights(11, 4, 2, 4, "late")            # beta* = k - i + 1
    assert w.tolist() == [0, 0, 4, 3, 2, 1, 4, 3, 2, 1, 4]
    w, n = O.loss_weights(11, 4, 2, 2, "late")            # only two simulated steps: slots 3, 4 carry no term
    assert w.tolist() == [0, 0, 4, 3, 0, 0, 4, 3, 0, 0, 4]
    assert O.loss_weights(8, 4, 0, 1, "early")[1] == 2 and O.loss_weights(9, 4, 0, 1, "early")[1] == 3


def test_block_loss_is_the_weighted_mean_of_block_forward_cross_entropies():
    head, w, rng = small_head(seed=82)
    B, S, k, off = 2, 13, 3, 1
    tokens = rng.integers(0, head.cfg.vocab, (B, S))
    hidden = rng.normal(size=(B, S, head.cfg.hidden))
    tl = rng.normal(size=(B, S, head.cfg.vocab)) * 2
    out = O.block_loss(head, tokens, hidden, k, off, "late", sim_steps=3, target_logits=tl)
    ref = 0.0
    for b in range(B):
        lg = O.block_forward(head, tokens[b], hidden[b], k, off, 3)["logits"]
        q = O.softmax_rows(lg); p = O.softmax_rows(tl[b])
        for pos in range(off + 1, S + 1):
            i = pos - O.visible_true_count(pos, k, off)
            ref += (k - i + 1) * -(p[pos - 1] * np.log(q[pos - 1])).sum()
    assert out["n_windows"] == 4
    np.testing.assert_allclose(out["loss"], ref / (B * 4), rtol=1e-12)
    early = O.block_loss(head, tokens, hidden, k, off, "early", target_ids=tokens)
    assert early["ce"].shape == (B, S) and early["loss"] > 0
    with pytest.raises(ValueError):
        O.block_loss(head, tokens, hidden, k, off, "early", sim_steps=2, target_ids=tokens)


# ----------------------------------------------------------------------------- dynamic draft tree

# ----------------------------------------------------------------------------- rotary option

def test_rope_rotation_by_hand_and_orthogonality():
    # d_h = 2: one pair, frequency 1: position pi/2 turns (1, 0) into (0, 1)
    x = np.array([[[1.0, 0.0]]])
    np.testing.assert_allclose(O.rope_rotate(x, np.array([np.pi / 2]), 10000.0), [[[0.0, 1.0]]], atol=1e-15)
    # d_h = 4, theta = 10000: pair (0, 2) turns by pos, pair (1, 3) by pos / 100
    x = np.array([[[1.0, 2.0, 3.0, 4.0]]])
    pos = 7.0
    a, b = pos, pos / 100.0
    want = [1 * np.cos(a) - 3 * np.sin(a), 2 * np.cos(b) - 4 * np.sin(b), 3 * np.cos(a) + 1 * np.sin(a), 4 * np.cos(b) + 2 * np.sin(b)]
    np.testing.assert_allclose(O.rope_rotate(x, np.array([pos]), 10000.0)[0, 0], want, atol=1e-14)
    rng = np.random.default_rng(3)
    y = rng.normal(size=(5, 3, 8))
    p5 = np.array([0, 1, 17, 400, 8191])
    r = O.rope_rotate(y, p5, 500000.0)
    np.testing.assert_allclose(r[0], y[0], atol=0)                                       # position 0: identity
    np.testing.assert_allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(y, axis=-1), rtol=1e-13)
    np.testing.assert_allclose(O.rope_rotate(r, p5, 500000.0, inverse=True), y, atol=1e-12)


def test_rope_scores_depend_on_relative_position_only():
    rng = np.random.default_rng(4)
    q, k = rng.normal(size=(1, 2, 16)), rng.normal(size=(1, 2, 16))
    def score(p, j):
        return np.sum(O.rope_rotate(q, np.array([p]), 10000.0) * O.rope_rotate(k, np.array([j]), 10000.0), axis=-1)
    np.testing.assert_allclose(score(9, 4), score(109, 104), atol=1e-12)
    np.testing.assert_allclose(score(9, 4), score(5, 0), atol=1e-12)
    assert np.max(np.abs(score(9, 4) - score(9, 5))) > 1e-3


@pytest.mark.parametrize("block,offset,sim_steps", [(4, 0, 4), (4, 3, 1), (3, 2, 2)])
def test_rope_block_forward_equals_sequential_drafting(block, offset, sim_steps):
    """With the rotary option both paths must place every query and every key (true or predicted) at the same
    position; and the option must change the result (key order now matters)."""
    head, w, rng = small_head(20 + block, rope_theta=10000.0)
    S = 17
    tokens = rng.integers(0, head.cfg.vocab, S)
    hidden = rng.normal(size=(S, head.cfg.hidden))
    out = O.block_forward(head, tokens, hidden, block, offset, sim_steps)
    ref_h, ref_z = sequential_reference(head, tokens, hidden, block, offset, sim_steps)
    np.testing.assert_allclose(out["hidden"], ref_h, atol=1e-10)
    np.testing.assert_allclose(out["logits"], ref_z, atol=1e-10)
    plain = O.block_forward(O.OracleHead(O.HeadConfig(*[getattr(head.cfg, f) for f in ("hidden", "n_q_heads", "n_kv_heads", "head_dim", "mlp_dim", "vocab")]), w),
                            tokens, hidden, block, offset, sim_steps)
    assert np.max(np.abs(plain["logits"][-1] - out["logits"][-1])) > 1e-3
    # position 1 of a sequence has no key and position 2 one key: rotations cannot change a one-key softmax
    np.testing.assert_allclose(plain["logits"][:2], out["logits"][:2], atol=1e-10)


# ----------------------------------------------------------------------------- gradients of the training losses

def _grad_fixture(seed, B=2, S=9, **kw):
    head, w, rng = small_head(seed=seed, d=16, hq=4, hkv=2, dh=4, m=24, V=19, std=0.4, **kw)
    tokens = rng.integers(0, 19, (B, S))
    hidden = rng.normal(0, 1.0, (B, S, 16))
    tgt = rng.normal(0, 2.0, (B, S, 19))
    return head, w, tokens, hidden, tgt


def test_smooth_l1_and_rmsnorm_backward_by_differences():
    r = np.array([-3.0, -1.0, -0.5, 0.0, 0.25, 1.0, 2.0])
    assert np.allclose(O.smooth_l1(r), [2.5, 0.5, 0.125, 0.0, 0.03125, 0.5, 1.5])
    rng = np.random.default_rng(5)
    v, g, dn = rng.normal(size=(3, 7)), 1 + rng.normal(0, 0.2, 7), rng.normal(size=(3, 7))
    dv, dg = O.rms_norm_backward(v, g, 1e-5, dn)
    f = lambda vv, gg: float(np.sum(O.rms_norm(vv, gg, 1e-5) * dn))
    e = 1e-6
    for idx in [(0, 0), (1, 3), (2, 6)]:
        vp, vm = v.copy(), v.copy(); vp[idx] += e; vm[idx] -= e
        assert abs((f(vp, g) - f(vm, g)) / (2 * e) - dv[idx]) < 1e-7
    for i in (0, 4):
        gp, gm = g.copy(), g.copy(); gp[i] += e; gm[i] -= e
        assert abs((f(v, gp) - f(v, gm)) / (2 * e) - dg[i]) < 1e-7


@pytest.mark.parametrize("block,offset,labels,norms,theta", [(3, 0, False, True, 0.0), (4, 2, True, True, 0.0), (2, 1, False, False, 0.0),
                                                             (3, 1, False, True, 10000.0)])
def test_early_stage_gradient_is_the_derivative_of_block_loss(block, offset, labels, norms, theta):
    """Eq. 4: central differences of block_loss (a separate function) in every parameter tensor,
    at the entries of largest gradient magnitude and at random ones."""
    head, w, tokens, hidden, tgt = _grad_fixture(31 + block, norm_q=norms, norm_mlp=norms, rope_theta=theta)
    ids = np.argmax(tgt, axis=-1)
    kw = dict(target_ids=ids) if labels else dict(target_logits=tgt)
    out = O.block_loss_grad(head, tokens, hidden, block, offset, "early", **kw)
    base = O.block_loss(head, tokens, hidden, block, offset, "early", **kw)["loss"]
    assert abs(out["loss"] - base) < 1e-12 and out["vloss"] >= 0 and out["total"] == out["loss"]
    rng = np.random.default_rng(7)
    e = 1e-5
    for name, g in out["grads"].items():
        if not norms and name in ("g_q", "g_mlp"):
            assert not g.any()
            continue
        flat = np.abs(g).reshape(-1)
        picks = list(np.argsort(flat)[-2:]) + list(rng.integers(0, flat.size, 2))
        for k in picks:
            idx = np.unravel_index(int(k), g.shape)
            vals = []
            for sgn in (1, -1):
                w2 = {n: a.copy() for n, a in w.items()}
                w2[name][idx] += sgn * e
                vals.append(O.block_loss(O.OracleHead(head.cfg, w2), tokens, hidden, block, offset, "early", **kw)["loss"])
            fd = (vals[0] - vals[1]) / (2 * e)
            assert abs(fd - g[idx]) < 1e-7 + 1e-5 * abs(fd), (name, idx, fd, g[idx])


def _torch_training_loss(torch, c, T, tokens, hidden, tgt, block, offset, stage, sim_steps, vcoef, pred_states):
    """An independent restatement with torch (float64, autograd): the final simulation step with the
    predicted states given as constants.  Rotary option in the usual rotate-half form
    x * cos + rotate_half(x) * sin with the angles repeated over the two halves."""
    Fn = torch.nn.functional

    def rope(x, pos):              # x [rows, H, d_h]
        if c.rope_theta <= 0:
            return x
        half = c.head_dim // 2
        inv = c.rope_theta ** (-torch.arange(0, half, dtype=torch.float64) * 2 / c.head_dim)
        ang = torch.as_tensor(pos, dtype=torch.float64)[:, None] * inv[None, :]
        emb = torch.cat([ang, ang], dim=-1)[:, None, :]
        rot = torch.cat([-x[..., half:], x[..., :half]], dim=-1)
        return x * emb.cos() + rot * emb.sin()

    B, S = tokens.shape
    w, n_windows = O.loss_weights(S, block, offset, sim_steps, stage)
    n_reg = B * int(np.count_nonzero(w))
    rms = lambda v, g: v * torch.rsqrt(v.pow(2).mean(-1, keepdim=True) + c.rms_eps) * g
    total_l, total_v = 0.0, 0.0
    for b in range(B):
        x = T["embed"][torch.tensor(tokens[b])]
        xn = rms(x, T["g_q"]) if c.norm_q else x
        q = rope(Fn.linear(xn, T["w_q"]).view(S, c.n_q_heads, c.head_dim), np.arange(S))
        hs = torch.tensor(hidden[b])
        rows = []
        for p in range(1, S + 1):
            n = O.visible_true_count(p, block, offset)
            extra = list(range(n, n + min(p - n, sim_steps) - 1))
            src = torch.cat([hs[:n], torch.tensor(pred_states[b][extra]).view(-1, c.hidden)]) if extra else hs[:n]
            if src.shape[0] == 0:
                rows.append(torch.zeros(c.n_q_heads * c.head_dim, dtype=torch.float64))
                continue
            k = rope(Fn.linear(src, T["w_k"]).view(-1, c.n_kv_heads, c.head_dim), np.array(list(range(n)) + extra)).repeat_interleave(c.group, dim=1)
            v = Fn.linear(src, T["w_v"]).view(-1, c.n_kv_heads, c.head_dim).repeat_interleave(c.group, dim=1)
            a = torch.einsum("hd,jhd->hj", q[p - 1], k) / math.sqrt(c.head_dim)
            rows.append(torch.einsum("hj,jhd->hd", torch.softmax(a, dim=-1), v).reshape(-1))
        o = torch.stack(rows)
        y = Fn.linear(o, T["w_o"]) + x
        yn = rms(y, T["g_mlp"]) if c.norm_mlp else y
        h = Fn.linear(Fn.silu(Fn.linear(yn, T["w_gate"])) * Fn.linear(yn, T["w_up"]), T["w_down"]) + y
        logq = torch.log_softmax(Fn.linear(h, T["w_lm"]), dim=-1)
        ce = -(torch.softmax(torch.tensor(tgt[b]), dim=-1) * logq).sum(-1)
        wt = torch.tensor(w)
        total_l = total_l + (wt * ce).sum() / (B * n_windows)
        reg = (wt > 0).to(torch.float64)[:, None]
        total_v = total_v + (reg * Fn.smooth_l1_loss(h, hs, reduction="none", beta=1.0)).sum() / (n_reg * c.hidden)
    return total_l, total_v, total_l + vcoef * total_v


@pytest.mark.parametrize("stage,block,offset,sim_steps,vcoef,theta", [("early", 3, 1, 1, 10.0, 0.0), ("late", 4, 0, 3, 10.0, 0.0),
                                                                      ("late", 3, 2, 3, 0.0, 0.0), ("early", 4, 2, 1, 10.0, 10000.0),
                                                                      ("late", 4, 1, 3, 0.0, 500000.0)])
def test_training_gradients_against_torch_autograd(stage, block, offset, sim_steps, vcoef, theta):
    """Eq. 4 / Eq. 7 plus the regression term of Appendix B: every parameter's gradient against
    automatic differentiation of an independent restatement; under simulation the predicted states
    are constants there as well (they come from the oracle's own forward)."""
    torch = pytest.importorskip("torch")
    head, w, tokens, hidden, tgt = _grad_fixture(50 + block, rope_theta=theta)
    c = head.cfg
    out = O.block_loss_grad(head, tokens, hidden, block, offset, stage, sim_steps, target_logits=tgt, vloss_coef=vcoef)
    pred = [O.block_forward(head, tokens[b], hidden[b], block, offset, sim_steps)["hidden"] for b in range(tokens.shape[0])]
    T = {n: torch.tensor(np.asarray(v), dtype=torch.float64, requires_grad=True) for n, v in w.items()}
    l, v, total = _torch_training_loss(torch, c, T, tokens, hidden, tgt, block, offset, stage, sim_steps, vcoef, pred)
    total.backward()
    assert abs(float(l.detach()) - out["loss"]) < 1e-10 and abs(float(v.detach()) - out["vloss"]) < 1e-10
    assert abs(out["loss"] - O.block_loss(head, tokens, hidden, block, offset, stage, sim_steps, target_logits=tgt)["loss"]) < 1e-12
    for name, g in out["grads"].items():
        ref = T[name].grad.numpy()
        assert np.max(np.abs(ref - g)) < 1e-10 * (1 + np.max(np.abs(ref))), name
        assert np.max(np.abs(ref)) > 0, name


def test_regression_term_alone_has_the_closed_form_gradient_in_w_down():
    """With the loss coefficient on the cross-entropy's side removed (labels that the draft already
    predicts with certainty are not needed: take vloss alone through total - loss), d vloss / d W_down
    = (clip(h - h_true, -1, 1) / (rows d))^T act."""
    head, w, tokens, hidden, tgt = _grad_fixture(77, B=1, S=6)
    a = O.block_loss_grad(head, tokens, hidden, 3, 0, "early", target_logits=tgt, vloss_coef=0.0)
    b = O.block_loss_grad(head, tokens, hidden, 3, 0, "early", target_logits=tgt, vloss_coef=4.0)
    kv_rows = []
    k_true, v_true = O.project_kv(head, hidden[0])
    for p in range(1, 7):
        n = O.visible_true_count(p, 3, 0)
        kv_rows.append((k_true[:n], v_true[:n]))
    f = O.draft_block(head, tokens[0], kv_rows)
    expect = (np.clip(f["h"] - hidden[0], -1, 1) / (6 * 16)).T @ f["act"]
    assert np.allclose((b["grads"]["w_down"] - a["grads"]["w_down"]) / 4.0, expect, atol=1e-12)
    assert abs(b["total"] - (a["loss"] + 4.0 * a["vloss"])) < 1e-12


def _tree_fixture(seed=90, n=9):
    head, w, rng = small_head(seed=seed)
    seq = O.OracleSequence(head)
    O.prefill_kv(head, seq, rng.normal(size=(n, head.cfg.hidden)))
    return head, seq, rng


def test_tree_with_one_child_per_node_is_chain_drafting():
    """topk = 1: the tree is a path, and it is exactly the greedy chain of draft_step with concat."""
    head, seq, rng = _tree_fixture()
    tree = O.draft_tree(head, seq, root_token=7, depth=4, topk=1, n_candidates=10)
    chain, lp = [], []
    tok = [7]
    for s in range(5):
        out = O.draft_step(head, [seq], tokens_in=tok if s == 0 else None, concat=True)
        chain.append(int(out["argmax"][0]))
        lp.append(O.log_softmax_rows(out["logits"][0])[chain[-1]])
    O.rollback(seq)
    assert tree["tokens"].tolist() == chain and tree["parents"].tolist() == [-1, 0, 1, 2, 3]
    np.testing.assert_allclose(tree["scores"], np.cumsum(lp), rtol=1e-12)


def test_tree_scores_are_path_log_probabilities_and_selection_is_closed():
    head, seq, rng = _tree_fixture(seed=91)
    K, D, N = 3, 3, 14
    tree = O.draft_tree(head, seq, root_token=11, depth=D, topk=K, n_candidates=N)
    tok, par, sc = tree["tokens"], tree["parents"], tree["scores"]
    assert len(tok) == N and len(tree["all_tokens"]) == K + D * K * K
    assert np.all(par < np.arange(N)) and np.all(par[tree["depths"] == 1] == -1)
    # every kept node's score is the sum of log q along its path, recomputed by forced chain drafting
    for n in range(N):
        path = []
        a = n
        while a >= 0:
            path.append(int(tok[a])); a = int(par[a])
        path = path[::-1]
        total, feed = 0.0, 11
        for t in path:
            out = O.draft_step(head, [seq], tokens_in=[feed], concat=True)
            total += O.log_softmax_rows(out["logits"][0])[t]
            feed = t
        O.rollback(seq)
        np.testing.assert_allclose(sc[n], total, rtol=1e-10, atol=1e-10)
        if par[n] >= 0:
            assert sc[par[n]] >= sc[n]
    # the kept set is the top-N of everything that was created, and siblings are distinct tokens
    assert np.sort(tree["all_scores"])[::-1][N - 1] <= sc.min() + 1e-15
    for p_ in set(par.tolist()):
        sib = tok[par == p_]
        assert len(set(sib.tolist())) == len(sib)
    # each expansion level forwards the topk best children of the level before
    a_sc, a_par = tree["all_scores"], tree["all_parents"]
    level = np.arange(K, K + K * K)
    np.testing.assert_array_equal(np.sort(tree["forward_nodes"][1]), np.sort(level[O.top_k_lowest(a_sc[level], K)]))


def test_top_k_lowest_and_tree_verification_by_hand():
    assert O.top_k_lowest(np.array([1.0, 3.0, 3.0, 2.0, 3.0]), 3).tolist() == [1, 2, 4]
    np.testing.assert_allclose(np.exp(O.log_softmax_rows(np.array([[0.0, np.log(3.0)]]))), [[0.25, 0.75]])
    #        root -> 0:'a'(5) -> 2:'c'(7) -> 4:'e'(9)
    #             -> 1:'b'(6) -> 3:'d'(8)
    tokens, parents = np.array([5, 6, 7, 8, 9]), np.array([-1, -1, 0, 1, 2])
    # target wants 6 at the root, then 8 after node 1, then 4 after node 3: path (1, 3), three tokens emitted
    a, out, path = O.verify_tree_greedy(tokens, parents, 6, np.array([0, 8, 0, 4, 0]))
    assert a == 2 and out.tolist() == [6, 8, 4] and path.tolist() == [1, 3]
    # nothing matches at the root: only the target's own token
    a, out, path = O.verify_tree_greedy(tokens, parents, 1, np.array([0, 8, 0, 4, 0]))
    assert a == 0 and out.tolist() == [1] and path.tolist() == []
    # a match that is not a child of the current node does not count (7 is a child of node 0, not of the root)
    a, out, _ = O.verify_tree_greedy(tokens, parents, 7, np.zeros(5, dtype=int))
    assert a == 0 and out.tolist() == [7]
    # lossless: the emitted tokens are exactly the target's greedy tokens along the accepted path
    a, out, path = O.verify_tree_greedy(tokens, parents, 5, np.array([7, 0, 9, 0, 2]))
    assert a == 3 and out.tolist() == [5, 7, 9, 2] and path.tolist() == [0, 2, 4]


# ----------------------------------------------------------------------------- storage mode

def test_round_bf16_ties_to_even_and_matches_torch():
    torch = pytest.importorskip("torch")
    # exact halves between two bf16 neighbours (spacing 2^-7 in [1, 2)) go to the even one
    np.testing.assert_array_equal(O.round_bf16(np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, -(1 + 2.0 ** -8), 0.0, 1.5])),
                                  [1.0, 1 + 2.0 ** -6, -1.0, 0.0, 1.5])
    # a float64 just above a half rounds up although float32 would first round it onto the half
    np.testing.assert_array_equal(O.round_bf16(np.array([1 + 2.0 ** -8 + 2.0 ** -40])), [1 + 2.0 ** -7])
    rng = np.random.default_rng(61)
    a = (rng.normal(size=20000) * 10.0 ** rng.uniform(-5, 5, size=20000)).astype(np.float32).astype(np.float64)
    t = torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(O.round_bf16(a), t)
    np.testing.assert_array_equal(O.round_bf16(t), t)                       # idempotent


def test_storage_mode_rounds_only_where_values_are_stored():
    head, w, rng = small_head(seed=62)
    c = head.cfg
    rounded = head.with_storage("bf16")
    assert rounded.w_q is head.w_q and head.cfg.storage is None            # shared arrays, default untouched
    states = rng.normal(size=(9, c.hidden))
    toks = [1, 2, 3]
    exact = O.draft_block(head, toks, [O.project_kv(head, states)] * 3)
    stored = O.draft_block(rounded, toks, [O.project_kv(rounded, states)] * 3)
    for name in ("q", "o", "y", "h"):                                       # stored values are bf16 numbers ...
        np.testing.assert_array_equal(O.round_bf16(stored[name]), stored[name])
        assert np.abs(stored[name] - exact[name]).max() > 0                 # ... and differ from the unrounded ones
        assert np.abs(stored[name] - exact[name]).max() <= 0.05 * (1 + np.abs(exact[name]).max())
    k, v = O.project_kv(rounded, states)
    np.testing.assert_array_equal(O.round_bf16(k), k)
    assert np.abs(O.round_bf16(stored["logits"]) - stored["logits"]).max() > 0      # logits are not rounded
    # a sequence driven through the cache API sees the same rounded keys
    seq = O.OracleSequence(rounded)
    O.prefill_kv(rounded, seq, states)
    np.testing.assert_array_equal(seq.k_true, k)
    with pytest.raises(ValueError):
        O.project_kv(head.with_storage("fp8"), states)


# ----------------------------------------------------------------------------- generators

def test_bf16_rounding_of_generator_matches_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(60)
    a = rng.normal(size=10000).astype(np.float32) * 3
    a[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]      # exact halves round to even
    r = WL.round_to_storage(a, "bf16")
    t = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(r, t)
    np.testing.assert_array_equal(WL.round_to_storage(a, "fp32"), a)


def test_workload_shapes_and_determinism():
    w = WL.WORKLOADS["c1_tiny_fp32"]
    a, b = WL.make_weights(w), WL.make_weights(w)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])
    assert a["w_gate"].shape == (688, 256) and a["w_lm"].shape == (1024, 256)
    w4 = WL.WORKLOADS["c4_llama3_8b_b32"]
    n = WL.make_context_lengths(w4, WL.data_rng(w4))
    assert n.shape == (32,) and n.min() >= 512 and n.max() <= 8192


# ----------------------------------------------------------------------------- FP8 option

def test_round_e4m3_hand_values_and_torch():
    """E4M3 by its definition: spacing 2^(e-3) in [2^e, 2^(e+1)), subnormal step 2^-9, largest value 448, ties to even."""
    x = np.array([0.0, 1.0, 1.0625, 1.1875, 1.3125, 17.0, 18.0, 19.0, 448.0, 1000.0, -460.0, 2.0 ** -9, 2.0 ** -10, 1.5 * 2.0 ** -9, 0.0179])
    want = np.array([0.0, 1.0, 1.0, 1.25, 1.25, 16.0, 18.0, 20.0, 448.0, 448.0, -448.0, 2.0 ** -9, 0.0, 2.0 ** -8, 0.017578125])
    np.testing.assert_array_equal(O.round_e4m3(x), want)
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("this torch has no float8_e4m3fn")
    rng = np.random.default_rng(8)
    v = np.concatenate([rng.normal(0, 100, 4000), rng.normal(0, 1, 4000), rng.normal(0, 0.01, 4000), rng.uniform(-448, 448, 4000)])
    v = v[np.abs(v) <= 448].astype(np.float32)
    t = torch.from_numpy(v).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    np.testing.assert_array_equal(O.round_e4m3(v.astype(np.float64)), t)
    # every one of the 2 x 127 finite codes is a fixed point
    codes = torch.arange(0, 256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    codes = codes[np.isfinite(codes)]
    np.testing.assert_array_equal(O.round_e4m3(codes), codes)


def test_fp8_lm_head_is_the_quantised_product_and_close_to_the_exact_one():
    head, w, rng = small_head(61, d=64, V=40)
    h = rng.normal(0, 1.5, (5, 64))
    z8 = O.lm_head_fp8(head, h)
    qh, sh = O.quantize_rows_e4m3(h)
    qw, sw = O.quantize_rows_e4m3(w["w_lm"])
    assert np.max(np.abs(qh)) == 448 and np.all(np.max(np.abs(qw), axis=1) == 448)          # the row maximum maps to the largest code
    for b in (0, 4):
        for v in (0, 39):
            assert abs(z8[b, v] - sh[b] * sw[v] * float(np.dot(qh[b], qw[v]))) < 1e-12
    z = O.lm_head(head, h)
    assert np.max(np.abs(z8 - z)) < 0.08 * np.max(np.abs(z))        # 3 fraction bits on both operands, averaged over 64 terms
    assert np.max(np.abs(z8 - z)) > 1e-4                            # and it is not the unquantised product
    np.testing.assert_array_equal(O.quantize_rows_e4m3(np.zeros((1, 8)))[0], np.zeros((1, 8)))


def test_quantize_rows_e4m3_hand_row_and_torch_cast():
    """The row-wise scale convention pinned by something other than its own formula: a row worked by hand whose scale is a power of
    two (every quotient exact), the reconstruction bound that 3 fraction bits imply, and torch's own FP8 cast of x / scale."""
    # max |x| = 224 = 448 / 2 -> scale 0.5; the quotients 2x are 448, -3, 17 (-> 16: tie to even), 19 (-> 20: tie to even), 0.25, 0
    x = np.array([[224.0, -1.5, 8.5, 9.5, 0.125, 0.0]])
    q, sc = O.quantize_rows_e4m3(x)
    assert sc.tolist() == [0.5]
    assert q.tolist() == [[448.0, -3.0, 16.0, 20.0, 0.25, 0.0]]
    # a second row with another sign and a scale that is again exact: max 56 -> scale 1/8, quotients 8x
    q, sc = O.quantize_rows_e4m3(np.array([[-56.0, 1.0, 0.3125, 2.0625]]))
    assert sc.tolist() == [0.125] and q.tolist() == [[-448.0, 8.0, 2.5, 16.0]]          # 16.5 ties to the even code 16
    # what the format guarantees: |x - scale q| <= scale * (spacing at |x / scale|) / 2, spacing 2^(e-3), subnormal step 2^-9
    rng = np.random.default_rng(77)
    xs = np.concatenate([rng.normal(0, 3, (6, 512)), rng.normal(0, 1e-3, (2, 512)), rng.uniform(-50, 50, (2, 512))]).astype(np.float32).astype(np.float64)
    q, sc = O.quantize_rows_e4m3(xs)
    ratio = np.abs(xs) / sc[:, None]
    spacing = np.exp2(np.maximum(np.floor(np.log2(np.maximum(ratio, 2.0 ** -6))), -6.0) - 3.0)
    assert np.all(np.abs(xs - sc[:, None] * q) <= sc[:, None] * spacing * 0.5 * (1 + 1e-6) + 1e-12)
    assert np.all(np.max(np.abs(q), axis=1) == 448.0)
    assert np.all(np.sign(q) * np.sign(xs) >= 0)
    # the library routine: torch's cast of the float32 quotient
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("this torch has no float8_e4m3fn")
    x32 = torch.from_numpy(xs.astype(np.float32))
    scale_t = x32.abs().amax(dim=1, keepdim=True) / 448.0
    q_t = (x32 / scale_t).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    np.testing.assert_array_equal(q, q_t)
    np.testing.assert_array_equal(sc, scale_t[:, 0].to(torch.float64).numpy())
