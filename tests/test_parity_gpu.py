"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle, element by element on
the same seeded inputs.  Sizes here finish in seconds on the oracle yet span several tiles, several
split-KV chunks and ragged tails; the full-size configurations live in test_parity_full_gpu.py."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2505_24544_b200 import workloads as WL
from parity_utils import assert_close, cache_rows_parity, check_tokens, oracle_head, run_chain_parity, to_dev

pytestmark = pytest.mark.gpu


def build(w: WL.Workload, **kw):
    from paper_2505_24544_b200.binding import BeagleHead
    weights = WL.make_weights(w)
    return BeagleHead.from_workload(w, weights, **kw), oracle_head(w, weights, rope_theta=kw.get("rope_theta", 0.0)), weights


SMALL_GQA = WL.WORKLOADS["c3_llama3_8b_b1"].scaled(name="small_gqa", hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=64,
                                                   mlp_dim=1400, vocab=4099, batch=3, ctx_min=1, ctx_max=700, gamma=5, seed=2001)
SMALL_MHA = WL.WORKLOADS["c2_llama2_7b_b1"].scaled(name="small_mha", hidden=768, n_q_heads=6, n_kv_heads=6, head_dim=128,
                                                   mlp_dim=2048, vocab=5000, batch=2, ctx_min=255, ctx_max=258, gamma=4, seed=2002)


def prefill_both(head_gpu, head_cpu, w, rng, slots, lengths):
    hidden = WL.make_hidden(w, rng, int(np.sum(lengths)))
    head_gpu.prefill_kv(slots, list(map(int, lengths)), to_dev(hidden, w.dtype) if len(hidden) else None)
    seqs, r = [], 0
    for n in lengths:
        s = O.OracleSequence(head_cpu)
        O.prefill_kv(head_cpu, s, hidden[r:r + n])
        seqs.append(s)
        r += n
    return seqs


def test_c1_tiny_fp32_chain_then_verify():
    w = WL.WORKLOADS["c1_tiny_fp32"]
    head_gpu, head_cpu, _ = build(w)
    rng = WL.data_rng(w)
    seqs = prefill_both(head_gpu, head_cpu, w, rng, [0], [64])
    first = WL.make_tokens(w, rng, (1,))
    drafted, drafted_ref, err = run_chain_parity(head_gpu, head_cpu, w, [0], seqs, first, w.gamma)
    assert err <= 1e-5
    assert head_gpu.slot_lengths(0) == (64, w.gamma - 1)
    # greedy verify against a random-logit target (agreement ~ 1/V) and a planted variant
    for planted_len in (0, 2, w.gamma):
        planted = np.full(w.gamma + 1, -1)
        planted[:planted_len] = drafted_ref[0, :planted_len]
        logits = WL.make_target_logits(w, rng, w.gamma + 1, planted)
        acc, out = head_gpu.verify_greedy(to_dev(drafted_ref.astype(np.int32), w.dtype), target_logits=to_dev(logits, "fp32")[None])
        acc_ref, out_ref = O.verify_greedy(drafted_ref, target_logits=logits[None])
        np.testing.assert_array_equal(acc.cpu().numpy(), acc_ref)
        np.testing.assert_array_equal(out.cpu().numpy(), out_ref)
        assert int(acc_ref[0]) >= planted_len


@pytest.mark.parametrize("rope", [0.0, 10000.0])
@pytest.mark.parametrize("w", [SMALL_GQA, SMALL_MHA], ids=lambda w: w.name)
def test_small_bf16_ragged_batch_sd_iterations(w, rope):
    """Several speculative-decoding iterations: draft chain, verify, append the accepted true states
    (also with the rotary option: positions continue across prefill, draft tail and reset)."""
    head_gpu, head_cpu, _ = build(w, max_ctx=w.ctx_max + 64, rope_theta=rope)
    rng = WL.data_rng(w)
    lengths = WL.make_context_lengths(w, rng)
    lengths[0] = w.ctx_min                           # the shortest cache (1 key for the GQA case)
    slots = list(range(w.batch))
    seqs = prefill_both(head_gpu, head_cpu, w, rng, slots, lengths)
    first = WL.make_tokens(w, rng, (w.batch,))
    for it in range(3):
        drafted, drafted_ref, _ = run_chain_parity(head_gpu, head_cpu, w, slots, seqs, first, w.gamma)
        target = WL.make_target_stream(w, rng, drafted_ref)
        acc, out = head_gpu.verify_greedy(to_dev(drafted_ref.astype(np.int32), w.dtype), target_ids=to_dev(target, w.dtype))
        acc_ref, out_ref = O.verify_greedy(drafted_ref, target_ids=target)
        np.testing.assert_array_equal(acc.cpu().numpy(), acc_ref)
        np.testing.assert_array_equal(out.cpu().numpy(), out_ref)
        new_len = (acc_ref + 1).astype(int)
        hidden = WL.make_hidden(w, rng, int(new_len.sum()))
        head_gpu.prefill_kv(slots, list(map(int, new_len)), to_dev(hidden, w.dtype))
        r = 0
        for b, s in enumerate(seqs):
            O.prefill_kv(head_cpu, s, hidden[r:r + new_len[b]])
            r += new_len[b]
            assert head_gpu.slot_lengths(b) == (s.n_true, 0)
        first = np.array([out_ref[b, acc_ref[b]] for b in range(w.batch)])


@pytest.mark.parametrize("batch,rope", [(9, 0.0), (20, 0.0), (20, 500000.0), (40, 0.0), (64, 0.0)])
def test_batched_serving_tensor_core_projections(batch, rope):
    """Batches above 8 rows take the tensor-core projections (weights as the wide operand, split
    reduction + finishing kernel); 9 / 20 / 40 / 64 rows cover the 16-, 32- and 64-column variants."""
    w = SMALL_GQA.scaled(batch=batch, ctx_min=3, ctx_max=300, gamma=3, seed=2003, mlp_dim=1416)
    head_gpu, head_cpu, _ = build(w, max_ctx=w.ctx_max + 64, rope_theta=rope)
    rng = WL.data_rng(w, batch)
    lengths = WL.make_context_lengths(w, rng)
    slots = list(rng.permutation(batch))                      # slot ids differ from batch rows
    slots = [int(s) for s in slots]
    seqs = prefill_both(head_gpu, head_cpu, w, rng, slots, lengths)          # > 64 rows: chunked / dense prefill
    first = WL.make_tokens(w, rng, (batch,))
    for it in range(2):
        drafted, drafted_ref, _ = run_chain_parity(head_gpu, head_cpu, w, slots, seqs, first, w.gamma)
        target = WL.make_target_stream(w, rng, drafted_ref)
        acc, out = head_gpu.verify_greedy(to_dev(drafted_ref.astype(np.int32), w.dtype), target_ids=to_dev(target, w.dtype))
        acc_ref, out_ref = O.verify_greedy(drafted_ref, target_ids=target)
        np.testing.assert_array_equal(acc.cpu().numpy(), acc_ref)
        new_len = (acc_ref + 1).astype(int)
        hidden = WL.make_hidden(w, rng, int(new_len.sum()))                  # 9..256 rows: tensor-core prefill in chunks
        head_gpu.prefill_kv(slots, list(map(int, new_len)), to_dev(hidden, w.dtype))
        r = 0
        for b, s in enumerate(seqs):
            O.prefill_kv(head_cpu, s, hidden[r:r + new_len[b]])
            r += new_len[b]
            assert head_gpu.slot_lengths(slots[b]) == (s.n_true, 0)
        first = np.array([out_ref[b, acc_ref[b]] for b in range(batch)])
    from paper_2505_24544_b200.binding import beagle_check_device
    beagle_check_device(head_gpu.ctx)


@pytest.mark.parametrize("batch", [4, 12])
def test_chain_continues_with_another_batch_composition(batch):
    """A step that continues from the device-resident greedy tokens may name fewer sequences, or another order, than the step
    before it (every sequence carries its own token, state and draft depth; batches of 8 rows or fewer and larger ones take different kernels)."""
    w = SMALL_GQA.scaled(batch=batch, ctx_min=5, ctx_max=200, gamma=4, seed=2011)
    head_gpu, head_cpu, _ = build(w, max_ctx=w.ctx_max + 64, max_draft=8)
    rng = WL.data_rng(w, batch)
    lengths = WL.make_context_lengths(w, rng)
    slots = [int(s) for s in rng.permutation(batch)]
    seqs = prefill_both(head_gpu, head_cpu, w, rng, slots, lengths)
    first = WL.make_tokens(w, rng, (batch,))
    drafted, _, _ = run_chain_parity(head_gpu, head_cpu, w, slots, seqs, first, 2)

    def step(rows, what):
        t, logits, hidden = head_gpu.draft_step([slots[r] for r in rows], tokens_in=None, want_logits=True, want_hidden=True)
        torch.cuda.synchronize()
        out = O.draft_step(head_cpu, [seqs[r] for r in rows], tokens_in=None)
        assert_close(logits.float().cpu().numpy(), out["logits"], w.dtype, what + " logits")
        assert_close(hidden.float().cpu().numpy(), out["h"], w.dtype, what + " hidden")
        gt = t.cpu().numpy()
        check_tokens(gt, out["logits"], what + " tokens")
        for r, tok in zip(rows, gt):
            seqs[r].pending_token = int(tok)              # near a tie either id is right: both sides go on from the library's

    for r in range(batch):
        seqs[r].pending_token = int(drafted[r, -1])
    sub = [batch - 1, 0, 2] + list(range(3, batch - 1, 2))
    step(sub, "permuted subset")
    step(sub, "same subset again")
    step(list(range(batch)), "all sequences, unequal depths")
    step(list(range(batch)), "all sequences again")
    from paper_2505_24544_b200.binding import beagle_check_device
    beagle_check_device(head_gpu.ctx)
    for r in range(batch):
        assert head_gpu.slot_lengths(slots[r]) == (int(lengths[r]), 5 if r in sub else 3)


@pytest.mark.parametrize("rope", [0.0, 10000.0])
def test_empty_cache_concat_off_and_rollback(rope):
    w = SMALL_GQA.scaled(batch=2)
    head_gpu, head_cpu, _ = build(w, rope_theta=rope)
    rng = WL.data_rng(w, 2)
    seqs = prefill_both(head_gpu, head_cpu, w, rng, [1, 0], [0, 300])      # slot 1 has no key at all
    first = WL.make_tokens(w, rng, (2,))
    run_chain_parity(head_gpu, head_cpu, w, [1, 0], seqs, first, 3, concat=False)
    assert head_gpu.slot_lengths(0) == (300, 0) and head_gpu.slot_lengths(1) == (0, 0)
    head_gpu.rollback([1, 0])
    for s in seqs:
        O.rollback(s)
    run_chain_parity(head_gpu, head_cpu, w, [1, 0], seqs, first, 4, concat=True)
    assert head_gpu.slot_lengths(1) == (0, 3)


@pytest.mark.parametrize("n", [127, 128, 129, 255, 256, 257, 513])
def test_split_kv_chunk_boundaries(n):
    w = SMALL_MHA.scaled(batch=1)
    head_gpu, head_cpu, _ = build(w, max_ctx=600)
    rng = WL.data_rng(w, n)
    seqs = prefill_both(head_gpu, head_cpu, w, rng, [0], [n])
    run_chain_parity(head_gpu, head_cpu, w, [0], seqs, WL.make_tokens(w, rng, (1,)), 2)


@pytest.mark.parametrize("block,offset,sim_steps,rope", [(4, 0, 1, 0.0), (4, 3, 1, 0.0), (4, 0, 4, 0.0), (4, 3, 4, 0.0), (3, 1, 2, 0.0), (1, 0, 1, 0.0),
                                                         (4, 3, 4, 10000.0), (5, 0, 4, 0.0)])
def test_block_forward_c1_fp32(block, offset, sim_steps, rope):
    w = WL.WORKLOADS["c1_tiny_fp32"]
    head_gpu, head_cpu, _ = build(w, rope_theta=rope)
    rng = WL.data_rng(w, 10 * block + offset)
    B, S = 2, 70
    tokens = WL.make_tokens(w, rng, (B, S))
    hidden = WL.make_hidden(w, rng, B * S).reshape(B, S, w.hidden)
    logits, argmax, hid = head_gpu.block_forward(to_dev(tokens, w.dtype), to_dev(hidden, w.dtype), block, offset, sim_steps)
    torch.cuda.synchronize()
    for b in range(B):
        ref = O.block_forward(head_cpu, tokens[b], hidden[b], block, offset, sim_steps)
        assert_close(logits[b].cpu().numpy(), ref["logits"], w.dtype, f"seq {b} logits")
        assert_close(hid[b].cpu().numpy(), ref["hidden"], w.dtype, f"seq {b} hidden")
        check_tokens(argmax[b].cpu().numpy(), ref["logits"], f"seq {b} argmax")


@pytest.mark.parametrize("sim_steps,rope", [(1, 0.0), (4, 0.0), (4, 10000.0)])
def test_block_forward_small_bf16_equals_oracle_and_sequential(sim_steps, rope):
    """Block forward against the oracle, and against the library's own step-by-step drafting
    (with the rotary option the two paths must also agree on every position)."""
    w = SMALL_GQA
    head_gpu, head_cpu, _ = build(w, max_slots=1, max_ctx=256, rope_theta=rope)
    rng = WL.data_rng(w, 77 + sim_steps)
    B, S, block, offset = 2, 131, 4, 2
    tokens = WL.make_tokens(w, rng, (B, S))
    hidden = WL.make_hidden(w, rng, B * S).reshape(B, S, w.hidden)
    tok_dev, hid_dev = to_dev(tokens, w.dtype), to_dev(hidden, w.dtype)
    logits, argmax, hid = head_gpu.block_forward(tok_dev, hid_dev, block, offset, sim_steps, want_logits=True)
    _, argmax_only, _ = head_gpu.block_forward(tok_dev, hid_dev, block, offset, sim_steps, want_logits=False, want_hidden=False)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(argmax.cpu().numpy(), argmax_only.cpu().numpy())
    for b in range(B):
        ref = O.block_forward(head_cpu, tokens[b], hidden[b], block, offset, sim_steps)
        assert_close(logits[b].cpu().numpy(), ref["logits"], w.dtype, f"seq {b} logits")
        assert_close(hid[b].float().cpu().numpy(), ref["hidden"], w.dtype, f"seq {b} hidden")
        check_tokens(argmax[b].cpu().numpy(), ref["logits"], f"seq {b} argmax")
    # the library's serve-time path reproduces its own block path (window starting after 66 states)
    n = O.visible_true_count(67, block, offset)
    head_gpu.prefill_kv([0], [n], hid_dev[0, :n].contiguous())
    for i in range(1, block + 1):
        _, lg, _ = head_gpu.draft_step([0], tokens_in=tok_dev[0, n + i - 1:n + i].contiguous(), concat=(i <= sim_steps), want_logits=True)
        assert_close(lg[0].cpu().numpy(), logits[0, n + i - 1].cpu().numpy().astype(np.float64), w.dtype, f"slot {i} block vs sequential")


@pytest.mark.parametrize("S,block,offset,sim_steps", [(200, 5, 0, 3), (64, 2, 7, 2), (193, 3, 190, 1), (130, 5, 2, 4)])
def test_block_forward_bf16_head_dim_128(S, block, offset, sim_steps):
    """Tensor-core block attention with 128-wide heads: several query/key tiles, a ragged last
    tile, an offset close to S (almost everything strict-causal) and the predicted-key band."""
    w = SMALL_MHA
    head_gpu, head_cpu, _ = build(w, max_slots=1, max_ctx=64)
    rng = WL.data_rng(w, 1000 + S)
    B = 2
    tokens = WL.make_tokens(w, rng, (B, S))
    hidden = WL.make_hidden(w, rng, B * S).reshape(B, S, w.hidden)
    logits, argmax, hid = head_gpu.block_forward(to_dev(tokens, w.dtype), to_dev(hidden, w.dtype), block, offset, sim_steps)
    torch.cuda.synchronize()
    for b in range(B):
        ref = O.block_forward(head_cpu, tokens[b], hidden[b], block, offset, sim_steps)
        assert_close(logits[b].cpu().numpy(), ref["logits"], w.dtype, f"seq {b} logits")
        assert_close(hid[b].float().cpu().numpy(), ref["hidden"], w.dtype, f"seq {b} hidden")
        check_tokens(argmax[b].cpu().numpy(), ref["logits"], f"seq {b} argmax")
    from paper_2505_24544_b200.binding import beagle_check_device
    beagle_check_device(head_gpu.ctx)


def rising_score_inputs(w, head_cpu, S, rng, top=14.0):
    """One repeated token and states h_j = a_j g + noise with g chosen so that query head 0's score of key j rises linearly
    from 0 to `top` (natural units) along the sequence; the other heads get other slopes, some falling."""
    tokens = np.full((1, S), int(WL.make_tokens(w, rng, (1,))[0]), dtype=np.int32)
    dh = w.head_dim
    q = O.rms_norm(O.embed_tokens(head_cpu, tokens[0][:1]), head_cpu.g_q, head_cpu.cfg.rms_eps)[0] @ head_cpu.w_q.T
    g = head_cpu.w_k[:dh].T @ q[:dh]
    gamma = np.linalg.norm(g)
    g /= gamma
    a = top * np.sqrt(dh) / gamma * np.arange(S) / (S - 1)
    hidden = WL.round_to_storage((a[:, None] * g[None, :] + 0.5 * WL.make_hidden(w, rng, S)).reshape(-1), w.dtype).reshape(1, S, w.hidden)
    k = hidden[0].astype(np.float64) @ head_cpu.w_k.T
    G = w.n_q_heads // w.n_kv_heads
    rise = np.array([(q[h * dh:(h + 1) * dh] @ (k[S - 8] - k[0])[(h // G) * dh:(h // G + 1) * dh]) / np.sqrt(dh) for h in range(w.n_q_heads)])
    return tokens, hidden, rise * np.log2(np.e)


@pytest.mark.parametrize("w,sim_steps", [(SMALL_MHA, 1), (SMALL_MHA, 3), (SMALL_GQA, 2)], ids=lambda v: getattr(v, "name", str(v)))
def test_block_attention_when_later_keys_dominate(w, sim_steps):
    """Scores that rise by 20 bits along the sequence for one query head (and fall for others): every row's largest scores lie in
    its LAST key tiles, so a kernel that keeps a reference point per row and accumulates against it has to move that point, and
    rescale what it has accumulated, several times per row.  Compared with the oracle in its bf16-storage mode (both sides then
    hold the same rounded q, k, v: at scores this large the unrounded oracle differs by what rounding k alone does to the weights)."""
    head_gpu, head_cpu, _ = build(w, max_slots=1, max_ctx=64)
    S, block = 330, 4
    tokens, hidden, rise_bits = rising_score_inputs(w, head_cpu, S, WL.data_rng(w, 4242 + sim_steps))
    assert rise_bits.max() > 16, rise_bits                       # the premise: more than two moves of 8 bits for some head
    logits, argmax, hid = head_gpu.block_forward(to_dev(tokens, w.dtype), to_dev(hidden, w.dtype), block, 0, sim_steps)
    torch.cuda.synchronize()
    ref = O.block_forward(head_cpu.with_storage("bf16"), tokens[0], hidden[0], block, 0, sim_steps)
    assert_close(hid[0].float().cpu().numpy(), ref["hidden"], w.dtype, "hidden")
    assert_close(logits[0].cpu().numpy(), ref["logits"], w.dtype, "logits")
    from paper_2505_24544_b200.binding import beagle_check_device
    beagle_check_device(head_gpu.ctx)


@pytest.mark.parametrize("name,stage,sim_steps,soft", [("c1", "early", 1, True), ("c1", "late", 3, False), ("gqa", "early", 1, False),
                                                        ("gqa", "late", 4, True), ("mha", "late", 2, True)])
def test_block_loss_forward(name, stage, sim_steps, soft):
    """Early (Eq. 4) and late (Eq. 7) losses: every position's cross-entropy and the weighted mean
    against the oracle.  c1 = fp32 (materialised logits), gqa / mha = bf16 (fused GEMM epilogue;
    V = 4099 / 5000 leave a ragged last column tile)."""
    w = {"c1": WL.WORKLOADS["c1_tiny_fp32"], "gqa": SMALL_GQA, "mha": SMALL_MHA}[name]
    head_gpu, head_cpu, _ = build(w, max_slots=1, max_ctx=64)
    rng = WL.data_rng(w, 500 + sim_steps)
    B, S, block, offset = 2, 75, 4, 2
    tokens = WL.make_tokens(w, rng, (B, S))
    hidden = WL.make_hidden(w, rng, B * S).reshape(B, S, w.hidden)
    tl = WL.round_to_storage((rng.standard_normal((B, S, w.vocab)) * 2).astype(np.float32).reshape(-1), w.dtype).reshape(B, S, w.vocab)
    ids = WL.make_tokens(w, rng, (B, S))
    kw = dict(target_logits=to_dev(tl, w.dtype)) if soft else dict(target_ids=to_dev(ids, w.dtype))
    loss, ce = head_gpu.block_loss(to_dev(tokens, w.dtype), to_dev(hidden, w.dtype), block, offset, stage, sim_steps=sim_steps, **kw)
    torch.cuda.synchronize()
    ref = O.block_loss(head_cpu, tokens, hidden, block, offset, stage, sim_steps=sim_steps,
                       **(dict(target_logits=tl) if soft else dict(target_ids=ids)))
    ce = ce.cpu().numpy().astype(np.float64)
    atol, rtol = (1e-4, 1e-4) if w.dtype == "fp32" else (3e-2, 1e-2)      # a cross-entropy moves by at most the largest logit error
    err = np.abs(ce - ref["ce"])
    assert np.all(err <= atol + rtol * np.abs(ref["ce"])), f"cross-entropy: max abs err {err.max():.3e}"
    # the scalar is the weighted mean of the library's own per-position values (fixed-order fp32 sum) ...
    own = float(np.sum(ce * ref["weights"][None, :]) / (B * ref["n_windows"]))
    assert abs(float(loss.item()) - own) <= 1e-5 * abs(own)
    # ... and agrees with the oracle's
    assert abs(float(loss.item()) - ref["loss"]) <= (1e-4 if w.dtype == "fp32" else 1e-2) * abs(ref["loss"])
    from paper_2505_24544_b200.binding import beagle_check_device
    beagle_check_device(head_gpu.ctx)


GRAD_TOL = {"fp32": (2e-4, 1e-5), "bf16": (4e-2, 2e-2)}     # (max error / max |ref|, Frobenius error / Frobenius norm)


@pytest.mark.parametrize("name,stage,sim_steps,soft,vcoef,rope", [("c1", "early", 1, True, 10.0, 0.0), ("c1", "late", 3, False, 0.0, 0.0),
                                                                   ("gqa", "early", 1, False, 10.0, 0.0), ("gqa", "late", 4, True, 10.0, 0.0),
                                                                   ("mha", "late", 2, True, 0.0, 0.0), ("c1", "late", 2, True, 10.0, 10000.0),
                                                                   ("mha", "late", 3, False, 10.0, 500000.0)])
def test_block_grad(name, stage, sim_steps, soft, vcoef, rope):
    """One training step (Eq. 4 / Eq. 7 plus the state regression of Appendix B): the three loss values and the
    gradient in every parameter against the oracle.  fp32: tight.  bf16: the intermediate gradients are stored
    in bf16 (relative 2^-9 each, a handful of stages deep) and each parameter gradient sums B*S of them, so the
    error is measured against the tensor's largest entry and in Frobenius norm."""
    w = {"c1": WL.WORKLOADS["c1_tiny_fp32"], "gqa": SMALL_GQA, "mha": SMALL_MHA}[name]
    head_gpu, head_cpu, _ = build(w, max_slots=1, max_ctx=64, rope_theta=rope)
    rng = WL.data_rng(w, 700 + sim_steps)
    B, S, block, offset = 2, 75, 4, 2
    tokens = WL.make_tokens(w, rng, (B, S))
    tokens[1, 5] = tokens[0, 7]                                            # a repeated token: its embedding rows add up
    hidden = WL.make_hidden(w, rng, B * S).reshape(B, S, w.hidden)
    tl = WL.round_to_storage((rng.standard_normal((B, S, w.vocab)) * 2).astype(np.float32).reshape(-1), w.dtype).reshape(B, S, w.vocab)
    ids = WL.make_tokens(w, rng, (B, S))
    kw = dict(target_logits=to_dev(tl, w.dtype)) if soft else dict(target_ids=to_dev(ids, w.dtype))
    losses, grads = head_gpu.block_grad(to_dev(tokens, w.dtype), to_dev(hidden, w.dtype), block, offset, stage, sim_steps=sim_steps,
                                        vloss_coef=vcoef, **kw)
    torch.cuda.synchronize()
    ref = O.block_loss_grad(head_cpu, tokens, hidden, block, offset, stage, sim_steps=sim_steps, vloss_coef=vcoef,
                            **(dict(target_logits=tl) if soft else dict(target_ids=ids)))
    got = losses.cpu().numpy().astype(np.float64)
    rel = 1e-4 if w.dtype == "fp32" else 1e-2
    assert abs(got[0] - ref["loss"]) <= rel * abs(ref["loss"])
    assert abs(got[1] - ref["vloss"]) <= rel * abs(ref["vloss"]) + 1e-7
    assert abs(got[2] - (got[0] + vcoef * got[1])) <= 1e-5 * abs(got[2])
    tol_max, tol_fro = GRAD_TOL[w.dtype]
    report = {}
    for pname, g_ref in ref["grads"].items():
        g = grads[pname].cpu().numpy().astype(np.float64)
        assert g.shape == g_ref.shape and np.all(np.isfinite(g)), pname
        scale = np.max(np.abs(g_ref))
        assert scale > 0, pname
        report[pname] = (np.max(np.abs(g - g_ref)) / scale, np.linalg.norm(g - g_ref) / np.linalg.norm(g_ref))
    bad = {k: v for k, v in report.items() if v[0] > tol_max or v[1] > tol_fro}
    assert not bad, f"gradient errors (max/max, fro/fro): {report}"
    from paper_2505_24544_b200.binding import beagle_check_device
    beagle_check_device(head_gpu.ctx)


def test_block_grad_subset_and_repeatability():
    """Only the requested gradients are written; two runs give the same bits for every fixed-order gradient."""
    w = SMALL_GQA
    head_gpu, _, _ = build(w, max_slots=1, max_ctx=64)
    rng = WL.data_rng(w, 733)
    B, S = 1, 41
    tokens = to_dev(WL.make_tokens(w, rng, (B, S)), w.dtype)
    hidden = to_dev(WL.make_hidden(w, rng, B * S).reshape(B, S, w.hidden), w.dtype)
    ids = to_dev(WL.make_tokens(w, rng, (B, S)), w.dtype)
    names = ("w_q", "w_k", "w_down", "g_mlp")
    l1, g1 = head_gpu.block_grad(tokens, hidden, 3, 0, "late", sim_steps=2, target_ids=ids, vloss_coef=10.0, params=names)
    l2, g2 = head_gpu.block_grad(tokens, hidden, 3, 0, "late", sim_steps=2, target_ids=ids, vloss_coef=10.0,
                                 params=("w_q", "w_k", "w_v", "w_o", "g_q", "g_mlp", "w_gate", "w_up", "w_down", "w_lm"))
    torch.cuda.synchronize()
    assert set(g1) == set(names)
    assert torch.equal(l1, l2)
    for n in names:
        assert torch.equal(g1[n], g2[n]), n


def test_verify_greedy_logits_both_dtypes_and_ties():
    w = SMALL_GQA.scaled(batch=5, gamma=6)
    head_gpu, _, _ = build(w)
    rng = WL.data_rng(w, 5)
    draft = WL.make_tokens(w, rng, (w.batch, w.gamma))
    planted = np.concatenate([draft, np.full((w.batch, 1), -1)], axis=1)
    planted[0, 3:] = -1; planted[1, :] = -1; planted[2, 5:] = -1; planted[3, 1:] = -1
    logits = WL.make_target_logits(w, rng, w.batch * (w.gamma + 1), planted.reshape(-1)).reshape(w.batch, w.gamma + 1, w.vocab)
    logits[4, 0, :] = 1.0                                  # an all-equal row: lowest index wins
    logits[4, 1, 7] = logits[4, 1, 4000] = 50.0            # a tie between two ids
    for dt in ("fp32", "bf16"):
        lg = WL.round_to_storage(logits.reshape(-1), dt).reshape(logits.shape)
        acc, out = head_gpu.verify_greedy(to_dev(draft, w.dtype), target_logits=to_dev(lg, dt))
        acc_ref, out_ref = O.verify_greedy(draft, target_logits=lg)
        np.testing.assert_array_equal(acc.cpu().numpy(), acc_ref)
        np.testing.assert_array_equal(out.cpu().numpy(), out_ref)
    assert out_ref[4, 0] == 0 or acc_ref[4] >= 0


@pytest.mark.parametrize("vocab", [50001, 8192, 37])
def test_verify_greedy_fused_slices_and_repeated_calls(vocab):
    """The one-launch verification from logits: rows cut into several slices (maxima planted at slice edges, in the unaligned
    head and tail of a slice, ties across slices), several batch / depth shapes on one context, and the same call twice in a
    row (the finishing CTA must leave the tickets ready for the next call).  Bit-exact against the oracle."""
    w = SMALL_GQA.scaled(vocab=vocab, batch=1, gamma=1)
    head_gpu, _, _ = build(w, max_slots=1, max_ctx=16)
    rng = WL.data_rng(w, vocab)
    for batch, gamma in ((1, 0), (1, 8), (3, 5), (32, 6), (64, 1)):
        logits = rng.standard_normal((batch, gamma + 1, vocab)).astype(np.float32)
        rows = logits.reshape(-1, vocab)
        edges = [0, vocab - 1] + [min(vocab - 1, max(0, e + d)) for e in range(4096, vocab, 4096) for d in (-9, -1, 0, 1, 8)]
        for r in range(rows.shape[0]):
            rows[r, edges[r % len(edges)]] = 30.0
            if r % 3 == 1:                                   # the same maximum again, further right: the lower index must win
                rows[r, min(vocab - 1, edges[r % len(edges)] + 4097)] = 30.0
        draft = rng.integers(0, vocab, (batch, gamma)).astype(np.int32)
        ids = O.argmax_lowest(logits)
        for b in range(batch):
            draft[b, :b % (gamma + 1)] = ids[b, :b % (gamma + 1)]
        for dt in ("fp32", "bf16"):
            lg = WL.round_to_storage(logits.reshape(-1), dt).reshape(logits.shape)
            acc_ref, out_ref = O.verify_greedy(draft, target_logits=lg)
            for _ in range(2):
                acc, out = head_gpu.verify_greedy(to_dev(draft, w.dtype), target_logits=to_dev(lg, dt))
                np.testing.assert_array_equal(acc.cpu().numpy(), acc_ref)
                np.testing.assert_array_equal(out.cpu().numpy(), out_ref)


def check_verify_sample(head_gpu, w, rng, batch, gamma, dt, temperature, logit_scale=2.0):
    """beagle_verify_sample against the oracle.  Integer outputs are bit-exact wherever the oracle's
    decision margins (|u - ratio| of the acceptance tests, distance of u_resample to a CDF
    boundary) exceed what fp32 sums over the vocabulary can move; those are all but a few rows."""
    V = w.vocab
    zq = (rng.standard_normal((gamma, batch, V)) * logit_scale).astype(np.float32)
    zp = WL.round_to_storage((zq.transpose(1, 0, 2)[:, :, :] * 0.7 + rng.standard_normal((batch, gamma, V)) * logit_scale * 0.7).reshape(-1), dt)
    zp = np.concatenate([zp.reshape(batch, gamma, V), WL.round_to_storage((rng.standard_normal((batch, 1, V)) * logit_scale).reshape(-1), dt).reshape(batch, 1, V)], axis=1)
    q = O.softmax_rows(zq, temperature)
    draft = np.array([[rng.choice(V, p=q[i, b]) for i in range(gamma)] for b in range(batch)], dtype=np.int32).reshape(batch, gamma)
    ua = rng.random((batch, gamma), dtype=np.float32)
    ur = rng.random(batch, dtype=np.float32)
    ref = O.verify_sample(draft, zq, zp, ua, ur, temperature)
    acc, out = head_gpu.verify_sample(to_dev(draft, w.dtype), to_dev(zq, "fp32"), to_dev(zp, dt), to_dev(ua, "fp32"), to_dev(ur, "fp32"), temperature)
    acc, out = acc.cpu().numpy(), out.cpu().numpy()
    # acceptance tests: exact wherever u is not within 1e-4 of the ratio (fp32 log-sum-exp over V moves it by ~1e-6)
    sure = ref["accept_margin"] > 1e-4
    assert sure.mean() >= 0.9
    np.testing.assert_array_equal(acc[sure], ref["accept_len"][sure])
    p_all = O.softmax_rows(zp, temperature)
    exact = 0
    for b in range(batch):
        a = int(acc[b])
        # every row: a valid result shape (accepted drafts, one extra token, padding)
        assert 0 <= a <= gamma and np.array_equal(out[b, :a], draft[b, :a]) and 0 <= out[b, a] < V and np.all(out[b, a + 1:] == -1)
        if a != ref["accept_len"][b]:
            continue
        # the extra token: u_resample must fall into the token's interval of the oracle's fp64 CDF, up to the 2e-5 that
        # an fp32 running sum over the vocabulary can be off (at V = 128256 the intervals themselves are ~1e-5 wide,
        # so only this statement, not equality, is meaningful there); equal to the oracle's token when r is clear of a boundary
        cdf = np.cumsum(O.residual_distribution(p_all[b, a], q[a, b] if a < gamma else None))
        v = int(out[b, a])
        lo = cdf[v - 1] if v > 0 else 0.0
        assert lo - 2e-5 <= ur[b] <= cdf[v] + 2e-5, (b, v, lo, float(ur[b]), cdf[v])
        if ref["resample_margin"][b] > 2e-5:
            assert v == ref["out_tokens"][b, a]
        exact += int(v == ref["out_tokens"][b, a])
    assert exact >= 0.5 * batch
    return ref


@pytest.mark.parametrize("dt,temperature", [("fp32", 1.0), ("bf16", 0.7)])
def test_verify_sample_small(dt, temperature):
    w = SMALL_GQA.scaled(batch=24, gamma=5)
    head_gpu, _, _ = build(w)
    rng = WL.data_rng(w, 31)
    ref = check_verify_sample(head_gpu, w, rng, 24, 5, dt, temperature)
    assert 0 < ref["accept_len"].mean() < 5                      # both rejections and acceptances occur
    check_verify_sample(head_gpu, w, rng, 3, 0, dt, temperature)  # gamma = 0: only the extra token, drawn from p_1
    # p == q: everything is accepted and the extra token comes from p_{gamma+1}
    z = rng.standard_normal((2, 4, w.vocab)).astype(np.float32)
    draft = rng.integers(0, w.vocab, (4, 2)).astype(np.int32)
    zp = np.concatenate([z.transpose(1, 0, 2), rng.standard_normal((4, 1, w.vocab)).astype(np.float32)], axis=1)
    ua, ur = rng.random((4, 2), dtype=np.float32), rng.random(4, dtype=np.float32)
    acc, out = head_gpu.verify_sample(to_dev(draft, w.dtype), to_dev(z, "fp32"), to_dev(zp, "fp32"), to_dev(ua, "fp32"), to_dev(ur, "fp32"))
    ref = O.verify_sample(draft, z, zp, ua, ur)
    assert acc.cpu().numpy().tolist() == [2, 2, 2, 2] == ref["accept_len"].tolist()
    np.testing.assert_array_equal(out.cpu().numpy(), ref["out_tokens"])


def tree_paths(tokens, parents, scores):
    """{token path from the root: score} of a tree given as parallel arrays."""
    out = {}
    for n in range(len(tokens)):
        path, a = [], n
        while a >= 0:
            path.append(int(tokens[a])); a = int(parents[a])
        out[tuple(path[::-1])] = float(scores[n])
    return out


@pytest.mark.parametrize("name,n_ctx,depth,topk,n_cand,seed,rope", [("gqa", 300, 3, 4, 20, 908, 0.0), ("mha", 130, 6, 10, 60, 904, 0.0),
                                                                     ("gqa", 0, 2, 3, 9, 903, 0.0), ("gqa", 77, 0, 5, 5, 900, 0.0),
                                                                     ("gqa", 300, 3, 4, 20, 908, 10000.0)])
def test_draft_tree_and_tree_verification(name, n_ctx, depth, topk, n_cand, seed, rope):
    """Dynamic draft tree against the oracle.  Which node wins a selection is a floating-point decision
    (dozens of top-k cuts with gaps down to 1e-3), so: what is unique is compared -- every kept path's
    score against the oracle's replay of that path, the kept set itself wherever the oracle's smallest
    selection gap is clear -- and the rest is checked to be valid: every kept child lies in the oracle's
    top-k of its parent up to the tolerance, and the sets overlap.  Then greedy acceptance along the tree."""
    w = {"gqa": SMALL_GQA, "mha": SMALL_MHA}[name].scaled(batch=1)
    from paper_2505_24544_b200.binding import BeagleHead
    weights = WL.make_weights(w)
    weights["w_lm"] = weights["w_lm"] * 32.0          # peaked next-token distributions (still exact in bf16)
    head_gpu = BeagleHead.from_workload(w, weights, max_slots=2, max_ctx=n_ctx + 8, max_draft=64, rope_theta=rope)
    head_cpu = oracle_head(w, weights, rope_theta=rope)
    rng = WL.data_rng(w, seed)
    seqs = prefill_both(head_gpu, head_cpu, w, rng, [1], [n_ctx])
    root = WL.make_tokens(w, rng, (1,))
    ref = O.draft_tree(head_cpu, seqs[0], int(root[0]), depth, topk, n_cand)
    tok, par, sc = head_gpu.draft_tree(1, to_dev(root, w.dtype), depth, topk, n_cand)
    torch.cuda.synchronize()
    tok, par, sc = tok.cpu().numpy(), par.cpu().numpy(), sc.cpu().numpy()
    assert head_gpu.slot_lengths(1) == (n_ctx, 0)
    assert np.all(par < np.arange(n_cand)) and np.all(par >= -1)
    got, want = tree_paths(tok, par, sc), tree_paths(ref["tokens"], ref["parents"], ref["scores"])
    assert len(got) == n_cand                                     # siblings are distinct tokens
    step_tol = 3e-2                                               # one log-probability of bf16 logits (2e-2 + 1e-2 |z|, |z| ~ 1)
    # (1) every kept path replayed by the oracle (forced chain drafting with concatenation): same score;
    #     every kept child within the oracle's top-k of its parent
    for path, score in got.items():
        total, feed = 0.0, int(root[0])
        for t in path:
            out = O.draft_step(head_cpu, seqs, tokens_in=[feed], concat=True)
            lq = O.log_softmax_rows(out["logits"][0])
            kth = np.sort(lq)[-topk]
            assert lq[t] >= kth - 2 * step_tol, (path, t, float(lq[t]), float(kth))
            total += lq[t]
            feed = t
        O.rollback(seqs[0])
        assert abs(score - total) <= len(path) * step_tol, (path, score, total)
    # (2) the kept set: identical where every selection gap of the oracle is clear, overlapping otherwise
    if ref["cut_margin"] > 2 * (depth + 1) * step_tol:
        assert set(got) == set(want), "the selected token paths differ although every selection margin is clear"
    assert len(set(got) & set(want)) >= 0.7 * n_cand
    worst_kept = min(want.values())
    assert min(got.values()) >= worst_kept - 2 * (depth + 1) * step_tol
    # greedy acceptance along the tree, on the library's own tree: follow one of its leaves, then deviate
    n = n_cand
    leaf = int(np.argmax([len(k) for k in tree_paths(tok, par, sc)]))          # a deepest node
    chain, a = [], leaf
    while a >= 0:
        chain.append(a); a = int(par[a])
    chain = chain[::-1]
    target = WL.make_tokens(w, rng, (n + 1,)).astype(np.int32)
    target[0] = tok[chain[0]]
    for i in range(len(chain) - 1):
        target[1 + chain[i]] = tok[chain[i + 1]]
    for cut_at in (len(chain), 1, 0):
        tgt = target.copy()
        if cut_at < len(chain):                                                   # break the path after cut_at nodes
            idx = 0 if cut_at == 0 else 1 + chain[cut_at - 1]
            tgt[idx] = (int(tgt[idx]) + 1) % w.vocab
            while any(par[j] == (chain[cut_at - 1] if cut_at else -1) and tok[j] == tgt[idx] for j in range(n)):
                tgt[idx] = (int(tgt[idx]) + 1) % w.vocab
        acc, out, path = head_gpu.verify_tree_greedy(to_dev(tok, w.dtype), to_dev(par, w.dtype), to_dev(tgt, w.dtype), depth + 2)
        a_ref, out_ref, path_ref = O.verify_tree_greedy(tok, par, int(tgt[0]), tgt[1:])
        assert int(acc.item()) == a_ref == cut_at
        assert out.cpu().numpy()[:a_ref + 1].tolist() == out_ref.tolist() and np.all(out.cpu().numpy()[a_ref + 1:] == -1)
        assert path.cpu().numpy()[:a_ref].tolist() == path_ref.tolist()
    from paper_2505_24544_b200.binding import beagle_check_device
    beagle_check_device(head_gpu.ctx)


def test_argmax_rules_nan_negative_zero_and_largest_call():
    """Arg-max conventions on the GPU (lowest index on ties, NaN never wins, -0 equals +0) and the
    largest verification call the ABI admits (64 sequences x gamma 64)."""
    w = SMALL_GQA.scaled(batch=64, gamma=64)
    head_gpu, _, _ = build(w, max_slots=1, max_ctx=16)
    rng = WL.data_rng(w, 64)
    V = w.vocab
    logits = rng.standard_normal((64, 65, V)).astype(np.float32)
    logits[0, 0, :] = np.nan                                   # an all-NaN row: id 0
    logits[0, 1, 5] = np.nan; logits[0, 1, 6] = 9.0            # NaN next to the maximum
    logits[0, 2, :] = -0.0; logits[0, 2, 17] = 0.0             # -0 == +0: lowest index wins, not the +0
    logits[0, 3, :] = -np.inf; logits[0, 3, 4098] = -1e30      # the last id of a row whose length is not a multiple of 8
    draft = rng.integers(0, V, (64, 64)).astype(np.int32)
    ref_ids = O.argmax_lowest(logits)
    draft[1, :] = ref_ids[1, :64]                              # one sequence accepts everything
    draft[2, :10] = ref_ids[2, :10]
    acc, out = head_gpu.verify_greedy(to_dev(draft, w.dtype), target_logits=to_dev(logits, "fp32"))
    acc_ref, out_ref = O.verify_greedy(draft, target_logits=logits)
    np.testing.assert_array_equal(acc.cpu().numpy(), acc_ref)
    np.testing.assert_array_equal(out.cpu().numpy(), out_ref)
    assert ref_ids[0, 0] == 0 and ref_ids[0, 1] == 6 and ref_ids[0, 2] == 0 and ref_ids[0, 3] == 4098
    assert acc_ref[1] == 64 and acc_ref[2] >= 10
    from paper_2505_24544_b200.binding import BeagleError
    with pytest.raises(BeagleError) as e:                      # one more sequence than a call admits
        head_gpu.verify_greedy(torch.zeros(65, 4, dtype=torch.int32, device="cuda"), target_ids=torch.zeros(65, 5, dtype=torch.int32, device="cuda"))
    assert e.value.status == 3


@pytest.mark.parametrize("batch", [2, 12])
def test_draft_chain_replays_from_a_cuda_graph(batch):
    """The draft chain enqueues kernels only (no host synchronisation, tokens fed device to device), so it
    can be captured once and replayed: the replay reproduces the eager tokens bit for bit."""
    w = SMALL_GQA.scaled(batch=batch, gamma=4)
    head_gpu, _, _ = build(w, max_ctx=400)
    rng = WL.data_rng(w, 123)
    lengths = WL.make_context_lengths(w.scaled(ctx_min=100, ctx_max=300), rng)
    slots = list(range(batch))
    hidden = to_dev(WL.make_hidden(w, rng, int(lengths.sum())), w.dtype)
    first = to_dev(WL.make_tokens(w, rng, (batch,)), w.dtype)
    target = to_dev(WL.make_tokens(w, rng, (batch, w.gamma + 1)), w.dtype)
    from paper_2505_24544_b200 import binding as B

    def chain(draft, acc, out):
        for s in range(w.gamma):
            B.beagle_draft_step(head_gpu.ctx, slots, first if s == 0 else None, True, draft[:, s])
        B.beagle_verify_greedy(head_gpu.ctx, draft, None, target, acc, out)

    def fresh():
        return (torch.zeros(batch, w.gamma, dtype=torch.int32, device="cuda"), torch.zeros(batch, dtype=torch.int32, device="cuda"),
                torch.zeros(batch, w.gamma + 1, dtype=torch.int32, device="cuda"))

    head_gpu.prefill_kv(slots, [int(n) for n in lengths], hidden)
    eager = fresh()
    chain(*eager)                                    # also the first call on this device: one-time set-up happens here
    torch.cuda.synchronize()
    head_gpu.rollback(slots)
    captured = fresh()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        chain(*captured)
    for _ in range(2):
        for t in captured:
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        for a, b in zip(eager, captured):
            assert torch.equal(a, b)
    assert int(eager[0].abs().sum()) > 0


def test_status_codes_for_capacity_and_state():
    from paper_2505_24544_b200.binding import BeagleError
    w = SMALL_GQA.scaled(batch=1, gamma=2)
    head_gpu, _, _ = build(w, max_ctx=16, max_draft=1)
    rng = WL.data_rng(w, 9)
    with pytest.raises(BeagleError) as e:
        head_gpu.prefill_kv([0], [17], to_dev(WL.make_hidden(w, rng, 17), w.dtype))
    assert e.value.status == 3
    with pytest.raises(BeagleError) as e:
        head_gpu.draft_step([0], tokens_in=None)
    assert e.value.status == 4
    head_gpu.prefill_kv([0], [16], to_dev(WL.make_hidden(w, rng, 16), w.dtype))
    tok = to_dev(WL.make_tokens(w, rng, (1,)), w.dtype)
    head_gpu.draft_step([0], tokens_in=tok)
    head_gpu.draft_step([0])
    with pytest.raises(BeagleError) as e:                  # the draft tail is full (max_draft = 1)
        head_gpu.draft_step([0])
    assert e.value.status == 3
    with pytest.raises(BeagleError) as e:
        head_gpu.draft_step([0, 0], tokens_in=torch.zeros(2, dtype=torch.int32, device="cuda"))
    assert e.value.status == 1
    torch.cuda.synchronize()


def test_status_codes_of_pack_weights():
    """Buffer too small: CAPACITY; misaligned: INVALID_ARG; an fp32 head accepts the call and needs no bytes."""
    import ctypes as C
    from paper_2505_24544_b200 import binding as B
    w = SMALL_GQA.scaled(batch=12)
    head, _, _ = build(w, pack_weights=False)
    lib, n = head.ctx.lib, B.beagle_packed_weights_bytes(head.cfg, False)
    assert n > 0 and head.ctx.packed_buf is None
    buf = torch.empty(n + 512, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    assert lib.beagle_pack_weights(head.ctx.handle, buf.data_ptr(), n - 1, stream) == 3
    assert "packed weights need" in lib.beagle_last_error(head.ctx.handle).decode()
    assert lib.beagle_pack_weights(head.ctx.handle, buf.data_ptr() + 16, n, stream) == 1
    assert lib.beagle_pack_weights(head.ctx.handle, buf.data_ptr(), n, stream) == 0
    assert lib.beagle_pack_weights(head.ctx.handle, None, 0, stream) == 0
    torch.cuda.synchronize()
    c1 = WL.WORKLOADS["c1_tiny_fp32"]
    head32, _, _ = build(c1)
    assert head32.ctx.packed_buf is None and B.beagle_packed_weights_bytes(head32.cfg, False) == 0
    assert lib.beagle_pack_weights(head32.ctx.handle, buf.data_ptr(), n, stream) == 0
    B.beagle_check_device(head.ctx)


def test_status_codes_of_the_training_entry_points():
    """Argument errors of beagle_block_loss / beagle_block_grad are reported before any launch."""
    from paper_2505_24544_b200.binding import BeagleError
    w = SMALL_GQA
    head_gpu, _, _ = build(w, max_slots=1, max_ctx=16)
    rng = WL.data_rng(w, 11)
    tokens = to_dev(WL.make_tokens(w, rng, (1, 12)), w.dtype)
    hidden = to_dev(WL.make_hidden(w, rng, 12).reshape(1, 12, w.hidden), w.dtype)
    ids = to_dev(WL.make_tokens(w, rng, (1, 12)), w.dtype)
    tl = torch.zeros(1, 12, w.vocab, dtype=torch.float32, device="cuda")
    for kw in (dict(stage="early", sim_steps=2, target_ids=ids),                 # the early stage has no simulation
               dict(stage="late", sim_steps=5, target_ids=ids),                  # sim_steps > block
               dict(stage="late", sim_steps=2),                                  # no target at all
               dict(stage="late", sim_steps=2, target_ids=ids, target_logits=tl),   # both targets
               dict(stage="late", sim_steps=2, target_ids=ids, vloss_coef=-1.0)):
        with pytest.raises(BeagleError) as e:
            head_gpu.block_grad(tokens, hidden, 4, 0, **kw)
        assert e.value.status == 1, kw
    with pytest.raises(BeagleError) as e:
        head_gpu.block_loss(tokens, hidden, 4, 12, "early", target_ids=ids)      # offset must lie inside the sequence
    assert e.value.status == 1
    # and a valid call still works afterwards
    losses, grads = head_gpu.block_grad(tokens, hidden, 4, 0, "late", sim_steps=2, target_ids=ids, vloss_coef=10.0, params=("w_o",))
    torch.cuda.synchronize()
    assert torch.isfinite(losses).all() and torch.isfinite(grads["w_o"]).all()


@pytest.mark.parametrize("name,S,block,offset,sim_steps", [("gqa", 1, 1, 0, 1), ("gqa", 2, 4, 0, 2), ("mha", 127, 4, 0, 4), ("mha", 128, 3, 1, 3),
                                                           ("gqa", 129, 5, 128, 2), ("gqa", 257, 4, 3, 4)])
def test_block_forward_and_grad_tile_edges(name, S, block, offset, sim_steps):
    """Sequence lengths around the 128-query / 64-key tiles of the tensor-core attention kernels (and the degenerate
    S = 1, where no query sees a key): forward logits and one training step against the oracle."""
    w = {"gqa": SMALL_GQA, "mha": SMALL_MHA}[name]
    head_gpu, head_cpu, _ = build(w, max_slots=1, max_ctx=64)
    rng = WL.data_rng(w, 900 + S)
    B = 2
    tokens = WL.make_tokens(w, rng, (B, S))
    hidden = WL.make_hidden(w, rng, B * S).reshape(B, S, w.hidden)
    ids = WL.make_tokens(w, rng, (B, S))
    tok_dev, hid_dev = to_dev(tokens, w.dtype), to_dev(hidden, w.dtype)
    logits, argmax, hid = head_gpu.block_forward(tok_dev, hid_dev, block, offset, sim_steps)
    torch.cuda.synchronize()
    for b in range(B):
        ref = O.block_forward(head_cpu, tokens[b], hidden[b], block, offset, sim_steps)
        assert_close(logits[b].cpu().numpy(), ref["logits"], w.dtype, f"seq {b} logits")
        check_tokens(argmax[b].cpu().numpy(), ref["logits"], f"seq {b} argmax")
    losses, grads = head_gpu.block_grad(tok_dev, hid_dev, block, offset, "late", sim_steps=sim_steps, target_ids=to_dev(ids, w.dtype),
                                        vloss_coef=10.0)
    torch.cuda.synchronize()
    ref = O.block_loss_grad(head_cpu, tokens, hidden, block, offset, "late", sim_steps=sim_steps, target_ids=ids, vloss_coef=10.0)
    assert abs(float(losses[0]) - ref["loss"]) <= 1e-2 * abs(ref["loss"]) + 1e-6
    tol_max, tol_fro = GRAD_TOL[w.dtype]
    for pname, g_ref in ref["grads"].items():
        g = grads[pname].cpu().numpy().astype(np.float64)
        scale = np.max(np.abs(g_ref))
        if scale == 0:       # no key, or a single key (softmax of one score is constant): no gradient reaches the query side
            assert np.max(np.abs(g)) <= 1e-8, pname      # the GPU's is rounding residue of delta = dO . bf16(O) against dO . V
            continue
        assert np.max(np.abs(g - g_ref)) <= tol_max * scale, (pname, np.max(np.abs(g - g_ref)) / scale)
        assert np.linalg.norm(g - g_ref) <= tol_fro * np.linalg.norm(g_ref), pname
    from paper_2505_24544_b200.binding import beagle_check_device
    beagle_check_device(head_gpu.ctx)


@pytest.mark.parametrize("dt", ["bf16", "fp32"])
def test_quantize_rows_e4m3_codes_are_bit_exact(dt):
    """The FP8 codes are an integer decision: the oracle takes it in the kernel's precision (float32 scale and quotient,
    round to nearest even, saturating), so codes and scales must agree exactly."""
    from paper_2505_24544_b200.binding import beagle_quantize_rows_e4m3
    rng = np.random.default_rng(77)
    x = (rng.standard_normal((37, 520)) * np.exp(rng.normal(0, 2, (37, 1)))).astype(np.float32)
    x[5] = 0.0                                                     # an all-zero row: scale 1, codes 0
    x[6, 3] = 3.0e4                                                # one dominant entry: the rest falls into the subnormals
    x = WL.round_to_storage(x.reshape(-1), dt).reshape(x.shape)
    q, scale = beagle_quantize_rows_e4m3(to_dev(x, dt))
    torch.cuda.synchronize()
    q_ref, s_ref = O.quantize_rows_e4m3(x)
    np.testing.assert_array_equal(scale.cpu().numpy().astype(np.float64), s_ref)
    got = q.view(torch.float8_e4m3fn).to(torch.float32).cpu().numpy().astype(np.float64)
    np.testing.assert_array_equal(got, q_ref)


@pytest.mark.parametrize("batch", [9, 33, 64])
def test_fp8_lm_head_batched_draft_steps(batch):
    """Optional FP8 LM head (draft steps of more than 8 rows): logits against the oracle's quantised product of the
    library's own states of that step, then the greedy tokens; the rest of the step is the ordinary bf16 path."""
    from paper_2505_24544_b200.binding import BeagleHead, beagle_workspace_buffer, beagle_check_device
    w = SMALL_GQA.scaled(batch=batch, ctx_min=3, ctx_max=200, gamma=3, seed=2005, vocab=4099)
    weights = WL.make_weights(w)
    head_gpu = BeagleHead.from_workload(w, weights, max_ctx=w.ctx_max + 64, fp8_lm_head=True)
    head_cpu = oracle_head(w, weights)
    rng = WL.data_rng(w, batch)
    lengths = WL.make_context_lengths(w, rng)
    slots = list(range(batch))
    prefill_both(head_gpu, head_cpu, w, rng, slots, lengths)
    first = to_dev(WL.make_tokens(w, rng, (batch,)), w.dtype)
    for step in range(3):
        tok, logits, _ = head_gpu.draft_step(slots, tokens_in=first if step == 0 else None, want_logits=True)
        torch.cuda.synchronize()
        h = beagle_workspace_buffer(head_gpu.ctx, "h", batch).float().cpu().numpy().astype(np.float64)
        z_ref = O.lm_head_fp8(head_cpu, h)
        z = logits.cpu().numpy().astype(np.float64)
        err = np.abs(z - z_ref)
        assert np.all(err <= 1e-3 + 1e-3 * np.abs(z_ref)), f"step {step}: max abs err {err.max():.3e}"   # fp32 sums of exact FP8 products
        check_tokens(tok.cpu().numpy(), z_ref, f"step {step} greedy token")
        # and the quantised head is a usable stand-in for the bf16 one (3 fraction bits, averaged over 512 terms)
        z_bf16 = O.lm_head(head_cpu, h)
        assert np.max(np.abs(z_ref - z_bf16)) < 0.1 * np.max(np.abs(z_bf16))
    beagle_check_device(head_gpu.ctx)


@pytest.mark.parametrize("batch,fp8", [(12, False), (33, False), (64, True)])
def test_packed_weight_copies_give_the_same_bits_and_follow_a_repack(batch, fp8):
    """The tile-major weight copies are a re-layout only: a chain of batched draft steps gives bit-identical logits,
    states and tokens with and without them (sizes that leave ragged tiles in both directions: 1416 and 4099 rows, 520-
    and 1416-element reductions); after a weight changes in place, a repack follows it and a head without copies agrees."""
    from paper_2505_24544_b200.binding import (BeagleHead, beagle_pack_weights, beagle_packed_weights_bytes, beagle_check_device,
                                               beagle_reset_slot)
    w = SMALL_GQA.scaled(batch=batch, hidden=528 if fp8 else 520, ctx_min=3, ctx_max=150, gamma=3, seed=2011, mlp_dim=1416, vocab=4099)
    weights = WL.make_weights(w)
    heads = [BeagleHead.from_workload(w, weights, max_ctx=w.ctx_max + 64, fp8_lm_head=fp8, pack_weights=pk) for pk in (True, False)]
    assert heads[0].ctx.packed_buf is not None and heads[1].ctx.packed_buf is None
    assert heads[0].ctx.packed_buf.numel() == beagle_packed_weights_bytes(heads[0].cfg, fp8)
    rng = WL.data_rng(w, batch)
    lengths = WL.make_context_lengths(w, rng)
    hidden = to_dev(WL.make_hidden(w, rng, int(np.sum(lengths))), w.dtype)
    first = to_dev(WL.make_tokens(w, rng, (batch,)), w.dtype)
    slots = list(range(batch))

    def chain(head):
        for slot in slots:
            beagle_reset_slot(head.ctx, slot)
        head.prefill_kv(slots, list(map(int, lengths)), hidden)
        out = []
        for step in range(3):
            out.append(head.draft_step(slots, tokens_in=first if step == 0 else None, want_logits=True, want_hidden=True))
        torch.cuda.synchronize()
        return out

    def same(a, b, what):
        for step, (x, y) in enumerate(zip(a, b)):
            for name, u, v in zip(("tokens", "logits", "hidden"), x, y):
                assert torch.equal(u, v), f"{what}: step {step} {name} differ"

    ref = chain(heads[1])
    same(chain(heads[0]), ref, "packed vs row-major")
    # a weight changes in place: the copies are stale until the repack, then both heads agree again
    for head in heads:
        head.ctx.weights["w_gate"].mul_(-0.5)
        head.ctx.weights["w_lm"][::3].mul_(0.25)
        if fp8:
            head.ctx.weights["w_lm_fp8"][::5] ^= 0x80          # flips the sign of every fifth row's codes
    ref2 = chain(heads[1])
    assert not torch.equal(ref2[0][1], ref[0][1])
    stale = chain(heads[0])
    assert torch.equal(stale[0][1], ref[0][1]), "the copies do not follow the weights by themselves"
    beagle_pack_weights(heads[0].ctx)
    same(chain(heads[0]), ref2, "after repack")
    beagle_pack_weights(heads[0].ctx, enable=False)
    same(chain(heads[0]), ref2, "copies dropped")
    for head in heads:
        beagle_check_device(head.ctx)


def test_bounded_wait_runs_out_and_is_reported_once():
    """The device error path without any fault or hang: a one-CTA kernel polls, with a short limit, a barrier that nothing
    completes and no copy targets; it gives up, raises the context's error word and returns.  beagle_check_device then
    reports BEAGLE_ERR_DEVICE exactly once, and the context keeps working (a draft step still matches the oracle)."""
    from paper_2505_24544_b200.binding import BeagleError, beagle_check_device, beagle_selftest_wait_timeout
    w = SMALL_GQA.scaled(batch=2, gamma=2)
    head_gpu, head_cpu, _ = build(w, max_ctx=64)
    rng = WL.data_rng(w, 321)
    seqs = prefill_both(head_gpu, head_cpu, w, rng, [0, 1], [20, 33])
    beagle_check_device(head_gpu.ctx)                       # nothing raised so far
    beagle_selftest_wait_timeout(head_gpu.ctx)
    with pytest.raises(BeagleError) as e:
        beagle_check_device(head_gpu.ctx)
    assert e.value.status == 7 and "bounded wait" in str(e.value)
    beagle_check_device(head_gpu.ctx)                       # reported once, then clear
    first = WL.make_tokens(w, rng, (2,))
    _, _, err = run_chain_parity(head_gpu, head_cpu, w, [0, 1], seqs, first, w.gamma)
    assert err <= 2e-2 + 1e-2 * 20
    beagle_check_device(head_gpu.ctx)


def test_first_call_inside_stream_capture_is_refused():
    """A context's first launching call zeroes device words and waits for that; inside a stream capture that work would only be
    recorded, so the call is refused with BEAGLE_ERR_STATE and nothing is launched.  After one ordinary call the same
    sequence captures and replays."""
    from paper_2505_24544_b200 import binding as B
    w = SMALL_GQA.scaled(batch=2, gamma=2)
    head_gpu, head_cpu, _ = build(w, max_ctx=64)
    rng = WL.data_rng(w, 99)
    hidden = to_dev(WL.make_hidden(w, rng, 30), w.dtype)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    launched = head_gpu.launch_count                         # the weight re-layout at construction
    with pytest.raises(B.BeagleError) as e:
        with torch.cuda.graph(g, stream=side):
            head_gpu.prefill_kv([0, 1], [10, 20], hidden)
    assert e.value.status == 4 and "capture" in str(e.value)
    assert head_gpu.slot_lengths(0) == (0, 0) and head_gpu.launch_count == launched
    torch.cuda.synchronize()
    head_gpu.prefill_kv([0, 1], [10, 20], hidden)            # the ordinary first call
    assert head_gpu.slot_lengths(1) == (20, 0)
    B.beagle_check_device(head_gpu.ctx)


@pytest.mark.parametrize("w", [SMALL_GQA, SMALL_MHA], ids=lambda w: w.name)
def test_dense_prefill_every_cache_row_across_tile_sequence_and_head_boundaries(w):
    """The tensor-core prefill (more than 512 rows: one GEMM over W_k and W_v side by side, cache rows written whole) on a
    ragged batch whose sequence boundaries fall inside the 128-row tiles; with 64-wide heads a 128-column tile holds two
    K/V heads.  EVERY cache row of every sequence is compared with the oracle's projection, then a second call appends
    another 600 rows behind the first ones (positions that do not start at zero) and is checked the same way."""
    w = w.scaled(batch=5)
    head_gpu, head_cpu, _ = build(w, max_slots=6, max_ctx=1000)
    rng = WL.data_rng(w, 512)
    slots = [4, 0, 3, 1, 5]
    base = {s: 0 for s in slots}
    for lengths in ([100, 130, 7, 300, 200], [129, 1, 255, 90, 125]):
        assert sum(lengths) > 512
        hidden = WL.make_hidden(w, rng, sum(lengths))
        head_gpu.prefill_kv(slots, lengths, to_dev(hidden, w.dtype))
        torch.cuda.synchronize()
        r = 0
        for s, n in zip(slots, lengths):
            cache_rows_parity(head_gpu, head_cpu, w, s, base[s], hidden[r:r + n], f"slot {s} rows {base[s]}..{base[s] + n}")
            r += n
            base[s] += n
            assert head_gpu.slot_lengths(s) == (base[s], 0)
    from paper_2505_24544_b200.binding import beagle_check_device
    beagle_check_device(head_gpu.ctx)
