"""The pins do catch mistakes: each case plants one plausible error in the CPU oracle (a dropped term,
a wrong sign or index, a transposed operand) and checks that a named pin of tests/test_oracle_pins.py
fails on it.  Everything here runs on the CPU and touches only the oracle."""
import numpy as np
import pytest

import oracle.beagle_oracle as M
import test_oracle_pins as P

F64 = np.float64


def _rms_norm_no_eps_mean_over_sum(v, g, eps):
    v = np.asarray(v, dtype=F64)
    return g * (v / np.sqrt(np.sum(v * v, axis=-1, keepdims=True) + eps))          # sum instead of mean


def _silu_wrong_sign(u):
    u = np.asarray(u, dtype=F64)
    return u / (1.0 + np.exp(u))


def _visible_includes_diagonal(p, block, offset):
    if p <= offset:
        return p                                                                   # key p visible to query p
    return offset + block * ((p - 1 - offset) // block)


def _visible_window_off_by_one(p, block, offset):
    if p <= offset:
        return p - 1
    return offset + block * ((p - offset) // block)                                # window boundary shifted by one


def _weights_unscaled(head, q, k_vis):
    c = head.cfg
    nv = k_vis.shape[0]
    w = np.zeros((c.n_q_heads, nv), dtype=F64)
    for h in range(c.n_q_heads):
        if nv:
            a = k_vis[:, h // c.group, :] @ q[h]                                   # no 1 / sqrt(d_h)
            e = np.exp(a - np.max(a))
            w[h] = e / np.sum(e)
    return w


def _weights_wrong_group(head, q, k_vis):
    c = head.cfg
    nv = k_vis.shape[0]
    w = np.zeros((c.n_q_heads, nv), dtype=F64)
    for h in range(c.n_q_heads):
        if nv:
            a = (k_vis[:, h % c.n_kv_heads, :] @ q[h]) / np.sqrt(F64(c.head_dim))  # interleaved instead of blocked groups
            e = np.exp(a - np.max(a))
            w[h] = e / np.sum(e)
    return w


def _argmax_highest_on_ties(z):
    z = np.asarray(z, dtype=F64)
    z = np.where(np.isnan(z), -np.inf, z)
    return (z.shape[-1] - 1 - np.argmax(z[..., ::-1], axis=-1)).astype(np.int64)


def _output_projection_without_residual(head, o, x):
    return o @ head.w_o.T


def _down_projection_transposed_residual(head, act, y):
    return np.asarray(act, dtype=F64) @ head.w_down.T - y                           # wrong sign of the residual


def _loss_weights_k_minus_i(S, block, offset, sim_steps, stage):
    w, n = _orig_loss_weights(S, block, offset, sim_steps, stage)
    return (np.where(w > 0, w - 1, w) if stage == "late" else w), n                # beta = k - i instead of k - i + 1


_orig_loss_weights = M.loss_weights


def _rms_backward_without_projection(v, g, eps, dn):
    v = np.asarray(v, dtype=F64)
    r = 1.0 / np.sqrt(np.mean(v * v, axis=-1, keepdims=True) + eps)
    return r * (g * dn), np.sum(dn * v * r, axis=0)                                 # the second term of dv dropped


def _smooth_l1_threshold_half(r):
    r = np.asarray(r, dtype=F64)
    a = np.abs(r)
    return np.where(a < 0.5, r * r, a - 0.25)


def _rope_wrong_pairing(x, pos, theta, inverse=False):
    x = np.asarray(x, dtype=F64)                                                    # pairs (2i, 2i+1) instead of (i, i + d_h/2)
    half = x.shape[-1] // 2
    freq = F64(theta) ** (-2.0 * np.arange(half, dtype=F64) / x.shape[-1])
    ang = np.asarray(pos, dtype=F64)[:, None] * freq[None, :] * (-1.0 if inverse else 1.0)
    cs, sn = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    out = np.empty_like(x)
    out[..., 0::2] = x[..., 0::2] * cs - x[..., 1::2] * sn
    out[..., 1::2] = x[..., 1::2] * cs + x[..., 0::2] * sn
    return out


def _residual_without_clamp(p, q):
    p = np.asarray(p, dtype=F64)
    if q is None:
        return p / np.sum(p)
    d = p - np.asarray(q, dtype=F64)                                                # max(0, .) dropped
    return d / np.sum(d) if np.sum(d) != 0 else p / np.sum(p)


def _softmax_unshifted_base2(logits, temperature=1.0):
    z = np.asarray(logits, dtype=F64) / temperature
    e = np.exp2(z - np.max(z, axis=-1, keepdims=True))                              # base 2 instead of e
    return e / np.sum(e, axis=-1, keepdims=True)


CASES = [
    ("rms_norm", _rms_norm_no_eps_mean_over_sum, P.test_norm_flags_and_rmsnorm_definition, ()),
    ("silu", _silu_wrong_sign, P.test_silu_values, ()),
    ("visible_true_count", _visible_includes_diagonal, P.test_mask_brute_force, ()),
    ("visible_true_count", _visible_window_off_by_one, P.test_mask_brute_force, ()),
    ("attention_weights", _weights_unscaled, P.test_hand_worked_draft_step_matches_golden, ()),
    ("attention_weights", _weights_wrong_group, P.test_gqa_equals_mha_with_repeated_kv_heads, ()),
    ("argmax_lowest", _argmax_highest_on_ties, P.test_argmax_ties_and_nan, ()),
    ("output_projection", _output_projection_without_residual, P.test_no_visible_key_gives_embedding_path_only, ()),
    ("down_projection", _down_projection_transposed_residual, P.test_zero_output_projections_reduce_to_embedding_times_lm_head, ()),
    ("loss_weights", _loss_weights_k_minus_i, P.test_loss_weights_follow_eq4_and_eq7, ()),
    ("rms_norm_backward", _rms_backward_without_projection, P.test_early_stage_gradient_is_the_derivative_of_block_loss, (3, 0, False, True, 0.0)),
    ("rms_norm_backward", _rms_backward_without_projection, P.test_training_gradients_against_torch_autograd, ("early", 3, 1, 1, 10.0, 0.0)),
    ("smooth_l1", _smooth_l1_threshold_half, P.test_smooth_l1_and_rmsnorm_backward_by_differences, ()),
    ("rope_rotate", _rope_wrong_pairing, P.test_rope_rotation_by_hand_and_orthogonality, ()),
    ("residual_distribution", _residual_without_clamp, P.test_verify_sample_first_token_follows_the_target_distribution, ()),
    ("softmax_rows", _softmax_unshifted_base2, P.test_cross_entropy_closed_forms, ()),
]


@pytest.mark.parametrize("name,mutant,pin,args", CASES, ids=[f"{c[0]}-{c[1].__name__.lstrip('_')}" for c in CASES])
def test_a_planted_mistake_fails_its_pin(monkeypatch, name, mutant, pin, args):
    pin(*args)                                                     # green on the oracle as it stands
    monkeypatch.setattr(M, name, mutant)
    import oracle as O
    if hasattr(O, name):
        monkeypatch.setattr(O, name, mutant)
    with pytest.raises(AssertionError):
        pin(*args)
