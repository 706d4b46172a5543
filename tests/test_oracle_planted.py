"""The pins must be able to fail: plant plausible mistakes in the oracle (on the CPU) and check
that the finite-difference / closed-form / library pins catch each of them."""
import numpy as np
import pytest

import synth
from oracle import hift_oracle as O
from test_oracle_math import _fd_check, mini


def _expect_caught(fn):
    with pytest.raises(AssertionError):
        fn()


def test_wrong_sign_in_rope_backward_is_caught(monkeypatch):
    orig = O.rope_apply
    monkeypatch.setattr(O, "rope_apply", lambda x, c, s, inverse=False: orig(x, c, s, inverse=False))
    _expect_caught(lambda: _fd_check(mini(2), n_samples=3))


def test_dropped_term_in_gelu_derivative_is_caught(monkeypatch):
    import math
    from scipy.special import erf
    monkeypatch.setattr(O, "gelu_bwd", lambda d, a: d * 0.5 * (1.0 + erf(a / math.sqrt(2.0))))   # a*pdf term dropped
    _expect_caught(lambda: _fd_check(mini(0), n_samples=3))


def test_missing_attention_scale_in_dk_is_caught(monkeypatch):
    orig = O.attention_bwd

    def bad(do, q, k, v, p, pmask=None):
        dq, dk, dv = orig(do, q, k, v, p, pmask)
        return dq, dk * np.sqrt(q.shape[-1]), dv
    monkeypatch.setattr(O, "attention_bwd", bad)
    _expect_caught(lambda: _fd_check(mini(1), n_samples=3))


def test_attention_probability_mask_left_out_of_a_gradient_is_caught(monkeypatch):
    from test_oracle_math import test_attention_probability_dropout_by_loops_and_its_element_numbering as pin_loops
    orig = O.attention_bwd
    # the mask forgotten on the way back to the softmax (dv still right)
    def no_mask_on_dp(do, q, k, v, p, pmask=None):
        dq, dk, _ = orig(do, q, k, v, p, None)
        _, _, dv = orig(do, q, k, v, p, pmask)
        return dq, dk, dv
    monkeypatch.setattr(O, "attention_bwd", no_mask_on_dp)
    _expect_caught(pin_loops)
    _expect_caught(lambda: _fd_check(mini(0), n_samples=3, drop=(0.0, 78, 1, 0.25)))
    # the mask applied before the normalisation instead of after it
    monkeypatch.setattr(O, "attention_bwd", orig)
    fwd = O.attention_fwd

    def renormalised(q, k, v, causal, lens=None, pmask=None):
        o, p = fwd(q, k, v, causal, lens, pmask)
        if pmask is not None:
            pd = p * pmask
            pd = pd / np.maximum(pd.sum(-1, keepdims=True), 1e-30)
            o = np.matmul(pd, v.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3)
        return o, p
    monkeypatch.setattr(O, "attention_fwd", renormalised)
    _expect_caught(pin_loops)


def test_key_padding_off_by_one_or_on_the_wrong_axis_is_caught(monkeypatch):
    from test_oracle_math import test_key_padding_equals_attention_on_the_unpadded_rows as pin_rows
    from test_oracle_math import test_padded_batch_equals_the_sequences_run_alone as pin_batch
    orig = O.attention_fwd
    # the key at position len still visible
    monkeypatch.setattr(O, "attention_fwd", lambda q, k, v, causal, lens=None, pmask=None:
                        orig(q, k, v, causal, None if lens is None else [min(int(l) + 1, q.shape[1]) for l in lens], pmask))
    _expect_caught(pin_rows)
    _expect_caught(pin_batch)

    # the table applied to queries instead of keys: padded query rows zeroed, padded keys still seen
    def on_queries(q, k, v, causal, lens=None, pmask=None):
        o, p = orig(q, k, v, causal, None, pmask)
        if lens is not None:
            o = o.copy()
            for b, l in enumerate(lens):
                o[b, int(l):] = 0.0
        return o, p
    monkeypatch.setattr(O, "attention_fwd", on_queries)
    _expect_caught(pin_rows)
    _expect_caught(pin_batch)


def test_layernorm_backward_without_mean_subtraction_is_caught(monkeypatch):
    def bad(dy, cache, g):
        xhat, rstd = cache
        dg = (dy * xhat).reshape(-1, xhat.shape[-1]).sum(axis=0)
        db = dy.reshape(-1, xhat.shape[-1]).sum(axis=0)
        dxh = dy * g
        return rstd * (dxh - xhat * (dxh * xhat).mean(axis=-1, keepdims=True)), dg, db
    monkeypatch.setattr(O, "layernorm_bwd", bad)
    _expect_caught(lambda: _fd_check(mini(0), n_samples=3))


def test_transposed_weight_gradient_is_caught():
    # a transposed dW has the wrong shape unless the layer is square: w_o is square, so plant it there
    cfg = mini(0)
    P = {k: v.astype(np.float64) for k, v in synth.init_params(cfg, 3, perturb=0.1).items()}
    tok, lab = synth.batch_for(cfg, 11, 0, dist="uniform")
    loss, cache = O.forward(cfg, P, tok, lab)
    G = O.backward(cfg, P, cache, None)
    h = 1e-5
    name, i, j = "b0.w_o", 3, 7
    P[name][i, j] += h
    lp, _ = O.forward(cfg, P, tok, lab)
    P[name][i, j] -= 2 * h
    lm, _ = O.forward(cfg, P, tok, lab)
    fd = (lp - lm) / (2 * h)
    assert abs(fd - G[name][i, j]) < 1e-6 * np.abs(G[name]).max()
    assert abs(fd - G[name].T[i, j]) > 1e-3 * np.abs(G[name]).max()       # the transposed entry would not pass


def test_bias_correction_with_global_step_is_caught():
    # Adam with the global step count instead of the group's update count gives a different update
    th, g = np.array([0.3]), np.array([0.02])
    a, _, _ = O.adamw_update(th, g, np.zeros(1), np.zeros(1), 1e-3, 0.9, 0.999, 1e-8, 0.0, 1)
    b, _, _ = O.adamw_update(th, g, np.zeros(1), np.zeros(1), 1e-3, 0.9, 0.999, 1e-8, 0.0, 7)
    assert abs(a[0] - (0.3 - 1e-3 * 0.02 / (0.02 + 1e-8))) < 1e-15
    assert abs(a[0] - b[0]) > 1e-5


def test_eps_inside_the_square_root_is_caught():
    th, g, eps = 0.5, 1e-6, 1e-8
    t1, _, _ = O.adamw_update(np.array(th), np.array(g), np.array(0.0), np.array(0.0), 1e-2, 0.9, 0.999, eps, 0.0, 1)
    outside = th - 1e-2 * g / (abs(g) + eps)
    inside = th - 1e-2 * g / np.sqrt(g * g + eps)
    assert abs(float(t1) - outside) < 1e-15 and abs(float(t1) - inside) > 1e-4
