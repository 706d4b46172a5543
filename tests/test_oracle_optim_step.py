"""Pins for the oracle's optimizers and the whole Algorithm-1 step: closed-form
scalar steps, torch.optim as a library routine, frozen-parameter identity,
exactly-once coverage, single group == full-parameter step.  No GPU."""
import math

import numpy as np
import pytest
import torch

import synth
from oracle import hift_oracle as O


# ---------------------------------------------------------------- P2: closed forms on one scalar
def test_adamw_closed_form_two_steps():
    th, g1, g2 = 0.7, -0.3, 0.05
    lr, b1, b2, eps, wd = 1e-2, 0.9, 0.999, 1e-8, 0.1
    t1, m1, v1 = O.adamw_update(np.array(th), np.array(g1), np.array(0.0), np.array(0.0), lr, b1, b2, eps, wd, 1)
    # step 1 from zero state: mhat = g, vhat = g^2  ->  theta(1-lr wd) - lr g/(|g|+eps)
    assert float(t1) == pytest.approx(th * (1 - lr * wd) - lr * g1 / (abs(g1) + eps), rel=1e-14)
    assert float(m1) == pytest.approx((1 - b1) * g1, rel=1e-15)
    assert float(v1) == pytest.approx((1 - b2) * g1 * g1, rel=1e-15)
    t2, m2, v2 = O.adamw_update(t1, np.array(g2), m1, v1, lr, b1, b2, eps, wd, 2)
    m2h = (b1 * (1 - b1) * g1 + (1 - b1) * g2) / (1 - b1 ** 2)
    v2h = (b2 * (1 - b2) * g1 ** 2 + (1 - b2) * g2 ** 2) / (1 - b2 ** 2)
    ref = float(t1) * (1 - lr * wd) - lr * m2h / (math.sqrt(v2h) + eps)
    assert float(t2) == pytest.approx(ref, rel=1e-14)


def test_adagrad_and_sgdm_closed_forms():
    th, g1, g2, lr = -1.5, 0.2, -0.4, 1e-2
    t1, a1 = O.adagrad_update(np.array(th), np.array(g1), np.array(0.0), lr, 1e-10)
    assert float(t1) == pytest.approx(th - lr * g1 / (abs(g1) + 1e-10), rel=1e-14)
    t2, a2 = O.adagrad_update(t1, np.array(g2), a1, lr, 1e-10)
    assert float(t2) == pytest.approx(float(t1) - lr * g2 / (math.sqrt(g1 * g1 + g2 * g2) + 1e-10), rel=1e-14)
    mu = 0.9
    s1, b1 = O.sgdm_update(np.array(th), np.array(g1), np.array(0.0), lr, mu)
    assert float(s1) == pytest.approx(th - lr * g1, rel=1e-15)
    s2, b2 = O.sgdm_update(s1, np.array(g2), b1, lr, mu)
    assert float(s2) == pytest.approx(th - lr * g1 - lr * (mu * g1 + g2), rel=1e-14)


def test_plain_sgd_closed_form_and_torch():
    th, g = np.array([0.5, -2.0]), np.array([0.25, 4.0])
    assert np.array_equal(O.sgd_update(th, g, 0.1), np.array([0.5 - 0.025, -2.0 - 0.4]))
    p = torch.nn.Parameter(torch.tensor(th))
    opt = torch.optim.SGD([p], lr=0.1)
    p.grad = torch.tensor(g)
    opt.step()
    assert np.allclose(O.sgd_update(th, g, 0.1), p.detach().numpy(), rtol=1e-15)


def test_adafactor_first_step_by_hand_and_against_torch():
    # 2 x 2 by hand at tau = 1: w = 1, so R, C are the row / column means of g^2
    th = np.array([[1.0, -2.0], [0.5, 4.0]])
    g = np.array([[0.1, -0.2], [0.3, 0.4]])
    R, Cc = (g * g).mean(1), (g * g).mean(0)
    V = np.outer(R, Cc) / R.mean()
    U = g / np.sqrt(V)
    U = U / max(1.0, math.sqrt((U * U).mean()))
    alpha = max(1e-3, math.sqrt((th * th).mean())) * min(1e-2, 1.0)
    got, s0, s1 = O.adafactor_update(th, g, np.zeros(2), np.zeros(2), 1e-2, 1e-30, 0.0, 1)
    assert np.allclose(got, th - alpha * U, rtol=1e-14) and np.allclose(s0, R) and np.allclose(s1, Cc)
    # several steps, a matrix and a vector, weight decay on, against the library routine
    rng = np.random.default_rng(8)
    for shape in ((7, 5), (11,)):
        p0 = rng.standard_normal(shape)
        grads = [rng.standard_normal(shape) * 1e-2 for _ in range(6)]
        p = torch.nn.Parameter(torch.tensor(p0))
        opt = torch.optim.Adafactor([p], lr=3e-3, eps=(1e-30, 1e-3), weight_decay=0.05, foreach=False)
        th = p0.copy()
        s0 = np.zeros(shape[0]) if len(shape) > 1 else np.zeros(shape)
        s1 = np.zeros(shape[1]) if len(shape) > 1 else np.zeros(0)
        for i, gr in enumerate(grads):
            p.grad = torch.tensor(gr)
            opt.step()
            th, s0, s1 = O.adafactor_update(th, gr, s0, s1, 3e-3, 1e-30, 0.05, i + 1)
            assert np.allclose(th, p.detach().numpy(), rtol=1e-11, atol=1e-14), (shape, i)


def test_optimizers_against_torch_optim_fp64():
    rng = np.random.default_rng(4)
    n, steps = 257, 5
    th0 = rng.standard_normal(n)
    grads = [rng.standard_normal(n) * 1e-2 for _ in range(steps)]

    def run_torch(make):
        p = torch.nn.Parameter(torch.tensor(th0))
        opt = make([p])
        for g in grads:
            p.grad = torch.tensor(g)
            opt.step()
        return p.detach().numpy()

    th, m, v = th0.copy(), np.zeros(n), np.zeros(n)
    for i, g in enumerate(grads):
        th, m, v = O.adamw_update(th, g, m, v, 3e-3, 0.9, 0.999, 1e-8, 0.05, i + 1)
    ref = run_torch(lambda ps: torch.optim.AdamW(ps, lr=3e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.05))
    assert np.allclose(th, ref, rtol=1e-12, atol=1e-14)

    th, acc = th0.copy(), np.zeros(n)
    for g in grads:
        th, acc = O.adagrad_update(th, g, acc, 1e-2, 1e-10)
    ref = run_torch(lambda ps: torch.optim.Adagrad(ps, lr=1e-2, eps=1e-10))
    assert np.allclose(th, ref, rtol=1e-12, atol=1e-14)

    th, buf = th0.copy(), np.zeros(n)
    for g in grads:
        th, buf = O.sgdm_update(th, g, buf, 1e-3, 0.9)
    ref = run_torch(lambda ps: torch.optim.SGD(ps, lr=1e-3, momentum=0.9))
    assert np.allclose(th, ref, rtol=1e-12, atol=1e-14)


# ---------------------------------------------------------------- P3: Eq. 2-3 invariants
def _cycle(cfg, gc, oc, steps, dist="uniform"):
    orc = O.HiFTOracle(cfg, gc, oc, synth.init_params(cfg, 1))
    losses, groups = [], []
    for t in range(steps):
        tok, lab = synth.batch_for(cfg, 5, t, dist)
        before = {k: v.copy() for k, v in orc.master.items()}
        s_before = {k: v.copy() for k, v in orc.s0.items()}
        g = orc.active_group()
        groups.append(g)
        losses.append(orc.step(tok, lab))
        names = set(orc.group_tensor_names(g))
        for k in orc.master:
            same = np.array_equal(orc.master[k], before[k])
            if k in names:
                assert not same, (t, k)                      # the active group moves
            else:
                assert same, (t, k)                          # everything else is bit-identical
                assert np.array_equal(orc.s0[k], s_before[k])
    return orc, losses, groups


def test_tiny_cycle_frozen_identity_and_exactly_once():
    cfg, gc, oc = synth.config_tiny_fp32()
    orc, losses, groups = _cycle(cfg, gc, oc, 6)
    assert groups == [0, 1, 2, 3, 4, 5]                     # bottom2up, one unit per group
    assert orc.tau == [1] * 6                                # one full cycle touches each group once
    covered = sorted(n for g in range(orc.k) for n in orc.group_tensor_names(g))
    assert covered == sorted(orc.master.keys())              # ... and every tensor belongs to exactly one group
    assert all(abs(l - math.log(512)) < 0.1 for l in losses)


def test_top2down_and_random_orders_drive_the_step():
    cfg, _, oc = synth.config_tiny_fp32()
    _, _, groups = _cycle(cfg, synth.GroupCfg(1, 0, synth.ORDER_TOP2DOWN), oc, 7)
    assert groups == [5, 4, 3, 2, 1, 0, 5]
    _, _, groups = _cycle(cfg, synth.GroupCfg(2, 1, synth.ORDER_RANDOM, 9), oc, 8)
    perm = O.group_order(4, 2, 9)
    assert groups == perm + perm


# ---------------------------------------------------------------- P4: one group == full step
@pytest.mark.parametrize("kind", [0, 1, 2])
def test_single_group_equals_full_parameter_step(kind):
    cfg, _, _ = synth.config_tiny_fp32()
    oc = synth.OptCfg(kind=kind, lr=1e-3, weight_decay=0.01, eps=1e-8, momentum=0.9)
    p0 = synth.init_params(cfg, 2, perturb=0.05)
    orc = O.HiFTOracle(cfg, synth.GroupCfg(layers_per_group=cfg.n_units), oc, p0)
    assert orc.k == 1
    tok, lab = synth.lm_batch(cfg, 3, 0, "uniform")
    loss = orc.step(tok, lab)
    # the standard step, spelled out without the scheduler
    P = {k: v.astype(np.float64) for k, v in p0.items()}
    loss_ref, cache = O.forward(cfg, P, tok, lab)
    G = O.backward(cfg, P, cache, None)
    assert loss == loss_ref
    for name in P:
        z = np.zeros_like(P[name])
        if kind == 0:
            ref = O.adamw_update(P[name], G[name], z, z, 1e-3, 0.9, 0.999, 1e-8, 0.01, 1)[0]
        elif kind == 1:
            ref = O.adagrad_update(P[name], G[name], z, 1e-3, 1e-8)[0]
        else:
            ref = O.sgdm_update(P[name], G[name], z, 1e-3, 0.9)[0]
        assert np.array_equal(orc.master[name], ref), name


def test_bias_correction_counts_group_updates_not_global_steps():
    cfg, gc, oc = synth.config_tiny_fp32()
    orc = O.HiFTOracle(cfg, gc, oc, synth.init_params(cfg, 1))
    for t in range(7):
        tok, lab = synth.lm_batch(cfg, 5, t, "uniform")
        orc.step(tok, lab)
    assert orc.tau == [2, 1, 1, 1, 1, 1]


def test_mixed_precision_model_reads_bf16_rounded_master():
    cfg = synth.ModelCfg(arch=2, n_blocks=1, d_model=16, n_heads=2, d_ffn=32, vocab=29,
                         dtype=synth.DTYPE_BF16, batch=1, seq=4, norm_eps=1e-6)
    orc = O.HiFTOracle(cfg, synth.GroupCfg(), synth.OptCfg(), synth.init_params(cfg, 0))
    P = orc.model_params()
    for k, v in P.items():
        assert np.array_equal(v, O.bf16_round(orc.master[k].astype(np.float32)).astype(np.float64))
