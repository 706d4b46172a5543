"""Helpers shared by the GPU parity tests (not a test module)."""
import numpy as np


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64).reshape(-1)
    b = np.asarray(b, dtype=np.float64).reshape(-1)
    den = np.linalg.norm(b)
    if den == 0.0:
        return float(np.linalg.norm(a))
    return float(np.linalg.norm(a - b) / den)


# ---------------------------------------------------------------- element-wise bounds
# Every kernel output is also held to a bound per element, |got - ref| <= rel * |ref| + slack, so that a
# single wrong element (an edge tile, a ragged row) fails where a whole-tensor norm would hide it.
#   rel:   the rounding of the store, U_BF16 = 2^-8 for a bf16 output (8-bit significand, round to
#          nearest: half a unit in the last place is at most 2^-8 of the value), U_F32 = 2^-24 for fp32.
#   slack: what the arithmetic before the store can be off by, in absolute terms, computed by the test
#          from the oracle's own values.  For a dot product of depth K accumulated in fp32 in ANY order
#          the classical bound is gamma_K * sum_k |a_k b_k|; tensor cores align the addends of a step and
#          may drop up to a unit in the last place of the running sum (unit 2^-23 instead of 2^-24), so
#          gemm_slack uses (K + 16) * 2^-23 * (|A| |B|).
U_BF16 = 2.0 ** -8
U_F32 = 2.0 ** -24


def gemm_slack(A, B):
    """Accumulation-error allowance of A @ B (A [m, K], B [K, n], the fp64 images of the operands)."""
    K = A.shape[-1]
    return (K + 16) * 2.0 ** -23 * (np.abs(A) @ np.abs(B))


def assert_elem(got, ref, rel, slack=0.0, what=""):
    """|got - ref| <= rel * |ref| + slack for every element (slack: scalar or array of ref's shape)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    tol = 1.01 * (rel * np.abs(ref) + slack) + 1e-300
    err = np.abs(got - ref)
    bad = ~(err <= tol)                       # NaN fails
    if bad.any():
        i = np.unravel_index(np.argmax(np.where(bad, err / tol, 0.0)), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())} of {bad.size} elements out of bound; worst at {i}: "
                             f"got {got[i]!r}, ref {ref[i]!r}, err {err[i]:.3e}, allowed {np.broadcast_to(tol, err.shape)[i]:.3e}")


def tile_rows(M, tile=128, seed=0):
    """Rows to sample from an output of M rows: one (seeded) in every `tile`-row tile, plus the first
    row, both sides of the first tile boundary and the last row."""
    rng = np.random.default_rng(seed + M)
    rows = {0, M - 1}
    for t0 in range(0, M, tile):
        rows.add(int(t0 + rng.integers(0, min(tile, M - t0))))
    for r in (tile - 1, tile):
        if r < M:
            rows.add(r)
    return np.array(sorted(rows), dtype=np.int64)


def attention_slack(q, k, v, p, do=None, u=U_BF16):
    """Allowances for softmax attention computed with bf16 probabilities (and, backward, bf16 dS), from the
    oracle's probabilities p [B,H,S,S] and the fp64 operands q, k, v (and do) [B,S,H,dh].
    Forward: P is rounded to bf16 before P V (2^-8 each), and a score error ds moves every probability by
    a factor e^ds; scores are fp32 dot products of depth dh.  Backward: P and dS are rounded to bf16, and
    the row term D = rowsum(dO o O) is formed from the bf16-rounded O the forward pass stored.
    u: rounding unit of the stored probabilities and dS (U_BF16 for the bf16 kernels, a few fp32 units for the fp32 ones).
    Returns (slack_o) or (slack_o, slack_dq, slack_dk, slack_dv), each [B,S,H,dh]."""
    B, S, H, dh = q.shape
    qh, kh, vh = (np.abs(t).transpose(0, 2, 1, 3) for t in (q, k, v))
    scale = 1.0 / np.sqrt(dh)
    ds_max = (dh + 16) * 2.0 ** -23 * np.matmul(qh, kh.transpose(0, 1, 3, 2)).max() * scale + 4e-7   # + exp2 approximation
    pe = u + 2.0 * ds_max
    s_o = (pe * np.matmul(p, vh)).transpose(0, 2, 1, 3)
    if do is None:
        return s_o
    doh = do.transpose(0, 2, 1, 3)
    vs = v.transpose(0, 2, 1, 3)
    dp = np.matmul(doh, vs.transpose(0, 1, 3, 2))
    D = (dp * p).sum(-1, keepdims=True)
    o = np.matmul(p, vs)
    dD = u * (np.abs(doh) * np.abs(o)).sum(-1, keepdims=True) + (dh + 16) * 2.0 ** -23 * (np.abs(doh) * np.abs(o)).sum(-1, keepdims=True)
    ddp = (dh + 16) * 2.0 ** -23 * np.matmul(np.abs(doh), vh.transpose(0, 1, 3, 2))
    e = (2 * pe + u) * p * np.abs(dp - D) + p * (dD + ddp)              # |error of dS|
    s_dq = scale * np.matmul(e, kh).transpose(0, 2, 1, 3)
    s_dk = scale * np.matmul(e.transpose(0, 1, 3, 2), qh).transpose(0, 2, 1, 3)
    s_dv = (pe * np.matmul(p.transpose(0, 1, 3, 2), np.abs(doh))).transpose(0, 2, 1, 3)
    return s_o, s_dq, s_dk, s_dv


def make_pair(cfg, gcfg, ocfg, seed=1, perturb=0.05):
    """A CUDA context and an oracle holding the same initial parameters."""
    import synth
    from oracle import hift_oracle as O
    from paper_2401_15207_b200 import HiFT
    p0 = synth.init_params(cfg, seed, perturb=perturb)
    h = HiFT(cfg, gcfg, ocfg)
    h.set_params(p0)
    orc = O.HiFTOracle(cfg, gcfg, ocfg, p0)
    return h, orc, p0


def _read_state(h, kind, n):
    if kind == 4:
        rows = h.tensor_info(n)[1][0]
        return [h.get_factored_state(n, 0)] + ([h.get_factored_state(n, 1)] if rows > 1 else [np.zeros(0, np.float32)])
    return [h.get_state(n, w) for w in range({0: 2, 1: 1, 2: 1}.get(kind, 0))]


def check_update_given_gradient(h, orc, ocfg, n, g, lr, master0, state0, tol=1e-6):
    """'Optimizer updates given identical gradients agree within 1e-6 relative': relative L2 of each
    post-update tensor (fp32 master, optimizer state); the update itself to 1e-4 plus the rounding of the
    fp32 value it is stored in."""
    from oracle import hift_oracle as O
    shape = orc.master[n].shape
    grad = h.get_grad(n).astype(np.float64).reshape(shape)
    m0 = master0.astype(np.float64).reshape(shape)
    tau = orc.tau_of(n, g)
    k = ocfg.kind
    if k == 0:
        ref = O.adamw_update(m0, grad, state0[0].astype(np.float64).reshape(shape), state0[1].astype(np.float64).reshape(shape),
                             lr, ocfg.beta1, ocfg.beta2, ocfg.eps, ocfg.weight_decay, tau)
    elif k == 1:
        ref = O.adagrad_update(m0, grad, state0[0].astype(np.float64).reshape(shape), lr, ocfg.eps)
    elif k == 2:
        ref = O.sgdm_update(m0, grad, state0[0].astype(np.float64).reshape(shape), lr, ocfg.momentum)
    elif k == 3:
        ref = (O.sgd_update(m0, grad, lr),)
    else:
        s0 = state0[0].astype(np.float64)
        s1 = state0[1].astype(np.float64)
        ref = O.adafactor_update(m0, grad, s0, s1, lr, ocfg.eps, ocfg.weight_decay, tau)
    after = h.get_param(n).astype(np.float64).reshape(shape)
    assert rel_l2(after, ref[0]) <= tol, (n, "master", rel_l2(after, ref[0]))
    d_ref = ref[0] - m0
    assert np.linalg.norm((after - m0) - d_ref) <= 1e-4 * np.linalg.norm(d_ref) + 2 * 6e-8 * np.linalg.norm(m0) + 1e-30, (n, "update")
    got_state = _read_state(h, k, n)
    for w, st in enumerate(got_state):
        if st.size:
            e = rel_l2(st.reshape(-1), np.asarray(ref[1 + w]).reshape(-1))
            assert e <= (2e-6 if k == 4 else tol), (n, "state", w, e)
    # the model copy the next forward pass reads: the round-to-nearest-even bf16 image of the new master
    if h.model.dtype == 1:
        assert np.array_equal(h.get_model_param(n).reshape(-1), O.bf16_round(h.get_param(n)).reshape(-1)), (n, "bf16 copy")


def lockstep(cfg, gcfg, ocfg, steps, dist, tol_loss, tol_grad, seed=1, data_seed=5, perturb=0.05,
             check_update=None, resync=False, lens=None):
    """Run `steps` iterations on both sides with the same batches and compare
    group choice (exact), learning rate (exact), loss, every gradient tensor of
    the active group, and frozen parameters (bit-exact).

    resync=True copies the library's updated fp32 master values into the oracle
    after every step, so that each step is compared from identical parameters
    (the tolerances are per step; without it the two parameter trajectories
    drift apart by the accumulated rounding of earlier updates).

    lens: optional function step -> list of real-token counts per batch entry
    (right-padded batches): both sides get the table, padded positions of a
    language-model batch carry label -1."""
    import torch
    import synth
    h, orc, p0 = make_pair(cfg, gcfg, ocfg, seed, perturb)
    assert h.num_groups() == orc.k
    names = h.tensor_names()
    assert sorted(names) == sorted(p0.keys())
    report = []
    try:
        for t in range(steps):
            tok, lab = synth.batch_for(cfg, data_seed, t, dist)
            kl = None
            if lens is not None:
                kl = [int(v) for v in lens(t)]
                h.set_key_lengths(kl)
                if lab.ndim == 2:
                    lab = lab.copy()
                    for b, l in enumerate(kl):
                        lab[b, l:] = -1
            g = h.active_group()
            assert g == orc.active_group(), (t, g, orc.active_group())
            assert h.current_lr() == orc.current_lr()
            active = set(orc.group_tensor_names(g))
            before = {n: h.get_param(n) for n in names}
            lr = orc.current_lr()
            state_before = {n: _read_state(h, ocfg.kind, n) for n in active}
            loss = h.step(torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda())
            loss_ref = orc.step(tok, lab, kl)
            assert abs(loss - loss_ref) <= tol_loss * abs(loss_ref), (t, loss, loss_ref)
            worst = 0.0
            for n in sorted(active):
                gg = h.get_grad(n).reshape(orc.last_grads[n].shape)
                gr = orc.last_grads[n]
                e = rel_l2(gg, gr)
                worst = max(worst, e)
                assert e <= tol_grad, (t, g, n, e)
            for n in sorted(active):
                # the update inside the step, given identical gradients: the library's own fp32 gradient and the
                # master / state it held before the step go through the oracle's optimizer with the oracle's
                # learning rate and update count; post-update master and state agree to 1e-6 relative
                check_update_given_gradient(h, orc, ocfg, n, g, lr, before[n], state_before[n])
            for n in names:
                after = h.get_param(n)
                if n in active:
                    assert not np.array_equal(after, before[n]), (t, n)
                    if check_update is not None:
                        # Elements whose gradient is numerically zero (e.g. the key bias, to which
                        # softmax is invariant) take a sign-of-noise Adam step: leave them out.
                        gr = np.abs(orc.last_grads[n].reshape(after.shape))
                        mask = gr > 1e-4 * gr.max()
                        upd = (orc.master[n].reshape(after.shape) - before[n].astype(np.float64))[mask]
                        err = (after.astype(np.float64) - orc.master[n].reshape(after.shape))[mask]
                        # plus half an ulp of the fp32 value the update is stored in
                        ulp = 6e-8 * np.linalg.norm(after[mask])
                        assert np.linalg.norm(err) <= check_update * np.linalg.norm(upd) + ulp + 1e-12, (t, n)
                    if resync:
                        orc.master[n] = after.astype(np.float64).reshape(orc.master[n].shape)
                        if ocfg.kind == 4:
                            orc.s0[n] = h.get_factored_state(n, 0).astype(np.float64)
                            if orc.master[n].ndim > 1:
                                orc.s1[n] = h.get_factored_state(n, 1).astype(np.float64)
                        elif ocfg.kind != 3:
                            orc.s0[n] = h.get_state(n, 0).astype(np.float64).reshape(orc.master[n].shape)
                        if ocfg.kind == 0:
                            orc.s1[n] = h.get_state(n, 1).astype(np.float64).reshape(orc.master[n].shape)
                else:
                    assert np.array_equal(after, before[n]), (t, n)       # Eq. 2-3: frozen bits untouched
            report.append((t, g, loss, loss_ref, worst))
        assert h.step_count() == orc.t
    finally:
        h.close()
    return report
