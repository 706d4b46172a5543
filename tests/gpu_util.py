"""Helpers shared by the GPU parity tests (not a test module)."""
import numpy as np


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64).reshape(-1)
    b = np.asarray(b, dtype=np.float64).reshape(-1)
    den = np.linalg.norm(b)
    if den == 0.0:
        return float(np.linalg.norm(a))
    return float(np.linalg.norm(a - b) / den)


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
