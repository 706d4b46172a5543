"""The two-halves form of the step (hift_step_begin / hift_grad_view / hift_step_end) and the
data-parallel arithmetic it exists for, emulated on ONE GPU: the "ranks" are contexts that run one
after another, never kernels that wait on each other."""
import numpy as np
import pytest

import synth
from gpu_util import rel_l2

pytestmark = pytest.mark.gpu


def _cfg(batch):
    return synth.ModelCfg(arch=2, n_blocks=2, d_model=256, n_heads=2, d_ffn=512, vocab=1000, norm_eps=1e-6,
                          dtype=synth.DTYPE_BF16, batch=batch, seq=128, init_std=0.05)


def test_split_step_is_bitwise_the_fused_step():
    import torch
    from paper_2401_15207_b200 import HiFT, HiftError
    cfg = _cfg(2)
    gc, oc = synth.GroupCfg(1), synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=1)
    p0 = synth.init_params(cfg, 2)
    a, b = HiFT(cfg, gc, oc), HiFT(cfg, gc, oc)
    a.set_params(p0)
    b.set_params(p0)
    for t in range(5):
        tok, lab = synth.lm_batch(cfg, 4, t)
        tt, ll = torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()
        la = a.step(tt, ll)
        lb = b.step_begin(tt, ll)
        with pytest.raises(HiftError):
            b.step(tt, ll)                                   # begin/end must alternate
        b.step_end()
        assert la == lb
    with pytest.raises(HiftError):
        b.step_end()
    for n in a.tensor_names():
        assert np.array_equal(a.get_param(n), b.get_param(n)), n
    a.close()
    b.close()


def test_two_emulated_ranks_average_gradients_and_stay_in_sync():
    import torch
    from paper_2401_15207_b200 import HiFT
    full, half = _cfg(4), _cfg(2)
    gc, oc = synth.GroupCfg(1), synth.OptCfg(kind=2, lr=1e-2, momentum=0.9, offload_state=1)
    p0 = synth.init_params(full, 5)
    ref, r0, r1 = HiFT(full, gc, oc), HiFT(half, gc, oc), HiFT(half, gc, oc)
    for h in (ref, r0, r1):
        h.set_params(p0)
    for t in range(4):
        tok, lab = synth.lm_batch(full, 8, t)
        g = ref.active_group()
        l_ref = ref.step(torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda())
        l0 = r0.step_begin(torch.from_numpy(tok[:2].copy()).cuda(), torch.from_numpy(lab[:2].copy()).cuda())
        l1 = r1.step_begin(torch.from_numpy(tok[2:].copy()).cuda(), torch.from_numpy(lab[2:].copy()).cuda())
        g0, g1 = r0.grad_view(), r1.grad_view()
        assert g0.numel() == g1.numel() and g0.dtype == torch.float32
        avg = (g0 + g1) * 0.5                                # what an all-reduce + 1/world would leave on both
        g0.copy_(avg)
        g1.copy_(avg)
        torch.cuda.synchronize()
        r0.step_end()
        r1.step_end()
        assert abs(0.5 * (l0 + l1) - l_ref) <= 2e-3 * abs(l_ref)
        lo, hi = ref.group_units(g)
        for n in ref.tensor_names():
            a0, a1 = r0.get_param(n), r1.get_param(n)
            assert np.array_equal(a0, a1), (t, n)            # replicas hold the same bits after every step
            if lo <= ref.tensor_info(n)[0] <= hi:
                # equal shards: the mean of the shard gradients is the full-batch gradient
                assert rel_l2(r0.get_grad(n), ref.get_grad(n)) <= 2e-2, (t, n)
                assert rel_l2(a0, ref.get_param(n)) <= 1e-4, (t, n)
    for h in (ref, r0, r1):
        h.close()
