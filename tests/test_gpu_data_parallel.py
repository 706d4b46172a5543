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


def test_overlapped_exchange_chunks_tile_the_gradient_and_change_no_bits():
    """The asynchronous first half + chunk list + hift_step_finish (what dist_util.data_parallel_step drives)
    on one rank: the chunks come in the order the backward pass finishes them (from the top of the span
    down), tile the flat gradient exactly once, respect the minimum size except for the last, and the step
    leaves the same bits as hift_step."""
    import torch
    from paper_2401_15207_b200 import HiFT, dist_util
    cfg = _cfg(2)
    gc, oc = synth.GroupCfg(layers_per_group=2), synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=2)
    p0 = synth.init_params(cfg, 2)
    a, b = HiFT(cfg, gc, oc), HiFT(cfg, gc, oc)
    a.set_params(p0)
    b.set_params(p0)
    b.set_grad_chunk_bytes(256 << 10)
    seen = []
    for t in range(2 * a.num_groups()):
        tok, lab = synth.lm_batch(cfg, 4, t)
        tt, ll = torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()
        la = a.step(tt, ll)
        if t % 2 == 0:
            lb = dist_util.data_parallel_step(b, tt, ll)          # no process group: a world of one
        else:
            b.step_begin_async(tt, ll)
            chunks = b.grad_chunks()
            n = b.grad_view().numel()
            assert sum(c[1] for c in chunks) == n
            ends = [c[0] + c[1] for c in chunks]
            assert ends[0] == n and chunks[-1][0] == 0
            assert all(chunks[i + 1][0] + chunks[i + 1][1] == chunks[i][0] for i in range(len(chunks) - 1))   # descending, gap-free
            assert all(c[1] >= (256 << 10) // 4 for c in chunks[:-1])
            seen.append(len(chunks))
            for i in range(len(chunks)):
                b.grad_chunk_wait(i, torch.cuda.current_stream().cuda_stream)
            assert int(b.gate_view().item()) == 0
            lb = b.step_finish()
        assert la == lb
    assert max(seen) > 3                                          # the block groups really were cut into several chunks
    for n in a.tensor_names():
        assert np.array_equal(a.get_param(n), b.get_param(n)), n
    a.close()
    b.close()


def test_two_emulated_ranks_exchange_chunk_by_chunk_and_share_the_gate():
    """Two contexts as two ranks (run one after the other on one GPU): gradients averaged chunk by chunk in
    the order the chunks complete keep the replicas bit-identical; and when one rank's step fails (a NaN
    planted in one of its frozen parameters), the MAX of the gate words calls the update off on both, both
    report the failure, and neither changes a bit."""
    import torch
    from paper_2401_15207_b200 import HiFT, HiftError
    half = _cfg(2)
    gc, oc = synth.GroupCfg(1), synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=1)
    p0 = synth.init_params(half, 5)
    r0, r1 = HiFT(half, gc, oc), HiFT(half, gc, oc)
    for h in (r0, r1):
        h.set_params(p0)
        h.set_grad_chunk_bytes(128 << 10)
    full = _cfg(4)
    st = torch.cuda.current_stream().cuda_stream

    def exchange(poison=False):
        g0, g1 = r0.grad_view(), r1.grad_view()
        c0, c1 = r0.grad_chunks(), r1.grad_chunks()
        assert c0 == c1                                            # same schedule on every rank, nothing to agree on
        for i, (off, n) in enumerate(c0):
            r0.grad_chunk_wait(i, st)
            r1.grad_chunk_wait(i, st)
            avg = (g0[off:off + n] + g1[off:off + n]) * 0.5
            g0[off:off + n].copy_(avg)
            g1[off:off + n].copy_(avg)
        f0, f1 = r0.gate_view(), r1.gate_view()
        m = torch.maximum(f0, f1)
        f0.copy_(m)
        f1.copy_(m)
        return int(m.item())

    for t in range(3):
        tok, lab = synth.lm_batch(full, 8, t)
        r0.step_begin_async(torch.from_numpy(tok[:2].copy()).cuda(), torch.from_numpy(lab[:2].copy()).cuda())
        r1.step_begin_async(torch.from_numpy(tok[2:].copy()).cuda(), torch.from_numpy(lab[2:].copy()).cuda())
        assert exchange() == 0
        r0.step_finish()
        r1.step_finish()
        for n in r0.tensor_names():
            assert np.array_equal(r0.get_param(n), r1.get_param(n)), (t, n)
    # a failing rank
    g = r1.active_group()
    lo, hi = r1.group_units(g)
    victim = [n for n in r1.tensor_names() if not (lo <= r1.tensor_info(n)[0] <= hi) and n.endswith("w_o")][0]
    good = r1.get_param(victim)
    bad = good.copy()
    bad[0, 0] = np.nan
    r1.set_param(victim, bad)
    before0 = {n: r0.get_param(n) for n in r0.tensor_names()}
    tok, lab = synth.lm_batch(full, 8, 7)
    r0.step_begin_async(torch.from_numpy(tok[:2].copy()).cuda(), torch.from_numpy(lab[:2].copy()).cuda())
    r1.step_begin_async(torch.from_numpy(tok[2:].copy()).cuda(), torch.from_numpy(lab[2:].copy()).cuda())
    assert exchange() == 101                                       # non-finite loss on rank 1, now known to both
    for h in (r0, r1):
        with pytest.raises(HiftError) as e:
            h.step_finish()
        assert e.value.status == 5
        assert h.step_count() == 3
    for n in r0.tensor_names():
        assert np.array_equal(r0.get_param(n), before0[n]), n      # rank 0 averaged a NaN gradient in, and still changed nothing
    r1.set_param(victim, good)
    for n in r0.tensor_names():
        assert np.array_equal(r0.get_param(n), r1.get_param(n)), n
    r0.close()
    r1.close()


@pytest.mark.parametrize("kind,dtype,offload", [(0, synth.DTYPE_BF16, 1), (0, synth.DTYPE_BF16, 0), (2, synth.DTYPE_FP32, 1)])
def test_sharded_optimizer_state_gives_the_unsharded_parameters(kind, dtype, offload):
    """Two emulated ranks that split every group's master and state in two pieces (one after the other on one
    GPU; the reduce to the owner and the broadcast of the updated pieces done by hand) against two ranks that
    each hold everything: identical model parameters after every step, master and state equal on the piece a
    rank holds, and about half the pinned state per rank."""
    import torch
    from paper_2401_15207_b200 import HiFT, HiftError
    half = synth.ModelCfg(arch=2, n_blocks=2, d_model=256, n_heads=2, d_ffn=512, vocab=1000, norm_eps=1e-6,
                          dtype=dtype, batch=2, seq=128, init_std=0.05)
    full = half.scaled(batch=4)
    gc = synth.GroupCfg(1)
    mk = lambda r, w: synth.OptCfg(kind=kind, lr=1e-3, momentum=0.9, weight_decay=0.01, offload_state=offload,
                                   prefetch_groups=2 if offload else 0, shard_rank=r, shard_world=w)
    p0 = synth.init_params(half, 5)
    whole = [HiFT(half, gc, mk(0, 0)) for _ in range(2)]
    shard = [HiFT(half, gc, mk(r, 2)) for r in range(2)]
    try:
        for h in whole + shard:
            h.set_params(p0)
        if offload:
            assert shard[0].pinned_host_bytes() + shard[1].pinned_host_bytes() <= 1.02 * whole[0].pinned_host_bytes()
        n_state = {0: 2, 2: 1}[kind]
        for t in range(2 * whole[0].num_groups()):
            tok, lab = synth.lm_batch(full, 8, t)
            parts = [(torch.from_numpy(tok[:2].copy()).cuda(), torch.from_numpy(lab[:2].copy()).cuda()),
                     (torch.from_numpy(tok[2:].copy()).cuda(), torch.from_numpy(lab[2:].copy()).cuda())]
            g = whole[0].active_group()
            for grp in (whole, shard):
                for h, (tt, ll) in zip(grp, parts):
                    h.step_begin(tt, ll)
                g0, g1 = grp[0].grad_view(), grp[1].grad_view()
                avg = (g0 + g1) * 0.5
                g0.copy_(avg)
                g1.copy_(avg)
                torch.cuda.synchronize()
                for h in grp:
                    h.step_end()
            # the broadcast of the updated pieces: rank r's piece of the group's parameters goes to the other rank
            v0, v1 = shard[0].param_view(), shard[1].param_view()
            for r, (src, dst) in enumerate(((v0, v1), (v1, v0))):
                lo, n = shard[r].shard_range(g, r)
                assert (lo, n) == shard[1 - r].shard_range(g, r)
                dst[lo:lo + n].copy_(src[lo:lo + n])
            torch.cuda.synchronize()
            for name in whole[0].tensor_names():
                ref = whole[0].get_model_param(name)
                for h in shard:
                    assert np.array_equal(h.get_model_param(name), ref), (t, name)
        # master and state on the piece a rank holds; the two pieces tile every tensor
        for name in whole[0].tensor_names():
            ref_m = whole[0].get_param(name).reshape(-1)
            model = whole[0].get_model_param(name).reshape(-1)
            ms = [h.get_param(name).reshape(-1) for h in shard]
            mine = [m != model for m in ms]                  # where a rank returned something other than the model value
            assert np.array_equal(np.where(mine[0], ms[0], ms[1]), np.where(mine[0] | mine[1], ref_m, model)), name
            for w in range(n_state):
                ref_s = whole[0].get_state(name, w).reshape(-1)
                got = sum(h.get_state(name, w).reshape(-1) for h in shard)      # zeros outside a rank's piece
                assert np.array_equal(got, ref_s), (name, w)
        with pytest.raises(HiftError):
            shard[0].save("/tmp/never_written.ckpt")                           # checkpoints are refused while sharded
    finally:
        for h in whole + shard:
            h.close()
    with pytest.raises(HiftError):
        HiFT(half, gc, synth.OptCfg(kind=4, lr=1e-2, eps=1e-30, shard_rank=0, shard_world=2))    # not with Adafactor
