"""Whole-step parity of the CUDA library against the fp64 oracle (through the C ABI)."""
import numpy as np
import pytest

import synth
from gpu_util import lockstep

pytestmark = pytest.mark.gpu

FP32_LOSS, FP32_GRAD = 1e-5, 1e-5
BF16_LOSS, BF16_GRAD = 1e-2, 2e-2


def mini(arch, dtype, **kw):
    base = dict(arch=arch, n_blocks=3, d_model=64, n_heads=4, d_ffn=128, vocab=203, max_pos=48,
                n_classes=2 if arch == 1 else 0, causal=0 if arch == 1 else 1, tie_head=0,
                norm_eps=1e-6 if arch == 2 else 1e-5, dtype=dtype, batch=3, seq=40, init_std=0.08)
    base.update(kw)
    return synth.ModelCfg(**base)


def test_config1_tiny_fp32_full_cycle():
    cfg, gc, oc = synth.config_tiny_fp32()
    rep = lockstep(cfg, gc, oc, 6, "uniform", FP32_LOSS, FP32_GRAD, perturb=0.0, check_update=1e-3, resync=True)
    assert [g for _, g, _, _, _ in rep] == [0, 1, 2, 3, 4, 5]


def test_config1_second_cycle_bias_correction():
    cfg, gc, oc = synth.config_tiny_fp32()
    lockstep(cfg, gc, oc, 8, "uniform", FP32_LOSS, FP32_GRAD, perturb=0.05, check_update=1e-3, resync=True)


@pytest.mark.parametrize("arch", [0, 1, 2])
@pytest.mark.parametrize("order", [0, 1, 2])
def test_mini_fp32_all_archs_orders(arch, order):
    cfg = mini(arch, synth.DTYPE_FP32, tie_head=1 if arch == 0 else 0)
    gc = synth.GroupCfg(layers_per_group=1, order=order, order_seed=11)
    oc = synth.OptCfg(kind=order, lr=1e-3, weight_decay=0.01, eps=1e-8, sched=1, total_cycles=3)
    lockstep(cfg, gc, oc, 7, "zipf", FP32_LOSS, FP32_GRAD, check_update=2e-3, resync=True)


@pytest.mark.parametrize("arch", [0, 1, 2])
def test_mini_fp32_grouped_and_split(arch):
    cfg = mini(arch, synth.DTYPE_FP32, n_blocks=4)
    lockstep(cfg, synth.GroupCfg(layers_per_group=2, split_emb_head=1, order=2, order_seed=3),
             synth.OptCfg(kind=0, lr=1e-3), 4, "zipf", FP32_LOSS, FP32_GRAD, resync=True)
    lockstep(cfg, synth.GroupCfg(layers_per_group=4, split_emb_head=0, order=1),
             synth.OptCfg(kind=2, lr=1e-3), 2, "zipf", FP32_LOSS, FP32_GRAD, resync=True)
    # one group holding every unit: the ordinary full-parameter step
    lockstep(cfg, synth.GroupCfg(layers_per_group=6), synth.OptCfg(kind=1, lr=1e-2, eps=1e-10), 2, "zipf",
             FP32_LOSS, FP32_GRAD, resync=True)


@pytest.mark.parametrize("arch", [0, 1, 2])
@pytest.mark.parametrize("dtype", [synth.DTYPE_FP32, synth.DTYPE_BF16])
def test_right_padded_batches_with_key_lengths(arch, dtype):
    """Batches of unequal length: the key-length table changes from step to step, padded language-model
    positions carry no label; loss and gradients follow the oracle's masked attention."""
    from paper_2401_15207_b200 import HiFT
    bf = dtype == synth.DTYPE_BF16
    cfg = mini(arch, dtype, **(dict(d_model=128, n_heads=2, d_ffn=256) if bf else {}))
    tables = [[40, 17, 1], [5, 40, 33], [40, 40, 40], [2, 3, 9], [29, 1, 40]]
    lockstep(cfg, synth.GroupCfg(layers_per_group=1, order=1), synth.OptCfg(kind=0, lr=1e-3), 5, "zipf",
             BF16_LOSS if bf else FP32_LOSS, BF16_GRAD if bf else FP32_GRAD, resync=True,
             lens=lambda t: tables[t])
    h = HiFT(cfg, synth.GroupCfg(), synth.OptCfg())
    try:
        for bad in ([0, 1, 1], [41, 1, 1]):
            with pytest.raises(RuntimeError):
                h.set_key_lengths(bad)
        h.set_key_lengths([1, 2, 3])
        h.set_key_lengths(None)
    finally:
        h.close()


@pytest.mark.parametrize("arch", [0, 2])
def test_uneven_caller_chosen_groups(arch):
    """Groups of unequal size given as a list of chunk lengths: the same step, the partition is the caller's."""
    from paper_2401_15207_b200 import HiFT
    cfg = mini(arch, synth.DTYPE_FP32, n_blocks=5)                      # 7 units
    gc = synth.GroupCfg(order=1, group_sizes=(2, 1, 3, 1))
    rep = lockstep(cfg, gc, synth.OptCfg(kind=0, lr=1e-3, weight_decay=0.01), 6, "zipf", FP32_LOSS, FP32_GRAD,
                   resync=True)
    assert [g for _, g, _, _, _ in rep] == [3, 2, 1, 0, 3, 2]
    cfgb = mini(arch, synth.DTYPE_BF16, n_blocks=5)
    lockstep(cfgb, synth.GroupCfg(order=0, group_sizes=(1, 4, 2)),
             synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=1), 4, "zipf", BF16_LOSS, BF16_GRAD,
             resync=True)
    for bad in [(2, 1, 3), (7, 0), (3, 3, 3)]:
        with pytest.raises(RuntimeError):
            HiFT(cfg, synth.GroupCfg(group_sizes=bad), synth.OptCfg())


@pytest.mark.parametrize("arch", [0, 1, 2])
@pytest.mark.parametrize("offload,prefetch", [(0, 0), (1, 0), (1, 1)])
def test_mini_bf16_paging_modes(arch, offload, prefetch):
    cfg = mini(arch, synth.DTYPE_BF16, tie_head=1 if arch == 0 else 0)
    gc = synth.GroupCfg(layers_per_group=1, order=0)
    oc = synth.OptCfg(kind=0, lr=1e-3, weight_decay=0.01, offload_state=offload, prefetch_groups=prefetch)
    lockstep(cfg, gc, oc, 7, "zipf", BF16_LOSS, BF16_GRAD, resync=True)


@pytest.mark.parametrize("kind", [1, 2])
def test_mini_bf16_gpt2_style_groups(kind):
    cfg = mini(0, synth.DTYPE_BF16, n_blocks=4, tie_head=1, d_model=128, n_heads=2, d_ffn=256)
    gc = synth.GroupCfg(layers_per_group=2, split_emb_head=1, order=2, order_seed=2401)
    oc = synth.OptCfg(kind=kind, lr=1e-2 if kind == 1 else 1e-3, eps=1e-10, momentum=0.9)
    lockstep(cfg, gc, oc, 5, "zipf", BF16_LOSS, BF16_GRAD, resync=True)


@pytest.mark.parametrize("dtype", [synth.DTYPE_FP32, synth.DTYPE_BF16])
def test_plain_sgd_pages_only_the_master(dtype):
    from paper_2401_15207_b200 import HiFT
    cfg = mini(2, dtype)
    oc = synth.OptCfg(kind=synth.OPT_SGD, lr=1e-2, offload_state=1, prefetch_groups=1)
    tol = (FP32_LOSS, FP32_GRAD) if dtype == synth.DTYPE_FP32 else (BF16_LOSS, BF16_GRAD)
    lockstep(cfg, synth.GroupCfg(1), oc, 6, "zipf", tol[0], tol[1], resync=True)
    h = HiFT(cfg, synth.GroupCfg(1), oc)
    # fp32 parameters + no state: nothing to page at all; bf16: the master alone, which is paged as its
    # low 16 bits + one rounding-carry bit per parameter (the bf16 copy on the GPU holds the rest)
    total = sum(synth.count_params(cfg))
    if dtype == synth.DTYPE_FP32:
        assert h.pinned_host_bytes() < 64
    else:
        assert 2.125 * total <= h.pinned_host_bytes() < 2.125 * total + 64 * 1024
    h.close()


@pytest.mark.parametrize("arch,dtype,offload", [(0, synth.DTYPE_FP32, 1), (2, synth.DTYPE_BF16, 1), (1, synth.DTYPE_BF16, 0)])
def test_adafactor_state_is_rows_plus_cols(arch, dtype, offload):
    from paper_2401_15207_b200 import HiFT
    cfg = mini(arch, dtype, tie_head=1 if arch == 0 else 0)
    oc = synth.OptCfg(kind=synth.OPT_ADAFACTOR, lr=1e-2, eps=1e-30, weight_decay=0.01, offload_state=offload,
                      prefetch_groups=1)
    tol = (FP32_LOSS, FP32_GRAD) if dtype == synth.DTYPE_FP32 else (BF16_LOSS, BF16_GRAD)
    lockstep(cfg, synth.GroupCfg(1), oc, 8, "zipf", tol[0], tol[1], resync=True,
             check_update=2e-3 if dtype == synth.DTYPE_FP32 else None)
    if offload and dtype == synth.DTYPE_FP32:
        h = HiFT(cfg, synth.GroupCfg(1), oc)
        # the whole optimizer state of the model: sum over tensors of rows + cols (vectors: their length)
        want = sum((s[0] + s[1]) if len(s) == 2 else s[0] for u in synth.unit_tensors(cfg) for _, s, _ in u)
        assert 4 * want <= h.pinned_host_bytes() <= 4 * want + 16 * 64
        h.close()


def test_free_running_trajectories_stay_close():
    """No resynchronisation: the two trajectories only share the initial weights."""
    cfg = mini(0, synth.DTYPE_BF16, tie_head=1)
    lockstep(cfg, synth.GroupCfg(1), synth.OptCfg(kind=2, lr=1e-3), 10, "zipf", BF16_LOSS, 2 * BF16_GRAD)


def test_head_dim_128_llama_shape_miniature():
    cfg = mini(2, synth.DTYPE_BF16, n_blocks=2, d_model=256, n_heads=2, d_ffn=344, vocab=1000, batch=2, seq=72)
    lockstep(cfg, synth.GroupCfg(1), synth.OptCfg(kind=0, lr=1e-4), 4, "zipf", BF16_LOSS, BF16_GRAD, resync=True)


def test_invalid_inputs_are_reported_not_faulted():
    import torch
    from paper_2401_15207_b200 import HiFT, HiftError
    cfg, gc, oc = synth.config_tiny_fp32()
    with pytest.raises(HiftError):
        HiFT(cfg.scaled(d_model=130), gc, oc)            # not a multiple of 8
    with pytest.raises(HiftError):
        HiFT(cfg.scaled(max_pos=8), gc, oc)              # position table shorter than seq
    h = HiFT(cfg, gc, oc)
    h.set_params(synth.init_params(cfg, 0))
    tok, lab = synth.lm_batch(cfg, 0, 0, "uniform")
    bad = tok.copy()
    bad[0, 0] = cfg.vocab + 5
    with pytest.raises(HiftError) as e:
        h.step_host(bad, lab)
    assert e.value.status == 4 and h.step_count() == 0   # rejected on the host, nothing ran
    with pytest.raises(HiftError) as e:
        h.step(torch.from_numpy(bad).cuda(), torch.from_numpy(lab).cuda())
    assert e.value.status == 4                            # clamped on the device and reported
    loss = h.step_host(tok, lab)                          # the context is still usable
    assert np.isfinite(loss)
    h.close()


def test_step_host_matches_step_and_is_deterministic():
    import torch
    from paper_2401_15207_b200 import HiFT
    cfg = mini(0, synth.DTYPE_BF16, tie_head=1)
    gc, oc = synth.GroupCfg(1), synth.OptCfg(kind=0, lr=1e-3)
    p0 = synth.init_params(cfg, 4)
    outs = []
    for mode in ("dev", "host", "dev"):
        h = HiFT(cfg, gc, oc)
        h.set_params(p0)
        losses = []
        for t in range(5):
            tok, lab = synth.lm_batch(cfg, 9, t)
            if mode == "dev":
                losses.append(h.step(torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()))
            else:
                losses.append(h.step_host(tok, lab))
        outs.append((losses, h.get_param("tok_emb"), h.get_param("b0.w_qkv")))
        h.close()
    for o in outs[1:]:
        assert o[0] == outs[0][0]                         # same bits, run to run and across entry points
        assert np.array_equal(o[1], outs[0][1]) and np.array_equal(o[2], outs[0][2])


def test_timeout_flag_path_reports_and_recovers():
    """Walk the time-out path without stalling anything: with the flag set, every tensor-core GEMM
    returns at once (releasing its tensor memory), the step reports HIFT_ERR_TIMEOUT, and after the
    flag is cleared the same context computes correct steps again."""
    import torch
    from paper_2401_15207_b200 import HiFT, HiftError, tc_error_flag
    cfg = synth.ModelCfg(arch=2, n_blocks=2, d_model=512, n_heads=4, d_ffn=1024, vocab=1000, norm_eps=1e-6,
                         dtype=synth.DTYPE_BF16, batch=2, seq=256)
    gc, oc = synth.GroupCfg(1), synth.OptCfg(kind=2, lr=1e-3)
    p0 = synth.init_params(cfg, 3)
    tok, lab = synth.lm_batch(cfg, 1, 0)
    tt, ll = torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()
    ref = HiFT(cfg, gc, oc)
    ref.set_params(p0)
    good = [ref.step(tt, ll) for _ in range(2)]
    ref.close()
    h = HiFT(cfg, gc, oc)
    h.set_params(p0)
    assert tc_error_flag() == 0
    try:
        assert tc_error_flag(2) == 2
        with pytest.raises(HiftError) as e:
            h.step(tt, ll)
        assert e.value.status == 6                      # HIFT_ERR_TIMEOUT
    finally:
        assert tc_error_flag(0) == 0
    assert h.step_count() == 0                          # the refused step did not count
    assert [h.step(tt, ll) for _ in range(2)] == good   # and changed nothing: the context goes on like the reference
    h.close()


@pytest.mark.parametrize("kind,offload,dtype", [(0, 1, synth.DTYPE_BF16), (0, 0, synth.DTYPE_BF16),
                                                (4, 1, synth.DTYPE_BF16), (2, 1, synth.DTYPE_FP32)])
def test_checkpoint_resume_is_bitwise(kind, offload, dtype, tmp_path):
    import torch
    from paper_2401_15207_b200 import HiFT, HiftError
    cfg = mini(2, dtype)
    gc = synth.GroupCfg(layers_per_group=2, order=synth.ORDER_RANDOM, order_seed=4)
    oc = synth.OptCfg(kind=kind, lr=1e-3, eps=1e-8 if kind != 4 else 1e-30, sched=1, total_cycles=5,
                      offload_state=offload, prefetch_groups=1)
    batches = [tuple(torch.from_numpy(a).cuda() for a in synth.lm_batch(cfg, 6, t)) for t in range(9)]
    a = HiFT(cfg, gc, oc)
    a.set_params(synth.init_params(cfg, 2))
    for t in range(4):
        a.step(*batches[t])
    path = str(tmp_path / "ckpt.bin")
    a.save(path)
    b = HiFT(cfg, gc, oc)
    b.load(path)
    assert b.step_count() == 4 and b.active_group() == a.active_group() and b.current_lr() == a.current_lr()
    for t in range(4, 9):
        assert a.step(*batches[t]) == b.step(*batches[t])
    for n in a.tensor_names():
        assert np.array_equal(a.get_param(n), b.get_param(n)), n
        assert np.array_equal(a.get_model_param(n), b.get_model_param(n)), n
    other = HiFT(cfg, gc, synth.OptCfg(kind=(kind + 1) % 3, lr=1e-3))
    with pytest.raises(HiftError):
        other.load(path)                                   # different optimizer: refused
    with pytest.raises(HiftError):
        b.load(str(tmp_path / "missing.bin"))
    regrouped = HiFT(cfg, synth.GroupCfg(order=synth.ORDER_RANDOM, order_seed=4, group_sizes=(1, 2, 2)), oc)
    assert regrouped.num_groups() == a.num_groups()
    with pytest.raises(HiftError):
        regrouped.load(path)                               # same number of groups, other partition: refused
    for h in (a, b, other, regrouped):
        h.close()


def _rne_bf16_bits(u):
    """bf16 bit pattern of fp32 bit patterns `u` (uint32), round to nearest even; finite inputs."""
    u = u.astype(np.uint64)
    return (((u + 0x7FFF + ((u >> 16) & 1)) >> 16) & 0xFFFF).astype(np.uint32)


@pytest.mark.parametrize("kind", [0, 2, synth.OPT_SGD])
def test_paged_master_round_trip_is_exact(kind):
    """With bf16 parameters the paged master is 16 low bits + a carry bit beside the bf16 copy.  Every
    fp32 value written must come back bit for bit, in particular the low half 0x8000 (a rounding tie,
    which lands on the same bf16 value from an even and from an odd upper half), both signs, zeros,
    denormals, the largest finite value and infinity; and the model copy must be the RNE bf16 value."""
    from paper_2401_15207_b200 import HiFT
    cfg = mini(2, synth.DTYPE_BF16)
    oc = synth.OptCfg(kind=kind, lr=1e-3, offload_state=1, prefetch_groups=1)
    h = HiFT(cfg, synth.GroupCfg(1), oc)
    try:
        name = [n for n in h.tensor_names() if h._numel(n) >= 4096][0]
        n = h._numel(name)
        rng = np.random.default_rng(7)
        u = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
        u &= np.uint32(0xFF7FFFFF)                       # keep the exponent below all-ones: finite
        lows = np.array([0, 1, 0x7FFF, 0x8000, 0x8001, 0xFFFF], dtype=np.uint32)
        k = 0
        for hi in (0x3F80, 0x3F81, 0xBF80, 0xBF81, 0x0000, 0x8000, 0x0001, 0x7F7F, 0xFF7F):
            for lo in lows:
                u[k] = np.uint32((hi << 16) | int(lo)); k += 1
        u[k] = 0x7F800000; u[k + 1] = 0xFF800000         # infinities
        h.set_param(name, u.view(np.float32))
        back = np.asarray(h.get_param(name), dtype=np.float32).reshape(-1).view(np.uint32)
        assert np.array_equal(back, u)
        model = np.asarray(h.get_model_param(name), dtype=np.float32).reshape(-1).view(np.uint32)
        fin = (u & 0x7F800000) != 0x7F800000
        assert np.array_equal(model[fin] >> 16, _rne_bf16_bits(u[fin]))
        assert np.all(model & 0xFFFF == 0)
    finally:
        h.close()


@pytest.mark.parametrize("kind", [0, 1, 2, synth.OPT_SGD])
def test_paged_and_resident_state_give_identical_bits(kind):
    """Keeping the state on the GPU (fp32 master) and paging it (compact master; one slot in the paper's
    order, two slots, or a ring of three / four slots whose uploads run one / two steps ahead) are storage
    forms of the same numbers: after two cycles every master value and state value agrees bit for bit."""
    import torch
    from paper_2401_15207_b200 import HiFT
    cfg = mini(0, synth.DTYPE_BF16, tie_head=1)
    gc = synth.GroupCfg(layers_per_group=1, order=1)
    p0 = synth.init_params(cfg, 3, perturb=0.05)
    ctxs = []
    for offload, prefetch in ((0, 0), (1, 1), (1, 0), (1, 2), (1, 3)):
        oc = synth.OptCfg(kind=kind, lr=1e-2, eps=1e-8, momentum=0.9, weight_decay=0.01, offload_state=offload,
                          prefetch_groups=prefetch)
        h = HiFT(cfg, gc, oc)
        h.set_params(p0)
        ctxs.append(h)
    try:
        k = ctxs[0].num_groups()
        for t in range(2 * k):
            tok, lab = synth.batch_for(cfg, 11, t, "zipf")
            dt, dl = torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()
            losses = [h.step(dt, dl) for h in ctxs]
            assert all(l == losses[0] for l in losses)
        n_state = {0: 2, 1: 1, 2: 1}.get(kind, 0)
        for name in ctxs[0].tensor_names():
            ref = np.asarray(ctxs[0].get_param(name)).view(np.uint32)
            for h in ctxs[1:]:
                assert np.array_equal(np.asarray(h.get_param(name)).view(np.uint32), ref), name
                assert np.array_equal(np.asarray(h.get_model_param(name)).view(np.uint32),
                                      np.asarray(ctxs[0].get_model_param(name)).view(np.uint32)), name
            for w in range(n_state):
                sref = np.asarray(ctxs[0].get_state(name, w)).view(np.uint32)
                for h in ctxs[1:]:
                    assert np.array_equal(np.asarray(h.get_state(name, w)).view(np.uint32), sref), (name, w)
    finally:
        for h in ctxs:
            h.close()


def _state_bits(h, n_state):
    out = {}
    for name in h.tensor_names():
        out[name] = [np.asarray(h.get_param(name)).view(np.uint32).copy(),
                     np.asarray(h.get_model_param(name)).view(np.uint32).copy()]
        for w in range(n_state):
            out[name].append(np.asarray(h.get_state(name, w)).view(np.uint32).copy())
        if h.opt.kind == 4:
            rows = h.tensor_info(name)[1][0]
            for w in range(1 if rows == 1 else 2):
                out[name].append(np.asarray(h.get_factored_state(name, w)).view(np.uint32).copy())
    return out


def _same_bits(a, b):
    for name in a:
        for x, y in zip(a[name], b[name]):
            assert np.array_equal(x, y), name


@pytest.mark.parametrize("prefetch", [0, 1, 2, 3])
@pytest.mark.parametrize("case", ["one_group", "forced", "two_groups", "forced_then_schedule", "sequence"])
def test_paging_when_a_group_trains_on_consecutive_steps(case, prefetch):
    """A group that is trained again before (or while) its write-back lands must be updated from its
    latest values: one group holding every unit (k = 1, the full-parameter identity of Eq. 2-3), a
    forced group, fewer groups than state slots, leaving a forced group with uploads of the
    schedule's groups outstanding, and a forced list of groups with repeats.  The paged run keeps the bits of the run with the state resident."""
    import torch
    from paper_2401_15207_b200 import HiFT
    cfg = mini(0, synth.DTYPE_BF16, tie_head=1)
    n = cfg.n_units
    gc = {"one_group": synth.GroupCfg(layers_per_group=n), "forced": synth.GroupCfg(1),
          "two_groups": synth.GroupCfg(layers_per_group=(n + 1) // 2),
          "forced_then_schedule": synth.GroupCfg(1), "sequence": synth.GroupCfg(1)}[case]
    p0 = synth.init_params(cfg, 3, perturb=0.05)
    ctxs = []
    for offload in (0, 1):
        h = HiFT(cfg, gc, synth.OptCfg(kind=0, lr=1e-2, weight_decay=0.01, offload_state=offload,
                                       prefetch_groups=prefetch if offload else 0))
        h.set_params(p0)
        ctxs.append(h)
    try:
        if case == "sequence":
            for h in ctxs:
                h.force_sequence([2, 0, 2, 3, 3, 1])
        for t in range(7):
            if case == "sequence":
                assert ctxs[1].active_group() == [2, 0, 2, 3, 3, 1][t % 6]
            if case == "forced":
                for h in ctxs:
                    h.force_group(2 if t < 4 else 1)
            if case == "forced_then_schedule":
                for h in ctxs:
                    h.force_group(3 if 2 <= t < 5 else -1)
            tok, lab = synth.batch_for(cfg, 11, t, "zipf")
            dt, dl = torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()
            assert ctxs[0].active_group() == ctxs[1].active_group()
            a, b = ctxs[0].step(dt, dl), ctxs[1].step(dt, dl)
            assert a == b, (t, a, b)
        _same_bits(_state_bits(ctxs[0], 2), _state_bits(ctxs[1], 2))
    finally:
        for h in ctxs:
            h.close()


@pytest.mark.parametrize("kind,offload,prefetch,dtype", [(0, 1, 2, synth.DTYPE_BF16), (0, 0, 0, synth.DTYPE_BF16),
                                                         (4, 1, 1, synth.DTYPE_BF16), (2, 1, 0, synth.DTYPE_FP32)])
def test_a_failed_step_changes_nothing(kind, offload, prefetch, dtype):
    """A step that reports a time-out (walked with the host-set flag: nothing stalls), a bad label or a
    non-finite loss (a NaN planted in a parameter of a frozen group through hift_set_param) leaves every
    parameter, master and state bit of every group as it was, does not advance t or the group's update
    count, and the same context then continues exactly like one that never saw the failure."""
    import torch
    from paper_2401_15207_b200 import HiFT, HiftError, tc_error_flag
    cfg = synth.ModelCfg(arch=2, n_blocks=2, d_model=256, n_heads=2, d_ffn=512, vocab=1000, norm_eps=1e-6,
                         dtype=dtype, batch=2, seq=128)
    gc = synth.GroupCfg(1)
    oc = synth.OptCfg(kind=kind, lr=1e-3, eps=1e-8 if kind != 4 else 1e-30, weight_decay=0.01,
                      offload_state=offload, prefetch_groups=prefetch)
    n_state = {0: 2, 1: 1, 2: 1}.get(kind, 0)
    p0 = synth.init_params(cfg, 3)
    batches = [tuple(torch.from_numpy(a).cuda() for a in synth.lm_batch(cfg, 1, t)) for t in range(6)]
    ref, h = HiFT(cfg, gc, oc), HiFT(cfg, gc, oc)
    try:
        for c in (ref, h):
            c.set_params(p0)
            for t in range(2):
                c.step(*batches[t])
        before = _state_bits(h, n_state)
        # (1) time-out flag (only the tensor-core path reads it)
        if dtype == synth.DTYPE_BF16:
            try:
                assert tc_error_flag(2) == 2
                with pytest.raises(HiftError) as e:
                    h.step(*batches[2])
                assert e.value.status == 6
            finally:
                assert tc_error_flag(0) == 0
            assert h.step_count() == 2 and h.active_group() == ref.active_group()
            _same_bits(before, _state_bits(h, n_state))
        # (2) a label beyond the vocabulary
        bad = batches[2][1].clone()
        bad[0, 3] = cfg.vocab + 7
        with pytest.raises(HiftError) as e:
            h.step(batches[2][0], bad)
        assert e.value.status == 4 and h.step_count() == 2
        _same_bits(before, _state_bits(h, n_state))
        # (3) non-finite loss: NaN in a tensor of a group that is not the active one
        g = h.active_group()
        lo, hi = h.group_units(g)
        victim = [n for n in h.tensor_names() if not (lo <= h.tensor_info(n)[0] <= hi) and n.endswith("w_o")][0]
        good = h.get_param(victim)
        poisoned = good.copy()
        poisoned[0, 0] = np.nan
        h.set_param(victim, poisoned)
        with_nan = _state_bits(h, n_state)
        with pytest.raises(HiftError) as e:
            h.step(*batches[2])
        assert e.value.status == 5 and h.step_count() == 2
        _same_bits(with_nan, _state_bits(h, n_state))
        h.set_param(victim, good)
        _same_bits(before, _state_bits(h, n_state))
        # and on it goes, bit for bit like the context that never failed
        for t in range(2, 6):
            assert h.step(*batches[t]) == ref.step(*batches[t])
        _same_bits(_state_bits(ref, n_state), _state_bits(h, n_state))
    finally:
        ref.close()
        h.close()


def test_warmup_then_decay_moves_once_per_cycle():
    """Linear schedule with a warm-up counted in cycles: the learning rate the library reports is
    bit-identical to the oracle's in every step, and the first cycle, run at rate 0, leaves every
    parameter untouched under SGD (so the reported rate is the one used)."""
    from paper_2401_15207_b200 import HiFT
    import torch
    cfg = mini(2, synth.DTYPE_FP32)
    oc = synth.OptCfg(kind=synth.OPT_SGD, lr=1e-2, sched=synth.SCHED_LINEAR, total_cycles=4, warmup_cycles=2, offload_state=0)
    gc = synth.GroupCfg(layers_per_group=2)
    h = HiFT(cfg, gc, oc)
    p0 = synth.init_params(cfg, 3, perturb=0.05)
    h.set_params(p0)
    k = h.num_groups()
    lrs = []
    for t in range(4 * k):
        lrs.append(h.current_lr())
        tok, lab = synth.batch_for(cfg, 9, t, "zipf")
        h.step(torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda())
        if t == k - 1:
            for name in h.tensor_names():
                assert np.array_equal(np.asarray(h.get_param(name)).reshape(-1), np.asarray(p0[name], dtype=np.float32).reshape(-1)), name
    h.close()
    from oracle import hift_oracle as O
    assert lrs == [O.lr_for_cycle(oc.lr, oc.sched, t // k, oc.total_cycles, oc.warmup_cycles) for t in range(4 * k)]
    assert lrs == pytest.approx([0.0] * k + [0.5e-2] * k + [1e-2] * k + [0.5e-2] * k, rel=1e-15, abs=0.0)


@pytest.mark.parametrize("switch", [0, 1])
@pytest.mark.parametrize("arch", [0, 2])
def test_dependent_launch_and_cta_pairs_change_no_bits(arch, switch):
    """Programmatic dependent launch lets a kernel start under its predecessor's tail (it must wait before it
    touches memory), and CTA-pair tiles split one output tile over two SMs: neither may change a bit.  The same
    two cycles with the switch on (the default) and off, on a model large enough for the tensor-core kernels:
    every loss and every parameter bit agree."""
    import hashlib
    import torch
    from paper_2401_15207_b200 import HiFT, code_path_switch
    cfg = synth.ModelCfg(arch=arch, n_blocks=3, d_model=256, n_heads=2 if arch == 2 else 4, d_ffn=768 if arch == 2 else 1024,
                         vocab=1000, max_pos=128, causal=1, tie_head=0, norm_eps=1e-6 if arch == 2 else 1e-5,
                         dtype=synth.DTYPE_BF16, batch=2, seq=128, init_std=0.05)
    oc = synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=1)
    outs = []
    old = code_path_switch(switch, -1)
    try:
        for value in (1, 0):
            code_path_switch(switch, value)
            h = HiFT(cfg, synth.GroupCfg(1), oc)
            try:
                h.set_params(synth.init_params(cfg, 4, perturb=0.05))
                losses = []
                for t in range(2 * h.num_groups()):
                    tok, lab = synth.batch_for(cfg, 21, t, "zipf")
                    losses.append(h.step(torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()))
                m = hashlib.sha256()
                for n in h.tensor_names():
                    m.update(np.ascontiguousarray(h.get_param(n)).tobytes())
                outs.append((m.hexdigest(), losses))
            finally:
                h.close()
    finally:
        code_path_switch(switch, old)
    assert outs[0] == outs[1]


@pytest.mark.parametrize("arch", [0, 1, 2])
def test_recomputing_frozen_blocks_changes_no_bits_and_saves_memory(arch):
    """recompute = 1: the frozen blocks above the active group keep only their input in the forward pass and
    are run again, one at a time, in the backward pass.  The kernels are deterministic, so the losses and every
    parameter bit are those of the keeping mode; the activation arena is smaller."""
    import torch
    from paper_2401_15207_b200 import HiFT
    cfg = mini(arch, synth.DTYPE_BF16, n_blocks=4, tie_head=1 if arch == 0 else 0)
    gc = synth.GroupCfg(layers_per_group=1, order=0)
    p0 = synth.init_params(cfg, 5, perturb=0.05)
    ctxs = []
    for rc in (0, 1):
        h = HiFT(cfg, gc, synth.OptCfg(kind=0, lr=1e-3, weight_decay=0.01, offload_state=1, prefetch_groups=1, recompute=rc))
        h.set_params(p0)
        ctxs.append(h)
    try:
        assert ctxs[1].peak_hbm_bytes() < ctxs[0].peak_hbm_bytes()
        for t in range(ctxs[0].num_groups()):
            tok, lab = synth.batch_for(cfg, 13, t, "zipf")
            dt, dl = torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()
            assert ctxs[0].step(dt, dl) == ctxs[1].step(dt, dl), t
        for name in ctxs[0].tensor_names():
            assert np.array_equal(np.asarray(ctxs[0].get_param(name)).view(np.uint32),
                                  np.asarray(ctxs[1].get_param(name)).view(np.uint32)), name
    finally:
        for h in ctxs:
            h.close()


def test_host_batches_from_pinned_and_pageable_memory_agree():
    """hift_step_host takes the batch from pageable memory (staged copy) or from pinned memory (read by a small
    kernel, so that it cannot queue behind the state transfers on a copy engine): same step either way."""
    import torch
    from paper_2401_15207_b200 import HiFT
    cfg = mini(2, synth.DTYPE_BF16)
    gc, oc = synth.GroupCfg(1), synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=1)
    p0 = synth.init_params(cfg, 6, perturb=0.05)
    a, b = HiFT(cfg, gc, oc), HiFT(cfg, gc, oc)
    try:
        a.set_params(p0)
        b.set_params(p0)
        for t in range(a.num_groups()):
            tok, lab = synth.batch_for(cfg, 17, t, "zipf")
            ptok, plab = torch.from_numpy(tok.astype(np.int32)).pin_memory(), torch.from_numpy(lab.astype(np.int32)).pin_memory()
            assert a.step_host(tok, lab) == b.step_host(ptok.numpy(), plab.numpy())
        for name in a.tensor_names():
            assert np.array_equal(a.get_param(name), b.get_param(name)), name
    finally:
        a.close()
        b.close()


def test_pinned_allocation_failure_is_reported_and_leaves_nothing_behind():
    """hift_create when the host runs out of pinned memory, without exhausting anything: the library's test
    switch makes the n-th pinned allocation fail.  Whichever one it is (the first group's blob, a later one, the
    mapped scalar words after all blobs), the call reports HIFT_ERR_OOM_PINNED, releases what it had allocated
    (device memory returns to its level), and the next hift_create succeeds."""
    import torch
    from paper_2401_15207_b200 import HiFT, HiftError, code_path_switch
    cfg = mini(0, synth.DTYPE_BF16)
    gc, oc = synth.GroupCfg(1), synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=2)
    warm = HiFT(cfg, gc, oc)                                  # loads the kernels, so that later memory readings are steady
    k = warm.num_groups()
    warm.close()
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for n in (0, 2, k):                                       # blobs are allocated first, one per group, then the scalar words
        try:
            code_path_switch(4, n)
            with pytest.raises(HiftError) as e:
                HiFT(cfg, gc, oc)
            assert e.value.status == 3 and "pinned" in str(e.value)
            assert code_path_switch(4, -1) == -1              # the injected failure was consumed
        finally:
            code_path_switch(4, -1)
        torch.cuda.synchronize()
        assert abs(torch.cuda.mem_get_info()[0] - free0) <= (4 << 20)
    h = HiFT(cfg, gc, oc)
    # what the context says it holds is what the driver handed out (allocation granularity aside)
    used = free0 - torch.cuda.mem_get_info()[0]
    assert h.peak_hbm_bytes() <= used <= h.peak_hbm_bytes() + (64 << 20)
    h.set_params(synth.init_params(cfg, 1))
    tok, lab = synth.batch_for(cfg, 2, 0, "zipf")
    assert np.isfinite(h.step(torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()))
    h.close()


@pytest.mark.parametrize("arch,dtype,big", [(0, synth.DTYPE_FP32, False), (1, synth.DTYPE_BF16, False), (2, synth.DTYPE_BF16, False),
                                            (0, synth.DTYPE_BF16, True), (1, synth.DTYPE_BF16, True), (2, synth.DTYPE_BF16, True)])
def test_checked_mode_no_kernel_writes_past_its_buffer(arch, dtype, big):
    """Checked mode puts a painted guard region behind every slice of the activation arena (work buffers,
    scratch slots, kept activations) and looks at them after the step: with ragged sizes on the CUDA-core
    kernels and with tile-sized ones on the tensor-core kernels, over a full cycle (every retention plan),
    not one region is touched.  Stands in for a memory checker on the arena, which holds every buffer the
    step's kernels write except parameters, gradients and state."""
    import torch
    from paper_2401_15207_b200 import HiFT, code_path_switch
    if big:
        cfg = synth.ModelCfg(arch=arch, n_blocks=2, d_model=256, n_heads=2 if arch == 2 else 4, d_ffn=640, vocab=1001,
                             max_pos=160, n_classes=2 if arch == 1 else 0, causal=0 if arch == 1 else 1,
                             norm_eps=1e-6 if arch == 2 else 1e-5, dtype=dtype, batch=2, seq=160, init_std=0.05)
    else:
        cfg = mini(arch, dtype)
    old = code_path_switch(5, 1)
    try:
        h = HiFT(cfg, synth.GroupCfg(1), synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=1, recompute=1 if big else 0))
    finally:
        code_path_switch(5, old)
    try:
        assert h.arena_guard_count() > 20
        h.set_params(synth.init_params(cfg, 2))
        for t in range(h.num_groups()):
            tok, lab = synth.batch_for(cfg, 4, t, "zipf")
            h.step(torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda())
            assert h.check_arena() == 0, (t, h.check_arena())
    finally:
        h.close()
    plain = HiFT(cfg, synth.GroupCfg(1), synth.OptCfg(kind=0, lr=1e-3))
    assert plain.check_arena() == -1 and plain.arena_guard_count() == -1
    plain.close()


@pytest.mark.parametrize("arch,dtype", [(0, synth.DTYPE_FP32), (1, synth.DTYPE_FP32), (2, synth.DTYPE_FP32),
                                        (0, synth.DTYPE_BF16), (1, synth.DTYPE_BF16), (2, synth.DTYPE_BF16)])
def test_dropout_masks_match_the_oracle(arch, dtype):
    """Dropout at the three kinds of site (embedding output, attention output, feed-forward output) with masks
    both sides draw from Philox4x32-10 keyed by (seed, step, site, element): a full cycle in lockstep, fp32 at
    1e-5 (a single differing mask bit would move the loss far more) and bf16 at the bf16 tolerances."""
    fp32 = dtype == synth.DTYPE_FP32
    if fp32:
        cfg = mini(arch, dtype, dropout=0.15, dropout_seed=0x1234_5678_9ABC)
    else:
        cfg = synth.ModelCfg(arch=arch, n_blocks=2, d_model=256, n_heads=2 if arch == 2 else 4, d_ffn=512, vocab=1001, max_pos=128,
                             n_classes=2 if arch == 1 else 0, causal=0 if arch == 1 else 1, norm_eps=1e-6 if arch == 2 else 1e-5,
                             dtype=dtype, batch=2, seq=128, init_std=0.05, dropout=0.1, dropout_seed=77)
    oc = synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=1)
    lockstep(cfg, synth.GroupCfg(1), oc, cfg.n_units + 1, "zipf", FP32_LOSS if fp32 else BF16_LOSS, FP32_GRAD if fp32 else BF16_GRAD,
             resync=True)


@pytest.mark.parametrize("arch,dtype", [(0, synth.DTYPE_FP32), (1, synth.DTYPE_FP32), (2, synth.DTYPE_FP32),
                                        (0, synth.DTYPE_BF16), (1, synth.DTYPE_BF16), (2, synth.DTYPE_BF16)])
@pytest.mark.parametrize("both", [0, 1])
def test_attention_probability_dropout_matches_the_oracle(arch, dtype, both):
    """Dropout on the attention probabilities (after the softmax, own rate, site 1000 + block, elements numbered with
    rows padded to a multiple of four), alone and together with the dropout of the residual branches: a full cycle
    in lockstep with the oracle.  The fp32 miniature has sequence length 40 with ragged key lengths and head size
    16; the bf16 configurations have head sizes 64 and 128, whose attention leaves the tensor-core kernels when
    this rate is above 0."""
    fp32 = dtype == synth.DTYPE_FP32
    extra = dict(attn_dropout=0.2, dropout_seed=0xABCDEF0123, dropout=0.1 if both else 0.0)
    if fp32:
        cfg = mini(arch, dtype, **extra)
    else:
        cfg = synth.ModelCfg(arch=arch, n_blocks=2, d_model=256, n_heads=2 if arch == 2 else 4, d_ffn=512, vocab=1001, max_pos=128,
                             n_classes=2 if arch == 1 else 0, causal=0 if arch == 1 else 1, norm_eps=1e-6 if arch == 2 else 1e-5,
                             dtype=dtype, batch=2, seq=128, init_std=0.05, **extra)
    oc = synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=1)
    lens = (lambda t: [cfg.seq - (3 * t + 5 * b) % (cfg.seq // 2) for b in range(cfg.batch)]) if fp32 and not both else None
    lockstep(cfg, synth.GroupCfg(1), oc, cfg.n_units + 1, "zipf", FP32_LOSS if fp32 else BF16_LOSS, FP32_GRAD if fp32 else BF16_GRAD,
             resync=True, lens=lens)


def test_dropout_is_reproducible_and_recompute_redraws_the_same_masks():
    import torch
    from paper_2401_15207_b200 import HiFT
    base = dict(arch=2, n_blocks=3, d_model=256, n_heads=2, d_ffn=512, vocab=1001, norm_eps=1e-6, dtype=synth.DTYPE_BF16,
                batch=2, seq=128, init_std=0.05)
    p0 = synth.init_params(synth.ModelCfg(**base), 4)

    def run(recompute=0, **kw):
        cfg = synth.ModelCfg(**base, **kw)
        h = HiFT(cfg, synth.GroupCfg(1), synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=2, recompute=recompute))
        try:
            h.set_params(p0)
            out = []
            for t in range(h.num_groups()):
                tok, lab = synth.lm_batch(cfg, 9, t)
                out.append(h.step(torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()))
            return out, [h.get_param(n).copy() for n in h.tensor_names()]
        finally:
            h.close()

    plain, _ = run()
    zero, _ = run(dropout=0.0, dropout_seed=5)
    a, pa = run(dropout=0.2, dropout_seed=5)
    b, pb = run(dropout=0.2, dropout_seed=5)
    c, _ = run(dropout=0.2, dropout_seed=6)
    r, pr = run(recompute=1, dropout=0.2, dropout_seed=5)
    ad, pad = run(attn_dropout=0.2, dropout_seed=5)
    adr, padr = run(recompute=1, attn_dropout=0.2, dropout_seed=5)
    assert ad != plain and ad != a            # the probabilities' masks act, and are not the branches' masks
    assert ad == adr and all(np.array_equal(x, y) for x, y in zip(pad, padr))
    assert plain == zero                      # p = 0 is the plain model, whatever the seed
    assert a == b and all(np.array_equal(x, y) for x, y in zip(pa, pb))
    assert a != plain and a != c              # the masks act, and follow the seed
    assert a == r and all(np.array_equal(x, y) for x, y in zip(pa, pr))   # a recomputed block draws its masks again


@pytest.mark.parametrize("arch,dtype,m,order", [(0, synth.DTYPE_FP32, 2, 0), (1, synth.DTYPE_FP32, 2, 1), (2, synth.DTYPE_FP32, 3, 2),
                                                (2, synth.DTYPE_FP32, 4, 0), (0, synth.DTYPE_BF16, 2, 0), (2, synth.DTYPE_BF16, 3, 1)])
def test_literal_queue_with_drifting_sets(arch, dtype, m, order):
    """Algorithm 1 c-d taken literally with m not dividing n (5 units): sets drift and wrap around (the top and
    the bottom unit trained together, which makes the backward pass run the whole depth with weight gradients at
    both ends only), every unit keeps its own state and update count.  A full period and more in lockstep with
    the oracle: set ids, learning rate (moves every k = floor(n/m) + 1 steps), loss, gradients, frozen bits, and
    the in-step update from the library's own gradient."""
    from paper_2401_15207_b200 import HiFT
    fp32 = dtype == synth.DTYPE_FP32
    cfg = mini(arch, dtype, tie_head=1 if arch == 0 else 0)
    gc = synth.GroupCfg(layers_per_group=m, order=order, order_seed=5, literal_queue=1)
    oc = synth.OptCfg(kind=0, lr=1e-3, weight_decay=0.01, sched=1, total_cycles=6, offload_state=1, prefetch_groups=2)
    h = HiFT(cfg, gc, oc)
    try:
        import math
        n = cfg.n_units
        assert h.num_groups() == n // m + 1 and h.num_sets() == n // math.gcd(n, m)
        from oracle import hift_oracle as O
        walk = O.queue_walk(n, m, order, h.num_sets(), 5)
        assert [h.set_units(s) for s in range(h.num_sets())] == [sorted(e) for e in walk]
    finally:
        h.close()
    lockstep(cfg, gc, oc, n // math.gcd(n, m) + 2, "zipf", FP32_LOSS if fp32 else BF16_LOSS, FP32_GRAD if fp32 else BF16_GRAD,
             resync=True)


def test_literal_queue_equals_the_fixed_partition_when_m_divides_n():
    import torch
    from paper_2401_15207_b200 import HiFT
    cfg = mini(2, synth.DTYPE_BF16, n_blocks=4)                 # 6 units, m = 2
    p0 = synth.init_params(cfg, 2)
    outs = []
    for lq in (0, 1):
        h = HiFT(cfg, synth.GroupCfg(layers_per_group=2, order=1, literal_queue=lq), synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=2))
        h.set_params(p0)
        assert h.num_sets() == h.num_groups() == 3
        losses = []
        for t in range(6):
            tok, lab = synth.lm_batch(cfg, 3, t)
            losses.append(h.step(torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()))
        outs.append((losses, [h.get_param(n).copy() for n in h.tensor_names()]))
        h.close()
    assert outs[0][0] == outs[1][0] and all(np.array_equal(a, b) for a, b in zip(outs[0][1], outs[1][1]))


@pytest.mark.parametrize("arch,big", [(0, True), (1, True), (2, True), (0, False), (2, False)])
def test_gradients_kept_in_bf16(arch, big):
    """grad_bf16: the weight-gradient GEMMs store bf16 from their fp32 accumulators (tensor-core and CUDA-core
    kernels), the reductions and the embedding scatter round once (a tied head's share and the embedding's share
    meet in bf16), the optimizer reads bf16.  In lockstep with the oracle at the bf16 tolerances; the update given
    the library's own (bf16) gradient still agrees to 1e-6; every stored gradient is a bf16 value; the gradient
    buffer is half the size."""
    import torch
    from paper_2401_15207_b200 import HiFT
    if big:
        cfg = synth.ModelCfg(arch=arch, n_blocks=2, d_model=256, n_heads=2 if arch == 2 else 4, d_ffn=512, vocab=1001, max_pos=128,
                             n_classes=2 if arch == 1 else 0, causal=0 if arch == 1 else 1, tie_head=1 if arch == 0 else 0,
                             norm_eps=1e-6 if arch == 2 else 1e-5, dtype=synth.DTYPE_BF16, batch=2, seq=128, init_std=0.05)
    else:
        cfg = mini(arch, synth.DTYPE_BF16, tie_head=1 if arch == 0 else 0)
    gc = synth.GroupCfg(1)
    oc = synth.OptCfg(kind=0, lr=1e-3, weight_decay=0.01, offload_state=1, prefetch_groups=2, grad_bf16=1)
    lockstep(cfg, gc, oc, cfg.n_units + 1, "zipf", BF16_LOSS, BF16_GRAD, resync=True)
    a, b = HiFT(cfg, gc, oc), HiFT(cfg, gc, synth.OptCfg(**{**oc.__dict__, "grad_bf16": 0}))
    try:
        biggest = max(sum(int(np.prod(a.tensor_info(n)[1])) for n in a.tensor_names() if a.tensor_info(n)[0] == u) for u in range(cfg.n_units))
        assert b.peak_hbm_bytes() - a.peak_hbm_bytes() >= 2 * biggest - 4096          # 4 -> 2 bytes per gradient element
        for h in (a, b):
            h.set_params(synth.init_params(cfg, 2))
        tok, lab = synth.batch_for(cfg, 3, 0, "zipf")
        tt, ll = torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()
        la, lb = a.step(tt, ll), b.step(tt, ll)
        assert la == lb                                                                  # the forward pass is the same
        for n in a.tensor_names():
            if a.tensor_info(n)[0] == 0:
                ga, gb = a.get_grad(n), b.get_grad(n)
                assert not (ga.view(np.uint32) & 0xFFFF).any()                           # bf16 values
                assert np.abs(ga - gb).max() <= 2.0 ** -8 * np.abs(gb).max() + 1e-30
        assert a.grad_view().dtype == torch.bfloat16 and b.grad_view().dtype == torch.float32
    finally:
        a.close()
        b.close()
    with pytest.raises(Exception):
        HiFT(cfg.scaled(dtype=synth.DTYPE_FP32), gc, oc)                                 # bf16 gradients need a bf16 model


@pytest.mark.parametrize("arch,dtype", [(0, synth.DTYPE_FP32), (2, synth.DTYPE_BF16)])
def test_embedding_gradient_with_more_tokens_than_one_occurrence_list(arch, dtype):
    """12288 tokens a step over a vocabulary of 31 ids: the commonest id sits at some thousands of positions,
    more than the embedding-gradient kernel lists at once, so its row is summed in several passes; the first
    step of the cycle trains the embedding group."""
    bf = dtype == synth.DTYPE_BF16
    cfg = mini(arch, dtype, n_blocks=1, vocab=31, batch=24, seq=512, max_pos=512, tie_head=1 if arch == 0 else 0)
    tok, _ = synth.batch_for(cfg, 5, 0, "zipf")
    assert np.bincount(tok.reshape(-1)).max() > 2048
    lockstep(cfg, synth.GroupCfg(layers_per_group=1, order=0), synth.OptCfg(kind=0, lr=1e-3), 1, "zipf",
             BF16_LOSS if bf else FP32_LOSS, BF16_GRAD if bf else FP32_GRAD, resync=True)
