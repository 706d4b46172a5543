"""Pins for the oracle's Algorithm-1 bookkeeping: grouping, order, delayed LR,
memory model.  None of these needs a GPU."""
import os

import numpy as np
import pytest

import synth
from oracle import hift_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_figures.txt")


def _golden():
    out = {}
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        kv = line.split("|")[0]
        k, v = kv.split("=")
        out[k.strip()] = float(v)
    return out


def test_k_formula_grid():
    # paper, Notation: k = n/m if m | n else floor(n/m)+1  == ceil(n/m)
    for n in range(1, 60):
        for m in range(1, n + 1):
            k = O.num_groups(n, m)
            assert k == -(-n // m)
            groups = O.build_groups(n, m)
            assert len(groups) == k
            assert sum(groups, []) == list(range(n))            # a partition, in order
            assert all(len(g) == m for g in groups[:-1])
            assert 1 <= len(groups[-1]) <= m


def test_llama_units_and_groups_match_paper():
    g = _golden()
    cfg, gc, _ = synth.config_llama_7b()
    assert cfg.n_units == g["llama7b_units_n"]
    assert len(O.build_groups(cfg.n_units, 1)) == g["llama7b_groups_k_at_m1"]


def test_split_grouping_gpt2_large():
    cfg, gc, _ = synth.config_gpt2_large()
    groups = O.build_groups(cfg.n_units, gc.layers_per_group, gc.split_emb_head)
    assert len(groups) == 20
    assert groups[0] == [0] and groups[-1] == [37]
    assert groups[1] == [1, 2] and groups[18] == [35, 36]


def test_caller_chosen_group_sizes():
    # the uniform rule written out as sizes gives the uniform partition; an uneven list is a partition of
    # 0..n-1 into consecutive runs of exactly those lengths; bad lists are refused
    assert O.build_groups(10, 3, sizes=(3, 3, 3, 1)) == O.build_groups(10, 3)
    assert O.build_groups(38, 2, 1, sizes=(1,) + (2,) * 18 + (1,)) == O.build_groups(38, 2, 1)
    g = O.build_groups(7, 1, sizes=(2, 1, 4))
    assert g == [[0, 1], [2], [3, 4, 5, 6]]
    assert sorted(u for grp in g for u in grp) == list(range(7))
    for bad in [(2, 1, 3), (2, 0, 5), (8,)]:
        with pytest.raises(ValueError):
            O.build_groups(7, 1, sizes=bad)


def test_orders():
    k = 20
    assert O.group_order(k, 0) == list(range(k))
    assert O.group_order(k, 1) == list(range(k))[::-1]
    r1 = O.group_order(k, 2, seed=2401)
    r2 = O.group_order(k, 2, seed=2401)
    assert r1 == r2 and sorted(r1) == list(range(k)) and r1 != list(range(k))
    assert O.group_order(k, 2, seed=7) != r1


def test_splitmix64_published_vector():
    # first outputs of SplitMix64 seeded with 1234567 (reference vector of the
    # public-domain implementation by S. Vigna)
    s = 1234567
    outs = []
    for _ in range(3):
        s, z = O.splitmix64(s)
        outs.append(z)
    assert outs == [6457827717110365317, 3203168211198807973, 9817491932198370423]


def test_queue_walk_equals_fixed_partition_when_m_divides_n():
    # Algorithm 1 c-d: pop m from the head, push to the tail.
    for n, m in [(6, 1), (6, 2), (6, 3), (34, 1), (34, 2), (12, 4)]:
        for order in (0, 1):
            groups = O.build_groups(n, m)
            seq = O.group_order(len(groups), order)
            walk = O.queue_walk(n, m, order, 3 * len(groups))
            for t, e in enumerate(walk):
                assert sorted(e) == groups[seq[t % len(groups)]]


def test_random_order_fixed_across_cycles_and_active_sequence():
    cfg, gc, oc = synth.config_tiny_fp32()
    gc = synth.GroupCfg(layers_per_group=1, order=2, order_seed=5)
    orc = O.HiFTOracle(cfg, gc, oc, synth.init_params(cfg, 0))
    perm = O.group_order(6, 2, 5)
    seq = []
    for t in range(18):
        seq.append(orc.active_group())
        orc.t += 1
    assert seq == perm * 3


def test_delayed_lr_constant_within_cycle():
    # last branch of Algorithm 1: the schedule moves only after all groups were updated
    k, C, lr0 = 14, 3, 2e-5
    lrs = [O.lr_for_cycle(lr0, 1, t // k, C) for t in range(k * C)]
    for c in range(C):
        chunk = lrs[c * k:(c + 1) * k]
        assert len(set(chunk)) == 1
    assert lrs[0] == lr0
    assert lrs[k] == pytest.approx(lr0 * 2 / 3, rel=1e-15)
    assert lrs[2 * k] == pytest.approx(lr0 / 3, rel=1e-15)
    assert all(O.lr_for_cycle(lr0, 0, c, C) == lr0 for c in range(5))
    assert O.lr_for_cycle(lr0, 1, 7, 3) == 0.0


def test_linear_schedule_with_warmup_in_cycles():
    # warm-up of the paper's hyper-parameter tables, counted in cycles (the rate moves once per cycle):
    # values by hand for C = 10, W = 2; W = 0 is the plain linear decay; the ramp meets the decay at lr0
    lr0, C, W = 1e-3, 10, 2
    got = [O.lr_for_cycle(lr0, 1, c, C, W) for c in range(12)]
    want = [0.0, 0.5e-3, 1e-3, 0.875e-3, 0.75e-3, 0.625e-3, 0.5e-3, 0.375e-3, 0.25e-3, 0.125e-3, 0.0, 0.0]
    assert got == pytest.approx(want, rel=1e-15, abs=0.0)
    assert max(got) == lr0 and got.index(lr0) == W
    for c in range(12):
        assert O.lr_for_cycle(lr0, 1, c, C, 0) == O.lr_for_cycle(lr0, 1, c, C)
        assert O.lr_for_cycle(lr0, 0, c, C, W) == lr0                      # the constant schedule ignores it
    # still a function of the cycle only: constant inside a cycle of k steps
    k = 6
    orc_lrs = [O.lr_for_cycle(lr0, 1, t // k, C, W) for t in range(k * C)]
    assert all(len(set(orc_lrs[c * k:(c + 1) * k])) == 1 for c in range(C))


def test_memory_model_against_paper():
    g = _golden()
    z1 = g["zeta1_7b_fp32_G"]
    # zeta1 itself: 7e9 parameters * 4 bytes in GiB
    assert 7e9 * 4 / 2**30 == pytest.approx(z1, abs=0.005)
    assert O.zeta_fpft(z1) == pytest.approx(g["zeta_fpft_7b_G"], abs=1e-9)
    zh = O.zeta_hift(z1, 34)
    assert zh == pytest.approx((34 + 3) / 34 * z1, rel=1e-15)
    assert O.zeta_fpft(z1) - zh == pytest.approx((3 * 34 - 3) / 34 * z1, rel=1e-12)
    # The printed worked value does not follow from the printed equations; the
    # oracle follows the equations.  Keep the discrepancy visible:
    assert zh == pytest.approx(28.38, abs=0.005)
    assert abs(zh - g["zeta_hift_printed_G"]) > 2.0
    assert g["zeta_fpft_7b_G"] - g["zeta_hift_printed_G"] == pytest.approx(g["zeta_saving_printed_G"], abs=0.005)
    # k = 1 degenerates to full fine-tuning
    assert O.zeta_hift(z1, 1) == pytest.approx(O.zeta_fpft(z1))


def test_peak_trainable_fraction():
    cfg, gc, _ = synth.config_llama_7b()
    up = synth.count_params(cfg)
    assert sum(up) == 6_738_415_616
    groups = O.build_groups(cfg.n_units, 1)
    frac = O.peak_trainable_fraction(up, groups)
    assert frac == pytest.approx(202_383_360 / 6_738_415_616)
    assert 0.029 < frac < 0.031
    # the paper's own figure for this quantity: 2.44 % at the 13B size (40 blocks, d 5120, SwiGLU 13824,
    # vocabulary 32000, m = 1: the largest group is one block)
    c13 = cfg.scaled(n_blocks=40, d_model=5120, n_heads=40, d_ffn=13824)
    frac13 = O.peak_trainable_fraction(synth.count_params(c13), O.build_groups(c13.n_units, 1))
    assert round(100 * frac13, 2) == _golden()["peak_trainable_fraction_13b_pct"]
    # names listed by the oracle agree with the synthetic tensor catalogue
    for cfgf in (synth.config_tiny_fp32, synth.config_roberta_base, synth.config_gpt2_large, synth.config_llama_7b):
        c = cfgf()[0]
        cat = synth.unit_tensors(c)
        for u in range(c.n_units):
            assert [n for n, _, _ in cat[u]] == O.tensor_names_of_unit(c, u)


# ---------------------------------------------------------------- the literal queue when m does not divide n
def test_drifting_queue_sets_follow_algorithm_1_and_cover_units_evenly():
    """Algorithm 1 c-d with m not dividing n: the sets are what a literal pop-m / append-to-tail walk gives, they
    repeat with period n / gcd(n, m), every unit is trained m / gcd(n, m) times per period, a set may wrap around
    (top and bottom unit together), and the learning-rate cycle stays k = floor(n / m) + 1 steps."""
    import math
    from collections import Counter, deque
    cfg = synth.ModelCfg(arch=0, n_blocks=3, d_model=16, n_heads=2, d_ffn=32, vocab=31, max_pos=8, batch=1, seq=4)
    n = cfg.n_units                                                # 5 units
    p0 = synth.init_params(cfg, 0)
    for m in (2, 3, 4):
        for order in (0, 1, 2):
            gc = synth.GroupCfg(layers_per_group=m, order=order, order_seed=9, literal_queue=1)
            orc = O.HiFTOracle(cfg, gc, synth.OptCfg(kind=2, lr=1e-2, sched=1, total_cycles=4), p0)
            assert orc.drifting and orc.k == n // m + 1 and orc.n_sets == n // math.gcd(n, m)
            # an independent walk with a deque
            q = deque(O.group_order(n, order, 9))
            seen = Counter()
            for t in range(2 * orc.n_sets):
                e = [q.popleft() for _ in range(m)]
                q.extend(e)
                assert orc.groups[t % orc.n_sets] == sorted(e)
                if t < orc.n_sets:
                    seen.update(e)
            assert set(seen.values()) == {m // math.gcd(n, m)} and len(seen) == n
            if order == 0 and m == 2:
                assert orc.groups[2] == [0, 4]                      # the wrap-around set
    # m dividing n: the flag changes nothing
    gc0, gc1 = synth.GroupCfg(layers_per_group=5), synth.GroupCfg(layers_per_group=5, literal_queue=1)
    assert not O.HiFTOracle(cfg, gc1, synth.OptCfg(), p0).drifting
    assert O.HiFTOracle(cfg, gc1, synth.OptCfg(), p0).groups == O.HiFTOracle(cfg, gc0, synth.OptCfg(), p0).groups


def test_drifting_queue_step_moves_only_the_popped_units_and_counts_updates_per_unit():
    cfg = synth.ModelCfg(arch=0, n_blocks=3, d_model=16, n_heads=2, d_ffn=32, vocab=31, max_pos=8, batch=2, seq=6, init_std=0.1)
    gc = synth.GroupCfg(layers_per_group=2, literal_queue=1)
    oc = synth.OptCfg(kind=0, lr=1e-2, sched=1, total_cycles=5)
    orc = O.HiFTOracle(cfg, gc, oc, synth.init_params(cfg, 1, perturb=0.1))
    lrs = []
    for t in range(7):
        units = orc.groups[orc.active_group()]
        before = {k: v.copy() for k, v in orc.master.items()}
        tok, lab = synth.batch_for(cfg, 3, t, "uniform")
        lrs.append(orc.current_lr())
        orc.step(tok, lab)
        for name in orc.master:
            moved = not np.array_equal(orc.master[name], before[name])
            assert moved == (orc.unit_of(name) in units), (t, name)
    # sets: [0,1] [2,3] [0,4] [1,2] [3,4] [0,1] [2,3]: after 7 steps units 0..3 have 3 updates, unit 4 has 2
    assert orc.tau == [3, 3, 3, 3, 2]
    # k = 3: the rate moves after steps 3 and 6
    assert lrs[0] == lrs[1] == lrs[2] and lrs[3] == lrs[4] == lrs[5] and lrs[2] > lrs[3] > lrs[6]
