"""The element-wise bounds the GPU parity tests use (tests/gpu_util.py), exercised on the CPU: a correctly
rounded result passes, and the mistakes a whole-tensor norm hides - one wrong element, one ragged last row
computed from the wrong row, one dropped block of the reduction - are caught."""
import numpy as np
import pytest

from gpu_util import U_BF16, U_F32, assert_elem, attention_slack, gemm_slack, rel_l2, tile_rows
from oracle import hift_oracle as O


def _problem(M=300, N=1280, K=640, seed=0):
    rng = np.random.default_rng(seed)
    A = O.bf16_round(rng.standard_normal((M, K)).astype(np.float32)).astype(np.float64)
    B = O.bf16_round((rng.standard_normal((K, N)) * 0.05).astype(np.float32)).astype(np.float64)
    ref = A @ B
    # what a correct kernel returns: fp32 accumulation (here: the fp64 product rounded to fp32), then one bf16 store
    good = O.bf16_round(ref.astype(np.float32)).astype(np.float64)
    return A, B, ref, good


def test_a_correctly_rounded_product_passes():
    A, B, ref, good = _problem()
    assert_elem(good, ref, U_BF16, gemm_slack(A, B))
    assert_elem(ref.astype(np.float32), ref, 2 * U_F32, gemm_slack(A, B))


def test_one_wrong_element_is_caught_where_the_norm_passes():
    A, B, ref, good = _problem()
    bad = good.copy()
    bad[299, 1279] = good[298, 1279]                      # last row, last column: a neighbour's value
    assert rel_l2(bad, ref) <= 6e-3                       # the tolerance the norm-based comparison allows
    with pytest.raises(AssertionError):
        assert_elem(bad, ref, U_BF16, gemm_slack(A, B))


def test_a_dropped_tail_of_the_reduction_in_one_row_is_caught():
    A, B, ref, good = _problem()
    bad = good.copy()
    bad[128] = O.bf16_round((A[128, :-4] @ B[:-4]).astype(np.float32))        # one row missing the last 4 of its 640 products
    assert rel_l2(bad, ref) <= 6e-3
    with pytest.raises(AssertionError):
        assert_elem(bad, ref, U_BF16, gemm_slack(A, B))


def test_half_an_ulp_too_much_is_caught():
    A, B, ref, good = _problem(M=64, N=64, K=64)
    i = np.unravel_index(np.argmax(np.abs(ref)), ref.shape)
    bad = good.copy()
    bad[i] = good[i] * (1 + 3 * U_BF16)                   # one and a half units in the last place off
    with pytest.raises(AssertionError):
        assert_elem(bad, ref, U_BF16, gemm_slack(A, B))


def test_tile_rows_cover_every_tile_and_the_edges():
    for M in (1, 127, 128, 129, 2048, 4096, 22016, 32000, 50257):
        r = tile_rows(M)
        assert r[0] == 0 and r[-1] == M - 1 and len(set(r.tolist())) == len(r)
        assert set(r // 128) == set(range((M + 127) // 128))
        if M > 128:
            assert 127 in r and 128 in r


def test_attention_bounds_accept_bf16_probabilities_and_catch_a_wrong_key():
    rng = np.random.default_rng(3)
    B, S, H, dh = 1, 70, 2, 16
    q, k, v, do = (O.bf16_round(rng.standard_normal((B, S, H, dh)).astype(np.float32)).astype(np.float64) for _ in range(4))
    o, p = O.attention_fwd(q, k, v, True)
    s_o, s_dq, s_dk, s_dv = attention_slack(q, k, v, p, do)
    # a kernel that rounds P to bf16 before the second product, and its output to bf16
    p16 = O.bf16_round(p.astype(np.float32)).astype(np.float64)
    o16 = O.bf16_round(np.matmul(p16, v.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3).astype(np.float32)).astype(np.float64)
    assert_elem(o16, o, U_BF16, s_o)
    # the same with the causal mask off by one for a single query row (it also sees the next key)
    p_bad = p.copy()
    row = 40
    sc = np.einsum("he,hte->ht", q[0, row], k[0, :row + 2].transpose(1, 0, 2)) / np.sqrt(dh)
    e = np.exp(sc - sc.max(-1, keepdims=True))
    p_bad[0, :, row, :row + 2] = e / e.sum(-1, keepdims=True)
    o_bad = np.matmul(p_bad, v.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3)
    assert rel_l2(o_bad, o) <= 6e-2
    with pytest.raises(AssertionError):
        assert_elem(o_bad, o, U_BF16, s_o)
    # gradients: exact values pass their bounds trivially; the bounds are finite and non-negative
    dq, dk, dv = O.attention_bwd(do, q, k, v, p)
    for g, s in ((dq, s_dq), (dk, s_dk), (dv, s_dv)):
        assert np.all(s >= 0) and np.isfinite(s).all()
        assert_elem(g, g, U_BF16, s)
        assert np.median(s) < 0.1 * np.abs(g).mean()      # and they are small against the values they guard
