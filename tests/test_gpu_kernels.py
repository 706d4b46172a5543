"""Per-kernel parity through the C ABI: each kernel against the oracle's fp64 definition of
the same operation, at shapes that span several tiles and a ragged tail, plus edge cases."""
import numpy as np
import pytest

import synth
from gpu_util import U_BF16, U_F32, assert_elem, attention_slack, gemm_slack, rel_l2
from oracle import hift_oracle as O

pytestmark = pytest.mark.gpu


def _t(a, dtype=None):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t if dtype is None else t.to(dtype)


def _bf(a):
    """bf16-rounded fp64 copy of an fp32 array (what the oracle sees of a bf16 operand)."""
    return O.bf16_round(np.asarray(a, dtype=np.float32)).astype(np.float64)


# ------------------------------------------------------------------ optimizer: 1e-6
@pytest.mark.parametrize("kind", [0, 1, 2])
@pytest.mark.parametrize("n", [1, 3, 1000, 4099, (1 << 20) + 5])
def test_fused_optimizer_matches_oracle_1e6(kind, n):
    import torch
    from paper_2401_15207_b200 import opt_step
    master, grad, s0, s1 = synth.flat_optimizer_inputs(n, seed=kind * 100 + 7, warm=True)
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01, momentum=0.9)
    if kind == 1:
        hp.update(lr=1e-2, eps=1e-10)
        s0 = np.abs(s0).astype(np.float32) ** 2            # accumulator is non-negative
    tm, tg, ts0, ts1 = _t(master), _t(grad), _t(s0), _t(s1)
    tp = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    m64, g64, a64, b64 = (x.astype(np.float64) for x in (master, grad, s0, s1))
    for tau in (3, 4):                                      # two consecutive updates, warm state
        opt_step(kind, n, tp, tm, tg, ts0, ts1, tau=tau, **hp)
        if kind == 0:
            m64, a64, b64 = O.adamw_update(m64, g64, a64, b64, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                                           hp["weight_decay"], tau)
        elif kind == 1:
            m64, a64 = O.adagrad_update(m64, g64, a64, hp["lr"], hp["eps"])
        else:
            m64, a64 = O.sgdm_update(m64, g64, a64, hp["lr"], hp["momentum"])
    torch.cuda.synchronize()
    gm = tm.cpu().numpy()
    assert rel_l2(gm, m64) <= 1e-6
    assert rel_l2(ts0.cpu().numpy(), a64) <= 1e-6
    if kind == 0:
        assert rel_l2(ts1.cpu().numpy(), b64) <= 1e-6
    # the update itself (theta_new - theta_old): 1e-4 relative plus the rounding of the fp32
    # value it is stored in (half an ulp of theta per update; the subtraction cancels)
    delta, delta_ref = gm.astype(np.float64) - master, m64 - master
    assert np.linalg.norm(delta - delta_ref) <= 1e-4 * np.linalg.norm(delta_ref) + 2 * 6e-8 * np.linalg.norm(master)
    # the bf16 model copy is the round-to-nearest-even image of the fp32 master, bit for bit
    assert np.array_equal(tp.float().cpu().numpy(), O.bf16_round(gm))


def test_plain_sgd_kernel_needs_no_state():
    import torch
    from paper_2401_15207_b200 import opt_step
    n = 100003
    master, grad, _, _ = synth.flat_optimizer_inputs(n, seed=11)
    tm, tg = _t(master), _t(grad)
    tp = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    opt_step(3, n, tp, tm, tg, None, None, lr=0.5, tau=1)
    ref = O.sgd_update(master.astype(np.float64), grad.astype(np.float64), 0.5)
    assert rel_l2(tm.cpu().numpy(), ref) <= 1e-6
    assert np.array_equal(tp.float().cpu().numpy(), O.bf16_round(tm.cpu().numpy()))


@pytest.mark.parametrize("rows,cols", [(1, 777), (5, 8), (300, 1280), (2050, 96)])
def test_adafactor_tensor_update_matches_oracle(rows, cols):
    import torch
    from paper_2401_15207_b200 import adafactor_step
    rng = np.random.default_rng(rows * 3 + cols)
    shape = (cols,) if rows == 1 else (rows, cols)
    theta = (rng.standard_normal(shape) * 0.02).astype(np.float32)
    n_state = cols if rows == 1 else rows + cols
    tm = _t(theta.reshape(-1))
    ts = torch.zeros(n_state, device="cuda")
    tp = torch.zeros(rows * cols, dtype=torch.bfloat16, device="cuda")
    scratch = torch.empty(2 * rows + 64 * cols + 8, device="cuda")
    th64 = theta.astype(np.float64)
    s0 = np.zeros(shape[0]) if rows > 1 else np.zeros(shape)
    s1 = np.zeros(cols) if rows > 1 else np.zeros(0)
    for tau in (1, 2, 3):
        g = (rng.standard_normal(shape) * 1e-3).astype(np.float32)
        adafactor_step(rows, cols, tp, tm, _t(g.reshape(-1)), ts, scratch, lr=1e-2, eps1=1e-30, weight_decay=0.01, tau=tau)
        th64, s0, s1 = O.adafactor_update(th64, g.astype(np.float64), s0, s1, 1e-2, 1e-30, 0.01, tau)
    torch.cuda.synchronize()
    gm = tm.cpu().numpy().reshape(shape)
    assert rel_l2(gm, th64) <= 1e-6
    st = ts.cpu().numpy()
    if rows > 1:
        assert rel_l2(st[:rows], s0) <= 2e-6 and rel_l2(st[rows:], s1) <= 2e-6
    else:
        assert rel_l2(st, s0) <= 2e-6
    assert np.array_equal(tp.float().cpu().numpy().reshape(shape), O.bf16_round(gm))


def test_fused_optimizer_fp32_params_and_argument_checks():
    import torch
    from paper_2401_15207_b200 import opt_step, HiftError
    n = 777
    master, grad, s0, s1 = synth.flat_optimizer_inputs(n, seed=3)
    tm, tg, ts0, ts1 = _t(master), _t(grad), _t(s0), _t(s1)
    opt_step(0, n, None, tm, tg, ts0, ts1, lr=1e-3, weight_decay=0.01, tau=1)
    ref, _, _ = O.adamw_update(master.astype(np.float64), grad.astype(np.float64), 0.0, 0.0, 1e-3, 0.9, 0.999,
                               1e-8, 0.01, 1)
    assert rel_l2(tm.cpu().numpy(), ref) <= 1e-6
    with pytest.raises(HiftError):
        opt_step(0, n, None, tm, tg, ts0, None, lr=1e-3)         # AdamW needs the second moment
    with pytest.raises(HiftError):
        opt_step(0, n - 1, None, tm[1:], tg, ts0, ts1, lr=1e-3)  # misaligned pointer
    with pytest.raises(HiftError):
        opt_step(5, n, None, tm, tg, ts0, ts1, lr=1e-3)
    opt_step(2, 0, None, tm, tg, ts0, None, lr=1e-3)             # empty input is a no-op


# ------------------------------------------------------------------ linear layers, three forms
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("M,N,K", [(70, 200, 96), (257, 129, 520), (1, 8, 8)])
def test_linear_three_forms(dtype, M, N, K):
    import torch
    from paper_2401_15207_b200 import k_linear
    rng = np.random.default_rng(M + N + K)
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.1).astype(np.float32)
    dy = rng.standard_normal((M, N)).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    res = rng.standard_normal((M, N)).astype(np.float32)
    td = torch.float32 if dtype == 0 else torch.bfloat16
    tol = 2e-6 if dtype == 0 else 6e-3
    u_out = 2 * U_F32 if dtype == 0 else U_BF16
    cvt = (lambda a: a.astype(np.float64)) if dtype == 0 else _bf
    X, W, DY, Bv = cvt(x), cvt(w), cvt(dy), cvt(bias)
    # forward with bias
    y = torch.empty((M, N), dtype=td, device="cuda")
    k_linear(0, dtype, M, N, K, _t(x, td), _t(w, td), y, bias=_t(bias, td))
    ref, slack = X @ W.T + Bv, gemm_slack(X, W.T) + 2 * U_F32 * np.abs(Bv)
    assert rel_l2(y.float().cpu().numpy(), ref) <= tol
    assert_elem(y.float().cpu().numpy(), ref, u_out, slack, "forward")
    # forward into the fp32 residual stream
    y32 = torch.empty((M, N), dtype=torch.float32, device="cuda")
    k_linear(0, dtype, M, N, K, _t(x, td), _t(w, td), y32, bias=_t(bias, td), residual=_t(res))
    assert rel_l2(y32.cpu().numpy(), ref + res) <= 2e-6
    assert_elem(y32.cpu().numpy(), ref + res, 2 * U_F32, slack + 2 * U_F32 * np.abs(res), "forward into the stream")
    # activation gradient
    dx = torch.empty((M, K), dtype=td, device="cuda")
    k_linear(1, dtype, M, N, K, _t(dy, td), _t(w, td), dx)
    assert rel_l2(dx.float().cpu().numpy(), DY @ W) <= tol
    assert_elem(dx.float().cpu().numpy(), DY @ W, u_out, gemm_slack(DY, W), "dX")
    # weight gradient (fp32 out)
    dw = torch.empty((N, K), dtype=torch.float32, device="cuda")
    k_linear(2, dtype, M, N, K, _t(dy, td), _t(x, td), dw)
    assert rel_l2(dw.cpu().numpy(), DY.T @ X) <= 2e-6
    assert_elem(dw.cpu().numpy(), DY.T @ X, 2 * U_F32, gemm_slack(DY.T, X), "dW")


# ------------------------------------------------------------------ attention
@pytest.mark.parametrize("dtype,dh", [(0, 32), (1, 64), (1, 128), (0, 8)])
@pytest.mark.parametrize("causal", [0, 1])
def test_attention_forward_backward(dtype, dh, causal):
    import torch
    from paper_2401_15207_b200 import k_attention_fwd, k_attention_bwd
    B, S, H = 2, 150, 3                                     # S spans tiles of 64/32 with a ragged tail
    d = H * dh
    rng = np.random.default_rng(dh + causal)
    qkv = rng.standard_normal((B * S, 3 * d)).astype(np.float32)
    do = rng.standard_normal((B * S, d)).astype(np.float32)
    td = torch.float32 if dtype == 0 else torch.bfloat16
    cvt = (lambda a: a.astype(np.float64)) if dtype == 0 else _bf
    q, k, v = (cvt(qkv)[:, i * d:(i + 1) * d].reshape(B, S, H, dh) for i in range(3))
    o_ref, p = O.attention_fwd(q, k, v, bool(causal))
    tq = _t(qkv, td)
    o = torch.empty((B * S, d), dtype=td, device="cuda")
    lse = torch.empty((B, H, S), dtype=torch.float32, device="cuda")
    k_attention_fwd(dtype, B, S, H, dh, causal, tq, o, lse)
    tol = 3e-6 if dtype == 0 else 6e-3
    assert rel_l2(o.float().cpu().numpy(), o_ref.reshape(B * S, d)) <= tol
    u = 16 * U_F32 if dtype == 0 else U_BF16
    sl = attention_slack(q, k, v, p, cvt(do).reshape(B, S, H, dh), u=u)
    assert_elem(o.float().cpu().numpy(), o_ref.reshape(B * S, d), u, sl[0].reshape(B * S, d), "o")
    # log-sum-exp against its definition
    s = np.einsum("bshe,bthe->bhst", q, k) / np.sqrt(dh)
    if causal:
        s = np.where(np.triu(np.ones((S, S), dtype=bool), 1), -np.inf, s)
    lse_ref = np.log(np.exp(s - s.max(-1, keepdims=True)).sum(-1)) + s.max(-1)
    assert np.allclose(lse.cpu().numpy(), lse_ref, rtol=1e-5, atol=1e-5)
    # backward: feed the oracle the same (rounded) o the kernel saved
    dqkv = torch.empty((B * S, 3 * d), dtype=td, device="cuda")
    dsum = torch.empty(B * S * H, dtype=torch.float32, device="cuda")
    k_attention_bwd(dtype, B, S, H, dh, causal, tq, o, lse, _t(do, td), dqkv, dsum)
    dq, dk, dv = O.attention_bwd(cvt(do).reshape(B, S, H, dh), q, k, v, p)
    ref = np.concatenate([t.reshape(B * S, d) for t in (dq, dk, dv)], axis=1)
    tolb = 5e-6 if dtype == 0 else 1.2e-2
    got = dqkv.float().cpu().numpy()
    for i in range(3):
        assert rel_l2(got[:, i * d:(i + 1) * d], ref[:, i * d:(i + 1) * d]) <= tolb, i
        assert_elem(got[:, i * d:(i + 1) * d], ref[:, i * d:(i + 1) * d], u, sl[1 + i].reshape(B * S, d), "dq dk dv"[3 * i:3 * i + 2])


@pytest.mark.parametrize("dh", [64, 128])
@pytest.mark.parametrize("B,S,H", [(1, 1, 1), (1, 64, 2), (3, 129, 1), (2, 300, 2), (1, 640, 1), (6, 300, 26)])
@pytest.mark.parametrize("causal", [0, 1])
def test_attention_tensor_core_edge_lengths(dh, B, S, H, causal):
    """bf16 attention on the tensor-core kernels at the degenerate and ragged sequence lengths: a single
    position, exactly one tile, one row past a tile, several tiles with a tail, more tiles than a CTA's
    double buffers; batch entries that share a tile with their neighbour; and more work items than SMs with a
    ragged tail (468 items: every CTA takes several, so an item's output is stored while the next one runs, and
    the last tile of every entry skips rows that belong to its neighbour)."""
    import torch
    from paper_2401_15207_b200 import k_attention_fwd, k_attention_bwd
    d = H * dh
    rng = np.random.default_rng(1000 * dh + 10 * S + causal)
    qkv = rng.standard_normal((B * S, 3 * d)).astype(np.float32)
    do = rng.standard_normal((B * S, d)).astype(np.float32)
    q, k, v = (_bf(qkv)[:, i * d:(i + 1) * d].reshape(B, S, H, dh) for i in range(3))
    o_ref, p = O.attention_fwd(q, k, v, bool(causal))
    tq = _t(qkv, torch.bfloat16)
    o = torch.full((B * S, d), 9.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, H, S), 9.0, dtype=torch.float32, device="cuda")
    k_attention_fwd(1, B, S, H, dh, causal, tq, o, lse)
    assert rel_l2(o.float().cpu().numpy(), o_ref.reshape(B * S, d)) <= 6e-3
    sl = attention_slack(q, k, v, p, _bf(do).reshape(B, S, H, dh))
    assert_elem(o.float().cpu().numpy(), o_ref.reshape(B * S, d), U_BF16, sl[0].reshape(B * S, d), "o")
    dqkv = torch.full((B * S, 3 * d), 9.0, dtype=torch.bfloat16, device="cuda")
    dsum = torch.empty(B * S * H, dtype=torch.float32, device="cuda")
    k_attention_bwd(1, B, S, H, dh, causal, tq, o, lse, _t(do, torch.bfloat16), dqkv, dsum)
    dq, dk, dv = O.attention_bwd(_bf(do).reshape(B, S, H, dh), q, k, v, p)
    ref = np.concatenate([t.reshape(B * S, d) for t in (dq, dk, dv)], axis=1)
    got = dqkv.float().cpu().numpy()
    for i in range(3):
        r = ref[:, i * d:(i + 1) * d]
        if np.linalg.norm(r) == 0.0:                         # S = 1: dq and dk vanish identically
            assert np.abs(got[:, i * d:(i + 1) * d]).max() <= 1e-3
        else:
            assert rel_l2(got[:, i * d:(i + 1) * d], r) <= 1.5e-2, i
        assert_elem(got[:, i * d:(i + 1) * d], r, U_BF16, sl[1 + i].reshape(B * S, d) + 1e-12, "dq dk dv"[3 * i:3 * i + 2])


@pytest.mark.parametrize("dtype,dh,B,S,H", [(1, 128, 6, 300, 26), (1, 64, 5, 200, 32), (0, 32, 2, 75, 3), (1, 16, 2, 130, 2)])
@pytest.mark.parametrize("causal", [0, 1])
def test_attention_with_probability_dropout(dtype, dh, B, S, H, causal):
    """Attention with dropout on the probabilities, kernel by kernel against the oracle with the same mask: the
    tcgen05 kernels at more work items than SMs with ragged tails (sequence lengths that are no multiple of the
    tile or of four, ragged key lengths on top), and the CUDA-core kernels in fp32 and bf16."""
    import torch
    from paper_2401_15207_b200 import k_attention_fwd_drop, k_attention_bwd_drop
    p_drop, seed, site, step = 0.3, 0x5EED_0123_4567, 1003, 17
    d = H * dh
    rng = np.random.default_rng(100 * dh + S + causal)
    qkv = rng.standard_normal((B * S, 3 * d)).astype(np.float32)
    do = rng.standard_normal((B * S, d)).astype(np.float32)
    lens = [S - (7 * b) % (S // 2) for b in range(B)]
    bf = dtype == 1
    cvt = _bf if bf else (lambda a: a.astype(np.float64))
    q, k, v = (cvt(qkv)[:, i * d:(i + 1) * d].reshape(B, S, H, dh) for i in range(3))
    Sp = (S + 3) // 4 * 4
    pm = O.dropout_mask(B * H * S * Sp, p_drop, seed, site, step).reshape(B, H, S, Sp)[..., :S]
    o_ref, p = O.attention_fwd(q, k, v, bool(causal), lens, pm)
    td = torch.bfloat16 if bf else torch.float32
    tq = _t(qkv, td)
    tl = _t(np.asarray(lens, dtype=np.int32))
    o = torch.full((B * S, d), 9.0, dtype=td, device="cuda")
    lse = torch.full((B, H, S), 9.0, dtype=torch.float32, device="cuda")
    k_attention_fwd_drop(dtype, B, S, H, dh, causal, tq, o, lse, p_drop, seed, site, step, key_lens=tl)
    got_o = o.float().cpu().numpy()
    u = U_BF16 if bf else 4 * U_F32
    sl = attention_slack(q, k, v, p * pm, cvt(do).reshape(B, S, H, dh), u)
    assert rel_l2(got_o, o_ref.reshape(B * S, d)) <= (6e-3 if bf else 3e-6)
    assert_elem(got_o, o_ref.reshape(B * S, d), u, sl[0].reshape(B * S, d) * (1.0 / (1.0 - p_drop)) + 1e-12, "o")
    dqkv = torch.full((B * S, 3 * d), 9.0, dtype=td, device="cuda")
    dsum = torch.empty(B * S * H, dtype=torch.float32, device="cuda")
    k_attention_bwd_drop(dtype, B, S, H, dh, causal, tq, o, lse, _t(do, td), dqkv, dsum, p_drop, seed, site, step, key_lens=tl)
    dq, dk, dv = O.attention_bwd(cvt(do).reshape(B, S, H, dh), q, k, v, p, pm)
    ref = np.concatenate([t.reshape(B * S, d) for t in (dq, dk, dv)], axis=1)
    got = dqkv.float().cpu().numpy()
    for i in range(3):
        assert rel_l2(got[:, i * d:(i + 1) * d], ref[:, i * d:(i + 1) * d]) <= (1.5e-2 if bf else 1e-5), i
    # the mask really is the oracle's: without it the output differs by far more than any tolerance
    o2, _ = O.attention_fwd(q, k, v, bool(causal), lens)
    assert rel_l2(got_o, o2.reshape(B * S, d)) > 0.1


@pytest.mark.parametrize("dtype,dh", [(0, 32), (1, 64), (1, 128)])
@pytest.mark.parametrize("causal", [0, 1])
def test_attention_key_lengths(dtype, dh, causal):
    """Right-padded batch entries: keys at or after an entry's length get no weight and no gradient.  Lengths
    of a full row, one past a tile, exactly a tile, a few keys and a single key."""
    import torch
    from paper_2401_15207_b200 import k_attention_fwd, k_attention_bwd
    B, S, H = 5, 300, 2
    lens = [300, 129, 128, 37, 1]
    d = H * dh
    rng = np.random.default_rng(77 + dh + causal)
    qkv = rng.standard_normal((B * S, 3 * d)).astype(np.float32)
    do = rng.standard_normal((B * S, d)).astype(np.float32)
    td = torch.float32 if dtype == 0 else torch.bfloat16
    cvt = (lambda a: a.astype(np.float64)) if dtype == 0 else _bf
    q, k, v = (cvt(qkv)[:, i * d:(i + 1) * d].reshape(B, S, H, dh) for i in range(3))
    o_ref, p = O.attention_fwd(q, k, v, bool(causal), lens)
    tq = _t(qkv, td)
    tl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    o = torch.full((B * S, d), 9.0, dtype=td, device="cuda")
    lse = torch.full((B, H, S), 9.0, dtype=torch.float32, device="cuda")
    k_attention_fwd(dtype, B, S, H, dh, causal, tq, o, lse, key_lens=tl)
    assert rel_l2(o.float().cpu().numpy(), o_ref.reshape(B * S, d)) <= (3e-6 if dtype == 0 else 6e-3)
    u = 16 * U_F32 if dtype == 0 else U_BF16
    sl = attention_slack(q, k, v, p, cvt(do).reshape(B, S, H, dh), u=u)
    assert_elem(o.float().cpu().numpy(), o_ref.reshape(B * S, d), u, sl[0].reshape(B * S, d), "o")
    dqkv = torch.full((B * S, 3 * d), 9.0, dtype=td, device="cuda")
    dsum = torch.empty(B * S * H, dtype=torch.float32, device="cuda")
    k_attention_bwd(dtype, B, S, H, dh, causal, tq, o, lse, _t(do, td), dqkv, dsum, key_lens=tl)
    dq, dk, dv = O.attention_bwd(cvt(do).reshape(B, S, H, dh), q, k, v, p)
    ref = np.concatenate([t.reshape(B * S, d) for t in (dq, dk, dv)], axis=1)
    got = dqkv.float().cpu().numpy()
    tolb = 5e-6 if dtype == 0 else 1.5e-2
    for i in range(3):
        assert rel_l2(got[:, i * d:(i + 1) * d], ref[:, i * d:(i + 1) * d]) <= tolb, i
        assert_elem(got[:, i * d:(i + 1) * d], ref[:, i * d:(i + 1) * d], u, sl[1 + i].reshape(B * S, d), "dq dk dv"[3 * i:3 * i + 2])
    g4 = got.reshape(B, S, 3, d)
    for b, l in enumerate(lens):
        assert np.all(g4[b, l:, 1:] == 0.0), b                # dk, dv of padded keys: exact zeros
    # the full-length table is the same computation as no table
    o2 = torch.empty_like(o)
    lse2 = torch.empty_like(lse)
    k_attention_fwd(dtype, B, S, H, dh, causal, tq, o2, lse2)
    k_attention_fwd(dtype, B, S, H, dh, causal, tq, o, lse, key_lens=torch.full((B,), S, dtype=torch.int32, device="cuda"))
    assert torch.equal(o, o2) and torch.equal(lse, lse2)


@pytest.mark.parametrize("dh", [64, 128])
@pytest.mark.parametrize("causal", [0, 1])
def test_attention_key_lengths_on_the_warp_level_kernels(dh, causal):
    """The same cases with the tcgen05 attention switched off: the mma.sync kernels behind it."""
    from paper_2401_15207_b200 import code_path_switch
    old = code_path_switch(2, 0), code_path_switch(3, 0)
    try:
        test_attention_key_lengths(1, dh, causal)
    finally:
        code_path_switch(2, old[0])
        code_path_switch(3, old[1])


# ------------------------------------------------------------------ rotary embedding fused into the qkv projection
def _rope_cs(S, dh, base=10000.0):
    cos, sin = O.rope_tables(S, dh, base)
    return np.concatenate([cos.reshape(-1), sin.reshape(-1)]).astype(np.float32), cos, sin


@pytest.mark.parametrize("M,N,K,rope_cols,bias", [(300, 768, 256, 512, False), (256, 640, 192, 640, True)])
def test_linear_with_rope_in_the_epilogue(M, N, K, rope_cols, bias):
    """qkv projection whose q and k column blocks leave the GEMM already rotated (head size 128):
    against linear -> RoPE of the oracle on the same bf16 operands.  Rows are positions r mod S with
    S = 100, so the tile's 128 rows span a wrap of the position."""
    import torch
    from paper_2401_15207_b200 import k_linear_rope
    dh, S = 128, 100
    rng = np.random.default_rng(M + N)
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32)
    b = (0.5 * rng.standard_normal(N)).astype(np.float32)
    cs, cos, sin = _rope_cs(S, dh)
    out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    tb = _t(b, torch.bfloat16) if bias else None
    k_linear_rope(M, N, K, _t(x, torch.bfloat16), _t(w, torch.bfloat16), out, tb, _t(cs), S, dh, rope_cols)
    y = _bf(x) @ _bf(w).T + (_bf(b) if bias else 0.0)
    pos = np.arange(M) % S
    ref = y.copy()
    heads = y[:, :rope_cols].reshape(1, M, rope_cols // dh, dh)      # rows play the sequence axis, each with its own angle
    ref[:, :rope_cols] = O.rope_apply(heads, cos[pos], sin[pos]).reshape(M, rope_cols)
    got = out.float().cpu().numpy()
    assert rel_l2(got[:, :rope_cols], ref[:, :rope_cols]) <= 4e-3
    assert rel_l2(got[:, rope_cols:], ref[:, rope_cols:]) <= 4e-3 or rope_cols == N
    # a rotated element mixes two accumulators with |cos|, |sin| <= 1 (fp32 tables: 2^-24 each)
    acc = gemm_slack(_bf(x), _bf(w).T) + 4 * U_F32 * np.abs(y)
    part = acc[:, :rope_cols].reshape(M, rope_cols // dh, 2, dh // 2)
    mixed = (part + part[:, :, ::-1, :]).reshape(M, rope_cols)
    ymix = np.abs(y[:, :rope_cols]).reshape(M, rope_cols // dh, 2, dh // 2)
    mixed = mixed + 4 * U_F32 * (ymix + ymix[:, :, ::-1, :]).reshape(M, rope_cols)
    assert_elem(got[:, :rope_cols], ref[:, :rope_cols], U_BF16, mixed, "rotated columns")
    if rope_cols < N:
        assert_elem(got[:, rope_cols:], ref[:, rope_cols:], U_BF16, acc[:, rope_cols:], "plain columns")


@pytest.mark.parametrize("M,f,K,keep,bias", [(300, 384, 256, True, False), (256, 128, 192, False, True), (520, 1152, 128, True, True)])
def test_gate_up_projection_with_swiglu_in_the_epilogue(M, f, K, keep, bias):
    """Gate | up GEMM whose epilogue stores silu(gate) * up (and the pre-activations when kept):
    against linear -> swiglu of the oracle on the same bf16 operands."""
    import torch
    from paper_2401_15207_b200 import k_linear_swiglu
    rng = np.random.default_rng(M + f)
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((2 * f, K)) * (2.0 / np.sqrt(K))).astype(np.float32)
    b = (0.5 * rng.standard_normal(2 * f)).astype(np.float32)
    gu = torch.full((M, 2 * f), 7.0, dtype=torch.bfloat16, device="cuda") if keep else None
    s = torch.empty((M, f), dtype=torch.bfloat16, device="cuda")
    k_linear_swiglu(M, f, K, _t(x, torch.bfloat16), _t(w, torch.bfloat16), gu, s, _t(b, torch.bfloat16) if bias else None)
    y = _bf(x) @ _bf(w).T + (_bf(b) if bias else 0.0)
    s_ref = O.swiglu_fwd(y[:, :f], y[:, f:])
    assert rel_l2(s.float().cpu().numpy(), s_ref) <= 4e-3
    acc = gemm_slack(_bf(x), _bf(w).T) + (2 * U_F32 * np.abs(_bf(b)) if bias else 0.0)
    # d(silu(g) u)/dg and /du from the oracle's own backward with a unit upstream gradient; the logistic function
    # comes from the hardware exp2 and reciprocal (a few fp32 units, relative to the value)
    dg1, du1 = O.swiglu_bwd(np.ones_like(s_ref), y[:, :f], y[:, f:])
    assert_elem(s.float().cpu().numpy(), s_ref, U_BF16 + 8 * U_F32,
                np.abs(dg1) * acc[:, :f] + np.abs(du1) * acc[:, f:], "silu(gate) * up")
    if keep:
        assert rel_l2(gu.float().cpu().numpy(), y) <= 4e-3
        assert_elem(gu.float().cpu().numpy(), y, U_BF16, acc, "kept pre-activations")


@pytest.mark.parametrize("M,N,f", [(300, 256, 416), (256, 128, 1024), (200, 192, 96)])
def test_down_projection_dx_with_swiglu_backward_in_the_epilogue(M, N, f):
    """ds = dy W_down and the activation's backward in one kernel: against linear dX -> swiglu_bwd of the
    oracle on the same bf16 operands (f spans several tiles with a ragged last one)."""
    import torch
    from paper_2401_15207_b200 import k_linear_dx_swiglu_bwd
    rng = np.random.default_rng(M + f)
    dy = rng.standard_normal((M, N)).astype(np.float32)
    w = (rng.standard_normal((N, f)) / np.sqrt(N)).astype(np.float32)
    gu = (1.5 * rng.standard_normal((M, 2 * f))).astype(np.float32)
    dgu = torch.empty((M, 2 * f), dtype=torch.bfloat16, device="cuda")
    k_linear_dx_swiglu_bwd(M, N, f, _t(dy, torch.bfloat16), _t(w, torch.bfloat16), _t(gu, torch.bfloat16), dgu)
    ds = _bf(dy) @ _bf(w)
    dg_ref, du_ref = O.swiglu_bwd(ds, _bf(gu)[:, :f], _bf(gu)[:, f:])
    got = dgu.float().cpu().numpy()
    assert rel_l2(got[:, :f], dg_ref) <= 4e-3
    assert rel_l2(got[:, f:], du_ref) <= 4e-3
    # both outputs are ds times a factor that depends on the saved pre-activations only
    acc = gemm_slack(_bf(dy), _bf(w))
    fg, fu = O.swiglu_bwd(np.ones_like(ds), _bf(gu)[:, :f], _bf(gu)[:, f:])
    assert_elem(got[:, :f], dg_ref, U_BF16 + 16 * U_F32, np.abs(fg) * acc, "d gate")
    assert_elem(got[:, f:], du_ref, U_BF16 + 16 * U_F32, np.abs(fu) * acc, "d up")


@pytest.mark.parametrize("M,N,K,keep,bias", [(300, 416, 256, True, True), (256, 1024, 192, False, False)])
def test_up_projection_with_gelu_in_the_epilogue(M, N, K, keep, bias):
    import torch
    from paper_2401_15207_b200 import k_linear_gelu
    rng = np.random.default_rng(M + N)
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * (2.0 / np.sqrt(K))).astype(np.float32)
    b = (0.5 * rng.standard_normal(N)).astype(np.float32)
    pre = torch.full((M, N), 7.0, dtype=torch.bfloat16, device="cuda") if keep else None
    act = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    k_linear_gelu(M, N, K, _t(x, torch.bfloat16), _t(w, torch.bfloat16), pre, act, _t(b, torch.bfloat16) if bias else None)
    y = _bf(x) @ _bf(w).T + (_bf(b) if bias else 0.0)
    assert rel_l2(act.float().cpu().numpy(), O.gelu_fwd(y)) <= 4e-3
    acc = gemm_slack(_bf(x), _bf(w).T) + (2 * U_F32 * np.abs(_bf(b)) if bias else 0.0)
    # the epilogue's normal CDF: 3e-7 absolute (times |y|), at most 0.4 % relative in the far tail
    assert_elem(act.float().cpu().numpy(), O.gelu_fwd(y), U_BF16 + 4e-3,
                np.abs(O.gelu_bwd(np.ones_like(y), y)) * acc + 3e-7 * np.abs(y), "gelu")
    if keep:
        assert rel_l2(pre.float().cpu().numpy(), y) <= 4e-3
        assert_elem(pre.float().cpu().numpy(), y, U_BF16, acc, "kept pre-activation")


@pytest.mark.parametrize("M,N,f", [(300, 256, 416), (200, 192, 96)])
def test_down_projection_dx_with_gelu_backward_in_the_epilogue(M, N, f):
    import torch
    from paper_2401_15207_b200 import k_linear_dx_gelu_bwd
    rng = np.random.default_rng(M + f)
    dy = rng.standard_normal((M, N)).astype(np.float32)
    w = (rng.standard_normal((N, f)) / np.sqrt(N)).astype(np.float32)
    a = (1.5 * rng.standard_normal((M, f))).astype(np.float32)
    da = torch.empty((M, f), dtype=torch.bfloat16, device="cuda")
    k_linear_dx_gelu_bwd(M, N, f, _t(dy, torch.bfloat16), _t(w, torch.bfloat16), _t(a, torch.bfloat16), da)
    ref = O.gelu_bwd(_bf(dy) @ _bf(w), _bf(a))
    assert rel_l2(da.float().cpu().numpy(), ref) <= 4e-3
    du = _bf(dy) @ _bf(w)
    fac = np.abs(O.gelu_bwd(np.ones_like(du), _bf(a)))
    # gelu'(a) = Phi(a) + a phi(a): the approximated CDF (3e-7 absolute) plus the density through exp2
    assert_elem(da.float().cpu().numpy(), ref, U_BF16 + 16 * U_F32, fac * gemm_slack(_bf(dy), _bf(w)) + 1e-6 * np.abs(du), "gelu backward")


# ------------------------------------------------------------------ norms
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("kind", [0, 1])
@pytest.mark.parametrize("rows,cols", [(37, 64), (300, 1280), (5, 4096)])
def test_norm_forward_backward(dtype, kind, rows, cols):
    import torch
    from paper_2401_15207_b200 import k_norm_fwd, k_norm_bwd
    rng = np.random.default_rng(rows + cols)
    x = (rng.standard_normal((rows, cols)) * 2 + 0.3).astype(np.float32)
    gain = (1 + 0.1 * rng.standard_normal(cols)).astype(np.float32)
    bias = (0.1 * rng.standard_normal(cols)).astype(np.float32)
    dy = rng.standard_normal((rows, cols)).astype(np.float32)
    add = rng.standard_normal((rows, cols)).astype(np.float32)
    td = torch.float32 if dtype == 0 else torch.bfloat16
    cvt = (lambda a: a.astype(np.float64)) if dtype == 0 else _bf
    eps = 1e-5 if kind == 0 else 1e-6
    y = torch.empty((rows, cols), dtype=td, device="cuda")
    stats = torch.empty(2 * rows, dtype=torch.float32, device="cuda")
    tx, tg, tb = _t(x), _t(gain, td), _t(bias, td)
    k_norm_fwd(dtype, kind, rows, cols, eps, tx, tg, tb if kind == 0 else None, y, stats)
    x64 = x.astype(np.float64)
    if kind == 0:
        y_ref, cache = O.layernorm_fwd(x64, cvt(gain), cvt(bias), eps)
    else:
        y_ref, cache = O.rmsnorm_fwd(x64, cvt(gain), eps)
    assert rel_l2(y.float().cpu().numpy(), y_ref) <= (2e-6 if dtype == 0 else 4e-3)
    # statistics in fp32 over `cols` elements: a few units of the row's scale
    xs = np.abs(x64).max(axis=1, keepdims=True) * np.asarray(cache[1]).reshape(-1, 1)
    assert_elem(y.float().cpu().numpy(), y_ref, (U_BF16 if dtype else 0.0) + 8 * U_F32,
                8 * U_F32 * (xs * np.abs(cvt(gain)) + (np.abs(cvt(bias)) if kind == 0 else 0.0)), "norm forward")
    dx = torch.empty((rows, cols), dtype=torch.float32, device="cuda")
    dgain = torch.empty(cols, dtype=torch.float32, device="cuda")
    dbias = torch.empty(cols, dtype=torch.float32, device="cuda")
    partial = torch.empty(2 * 64 * cols, dtype=torch.float32, device="cuda")
    k_norm_bwd(dtype, kind, rows, cols, _t(dy, td), tx, stats, tg, _t(add), dx, dgain,
               dbias if kind == 0 else None, partial)
    if kind == 0:
        dx_ref, dg_ref, db_ref = O.layernorm_bwd(cvt(dy), cache, cvt(gain))
        assert rel_l2(dbias.cpu().numpy(), db_ref) <= 3e-6
    else:
        dx_ref, dg_ref = O.rmsnorm_bwd(cvt(dy), cache, cvt(gain))
    assert rel_l2(dx.cpu().numpy(), dx_ref + add) <= 3e-6
    assert rel_l2(dgain.cpu().numpy(), dg_ref) <= 5e-6
    # every term of dx is rstd * (gain dy) times a factor of at most 1 + |xhat|^2: bound per row
    gdy = np.abs(cvt(dy) * cvt(gain))
    rstd = np.asarray(cache[1]).reshape(-1, 1)                 # both norms keep (xhat or x, 1 / sigma)
    xhat = np.abs(cache[0]) if kind == 0 else np.abs(cache[0] * cache[1])
    rowscale = rstd * (gdy + gdy.mean(axis=1, keepdims=True) * (1.0 + xhat) + (gdy * xhat).mean(axis=1, keepdims=True) * xhat)
    assert_elem(dx.cpu().numpy(), dx_ref + add, 2 * U_F32, 32 * U_F32 * rowscale + 2 * U_F32 * np.abs(add), "norm dx")
    colscale = (np.abs(cvt(dy)) * xhat).sum(axis=0)
    assert_elem(dgain.cpu().numpy(), dg_ref, 2 * U_F32, 64 * U_F32 * colscale, "d gain")
    if kind == 0:
        assert_elem(dbias.cpu().numpy(), db_ref, 2 * U_F32, 64 * U_F32 * np.abs(cvt(dy)).sum(axis=0), "d bias")


# ------------------------------------------------------------------ cross-entropy
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("rows,vocab,ld", [(64, 512, 512), (33, 50257, 50304), (16, 2, 2)])
def test_cross_entropy(dtype, rows, vocab, ld):
    import torch
    from paper_2401_15207_b200 import k_cross_entropy
    rng = np.random.default_rng(vocab)
    logits = (rng.standard_normal((rows, ld)) * 3).astype(np.float32)
    labels = rng.integers(0, vocab, rows).astype(np.int32)
    if rows > 8:
        labels[3] = -1                                       # an ignored row
    td = torch.float32 if dtype == 0 else torch.bfloat16
    cvt = (lambda a: a.astype(np.float64)) if dtype == 0 else _bf
    tl = _t(logits, td)
    rowloss = torch.empty(rows, dtype=torch.float32, device="cuda")
    out = torch.zeros(4, dtype=torch.float32, device="cuda")
    k_cross_entropy(dtype, rows, vocab, ld, tl, _t(labels), rowloss, out)
    loss_ref, d_ref = O.cross_entropy(cvt(logits)[:, :vocab], labels)
    o = out.cpu().numpy()
    assert abs(o[0] - loss_ref) <= 2e-6 * abs(loss_ref)
    assert o[1:3].view(np.int32).tolist() == [int((labels >= 0).sum()), 0]
    got = tl.float().cpu().numpy()
    assert rel_l2(got[:, :vocab], d_ref) <= (3e-6 if dtype == 0 else 4e-3)
    # softmax in fp32: the exponent's argument (|logit| up to ~15) and the row sum carry a few units each
    nv = max(int((labels >= 0).sum()), 1)
    p_ref = np.abs(d_ref) + (np.abs(d_ref) > 0.5 / nv) * (1.0 / nv)      # the probability itself, also at the label
    assert_elem(got[:, :vocab], d_ref, (U_BF16 if dtype else 0.0) + 4 * U_F32, 64 * U_F32 * p_ref, "d logits")
    assert not got[:, vocab:].any()                          # padding columns carry no gradient
    if rows > 8:
        assert not got[3].any()


def test_cross_entropy_flags_bad_label():
    import torch
    from paper_2401_15207_b200 import k_cross_entropy
    logits = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
    labels = _t(np.array([1, 9, 2, 3], dtype=np.int32))     # 9 >= vocab
    out = torch.zeros(4, dtype=torch.float32, device="cuda")
    k_cross_entropy(0, 4, 8, 8, logits, labels, torch.empty(4, device="cuda"), out)
    assert out.cpu().numpy()[2:3].view(np.int32)[0] == 1


# ------------------------------------------------------------------ tensor-core GEMM (tcgen05), forced
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (256, 512, 640), (300, 328, 200), (1024, 128, 1096),
                                   (130, 72, 72)])
def test_linear_tensor_core_three_forms(M, N, K):
    import torch
    from paper_2401_15207_b200 import k_linear
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.1).astype(np.float32)
    dy = rng.standard_normal((M, N)).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    bf = torch.bfloat16
    tx, tw, tdy, tb = _t(x, bf), _t(w, bf), _t(dy, bf), _t(bias, bf)
    # forward, bf16 out with bias
    y = torch.zeros((M, N), dtype=bf, device="cuda")
    k_linear(0, 1, M, N, K, tx, tw, y, bias=tb, path=2)
    ref = _bf(x) @ _bf(w).T + _bf(bias)
    slack = gemm_slack(_bf(x), _bf(w).T) + 2 * U_F32 * np.abs(_bf(bias))
    assert rel_l2(y.float().cpu().numpy(), ref) <= 6e-3
    assert_elem(y.float().cpu().numpy(), ref, U_BF16, slack, "forward")
    # forward into the fp32 residual stream
    res = rng.standard_normal((M, N)).astype(np.float32)
    y32 = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    k_linear(0, 1, M, N, K, tx, tw, y32, bias=tb, residual=_t(res), path=2)
    assert rel_l2(y32.cpu().numpy(), ref + res) <= 1e-5
    assert_elem(y32.cpu().numpy(), ref + res, 2 * U_F32, slack + 2 * U_F32 * np.abs(res), "forward into the stream")
    # activation gradient: dx[M,K] = dy[M,N] w[N,K]   (B operand N-major)
    if K >= 64 and N >= 64:
        dx = torch.zeros((M, K), dtype=torch.float32, device="cuda")
        k_linear(1, 1, M, N, K, tdy, tw, dx, residual=torch.zeros((M, K), dtype=torch.float32, device="cuda"), path=2)
        assert rel_l2(dx.cpu().numpy(), _bf(dy) @ _bf(w)) <= 1e-5
        assert_elem(dx.cpu().numpy(), _bf(dy) @ _bf(w), 2 * U_F32, gemm_slack(_bf(dy), _bf(w)), "dX")
    # weight gradient: dw[N,K] = dy^T x   (both operands MN-major); needs N >= 128 rows of output
    if N >= 128:
        dw = torch.zeros((N, K), dtype=torch.float32, device="cuda")
        k_linear(2, 1, M, N, K, tdy, tx, dw, path=2)
        assert rel_l2(dw.cpu().numpy(), _bf(dy).T @ _bf(x)) <= 1e-5
        assert_elem(dw.cpu().numpy(), _bf(dy).T @ _bf(x), 2 * U_F32, gemm_slack(_bf(dy).T, _bf(x)), "dW")


def test_tensor_core_path_refuses_ineligible_shapes():
    import torch
    from paper_2401_15207_b200 import k_linear, HiftError
    bf = torch.bfloat16
    a = torch.zeros((64, 64), dtype=bf, device="cuda")
    with pytest.raises(HiftError):
        k_linear(0, 1, 64, 64, 64, a, a, torch.zeros((64, 64), dtype=bf, device="cuda"), path=2)   # M < 128
    a = torch.zeros((128, 100), dtype=bf, device="cuda")
    w = torch.zeros((64, 100), dtype=bf, device="cuda")
    with pytest.raises(HiftError):
        k_linear(0, 1, 128, 64, 100, a, w, torch.zeros((128, 64), dtype=bf, device="cuda"), path=2)  # ld % 8 != 0
