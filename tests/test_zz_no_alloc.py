"""The allocation-free norm-backward entry point.

Some users of this library cannot allocate device memory at the point where they call it: the
call sits inside a memory pool that is already fully handed out, or in a loop that cannot take
the implicit synchronisation of cudaMalloc/cudaFree, or in a process that only borrows buffers.
hift_k_norm_bwd_static serves them: it keeps its reduction scratch in an array built into the
library and allocates nothing.  This test checks it against hift_k_norm_bwd (which takes the
scratch from the caller) on two calls in a row; the second call uses narrower rows so that it
runs over whatever the first one left in the shared array.  Both entry points launch the same
kernels with the same summation order, so their results must agree bit for bit; one case is also
held against the CPU oracle's definition of the norm's backward pass.

The file name sorts last on purpose: if this test fails in a run that stops at the first
failure, every other test has already run.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _case(dtype, kind, rows, cols, seed, against_oracle=False):
    import torch
    from paper_2401_15207_b200 import k_norm_fwd, k_norm_bwd, k_norm_bwd_static
    rng = np.random.default_rng(seed)
    td = torch.float32 if dtype == 0 else torch.bfloat16
    x = torch.from_numpy((rng.standard_normal((rows, cols)) * 2 + 0.3).astype(np.float32)).cuda()
    gain = torch.from_numpy((1 + 0.1 * rng.standard_normal(cols)).astype(np.float32)).cuda().to(td)
    bias = torch.from_numpy((0.1 * rng.standard_normal(cols)).astype(np.float32)).cuda().to(td)
    dy = torch.from_numpy(rng.standard_normal((rows, cols)).astype(np.float32)).cuda().to(td)
    add = torch.from_numpy(rng.standard_normal((rows, cols)).astype(np.float32)).cuda()
    y = torch.empty((rows, cols), dtype=td, device="cuda")
    stats = torch.empty(2 * rows, dtype=torch.float32, device="cuda")
    k_norm_fwd(dtype, kind, rows, cols, 1e-5, x, gain, bias if kind == 0 else None, y, stats)
    outs = []
    for static in (False, True):
        dx = torch.full((rows, cols), float("nan"), dtype=torch.float32, device="cuda")
        dgain = torch.full((cols,), float("nan"), dtype=torch.float32, device="cuda")
        dbias = torch.full((cols,), float("nan"), dtype=torch.float32, device="cuda")
        db = dbias if kind == 0 else None
        if static:
            k_norm_bwd_static(dtype, kind, rows, cols, dy, x, stats, gain, add, dx, dgain, db)
        else:
            partial = torch.empty(2 * 64 * cols, dtype=torch.float32, device="cuda")
            k_norm_bwd(dtype, kind, rows, cols, dy, x, stats, gain, add, dx, dgain, db, partial)
        torch.cuda.synchronize()
        outs.append((dx.cpu().numpy(), dgain.cpu().numpy(), dbias.cpu().numpy() if kind == 0 else None))
    (dx0, dg0, db0), (dx1, dg1, db1) = outs
    assert np.isfinite(dx1).all() and np.isfinite(dg1).all()
    # same kernels and the same summation order: the same bits
    assert np.array_equal(dx1, dx0) and np.array_equal(dg1, dg0)
    if kind == 0:
        assert np.isfinite(db1).all() and np.array_equal(db1, db0)
    if against_oracle:
        from oracle import hift_oracle as O
        f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
        if kind == 0:
            _, cache = O.layernorm_fwd(f64(x), f64(gain), f64(bias), 1e-5)
            dx_ref, dg_ref, db_ref = O.layernorm_bwd(f64(dy), cache, f64(gain))
            assert np.linalg.norm(db1 - db_ref) <= 3e-6 * np.linalg.norm(db_ref)
        else:
            _, cache = O.rmsnorm_fwd(f64(x), f64(gain), 1e-5)
            dx_ref, dg_ref = O.rmsnorm_bwd(f64(dy), cache, f64(gain))
        dx_ref = dx_ref + f64(add)
        assert np.linalg.norm(dx1 - dx_ref) <= 3e-6 * np.linalg.norm(dx_ref)      # the norm tests' tolerances
        assert np.linalg.norm(dg1 - dg_ref) <= 5e-6 * np.linalg.norm(dg_ref)


def test_static_scratch_norm_backward_matches_on_two_calls_in_a_row():
    _case(1, 0, 300, 4096, seed=1)       # first call: wide rows, fills much of the shared array
    _case(1, 0, 37, 64, seed=2, against_oracle=True)     # second call: runs over the first call's leftovers
    _case(0, 1, 130, 1280, seed=3, against_oracle=True)  # RMSNorm, fp32 operands
    _case(1, 1, 65, 8192, seed=4)        # exactly the built-in capacity


def test_static_scratch_rejects_rows_wider_than_its_capacity():
    import torch
    from paper_2401_15207_b200 import k_norm_bwd_static, HiftError
    from paper_2401_15207_b200.binding import STATIC_SCRATCH_MAX_COLS
    cols = STATIC_SCRATCH_MAX_COLS + 8
    z = torch.zeros((2, cols), dtype=torch.float32, device="cuda")
    g = torch.ones(cols, dtype=torch.float32, device="cuda")
    st = torch.ones(4, dtype=torch.float32, device="cuda")
    out = torch.zeros(cols, dtype=torch.float32, device="cuda")
    with pytest.raises(HiftError) as e:
        k_norm_bwd_static(0, 1, 2, cols, z, z, st, g, None, None, out, None)
    assert e.value.status == 8 and "capacity" in str(e.value)
    assert not out.any()                 # nothing was launched
    # a missing input with an output requested is refused on the host as well (nothing is launched)
    ok = torch.zeros((2, 64), dtype=torch.float32, device="cuda")
    g64 = torch.ones(64, dtype=torch.float32, device="cuda")
    dst = torch.zeros((2, 64), dtype=torch.float32, device="cuda")
    for args in ((None, ok, st, g64), (ok, None, st, g64), (ok, ok, None, g64), (ok, ok, st, None)):
        with pytest.raises(HiftError) as e:
            k_norm_bwd_static(0, 1, 2, 64, args[0], args[1], args[2], args[3], None, dst, None, None)
        assert e.value.status == 4
    assert not dst.any()
