"""Pins for the oracle's layer math: finite differences, analytic identities,
brute force on tiny inputs, and special cases that reduce to library routines
(torch CPU, fp64).  No GPU."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import synth
from oracle import hift_oracle as O

torch.set_num_threads(4)


def mini(arch, **kw):
    base = dict(arch=arch, n_blocks=2, d_model=32, n_heads=4, d_ffn=64, vocab=61, max_pos=16,
                n_classes=2 if arch == 1 else 0, causal=0 if arch == 1 else 1, tie_head=0,
                norm_eps=1e-5 if arch != 2 else 1e-6, dtype=synth.DTYPE_FP32, batch=2, seq=8,
                init_std=0.2)
    base.update(kw)
    return synth.ModelCfg(**base)


def params64(cfg, seed=3):
    return {k: v.astype(np.float64) for k, v in synth.init_params(cfg, seed, perturb=0.1).items()}


def batch(cfg, seed=11, ignore=False):
    tok, lab = synth.batch_for(cfg, seed, 0, dist="uniform")
    if ignore and lab.ndim == 2:
        lab = lab.copy()
        lab[0, 1] = -1
        lab[1, -1] = -1
    return tok, lab


# ---------------------------------------------------------------- P1: finite differences
def _fd_check(cfg, n_samples=5, h=1e-5, rel=2e-6, ignore=False, lens=None, drop=None):
    P = params64(cfg)
    tok, lab = batch(cfg, ignore=ignore)
    if lens is not None and lab.ndim == 2:                      # padded positions carry no label
        lab = lab.copy()
        for b, l in enumerate(lens):
            lab[b, l:] = -1
    loss, cache = O.forward(cfg, P, tok, lab, lens, drop)
    G = O.backward(cfg, P, cache, None)
    rng = np.random.default_rng(0)
    assert set(G.keys()) == set(P.keys())
    for name, g in G.items():
        assert g.shape == P[name].shape, name
        scale = np.abs(g).max() + 1e-12
        flat = P[name].reshape(-1)
        # sample random entries plus the largest-gradient entry
        idx = list(rng.integers(0, flat.size, size=n_samples)) + [int(np.abs(g).argmax())]
        if name == "tok_emb":
            idx += [int(tok[0, 0]) * cfg.d_model + 1]          # a row that is actually gathered
        for i in idx:
            old = flat[i]
            flat[i] = old + h
            lp, _ = O.forward(cfg, P, tok, lab, lens, drop)
            flat[i] = old - h
            lm, _ = O.forward(cfg, P, tok, lab, lens, drop)
            flat[i] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - g.reshape(-1)[i]) <= rel * scale + 1e-9, (name, i, fd, g.reshape(-1)[i])


def test_fd_tiny_config_tied_head():
    cfg, _, _ = synth.config_tiny_fp32()
    _fd_check(cfg.scaled(init_std=0.08), n_samples=3)


def test_fd_preln_untied_with_ignored_labels():
    _fd_check(mini(0), ignore=True)


def test_fd_postln_classifier():
    _fd_check(mini(1))


def test_fd_llama():
    _fd_check(mini(2))
    _fd_check(mini(2, tie_head=1), n_samples=2)


def test_fd_with_key_padding():
    _fd_check(mini(1), lens=[5, 8], n_samples=3)
    _fd_check(mini(0), lens=[3, 6], n_samples=3)
    _fd_check(mini(2), lens=[8, 1], n_samples=2)


# ---------------------------------------------------------------- dropout from a counter-based generator
def test_philox_known_answers():
    """Philox4x32-10 against the known-answer vectors published with the generator (zero, all-ones and
    digits-of-pi counters and keys)."""
    kat = [((0, 0, 0, 0), (0, 0), (0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8)),
           ((0xFFFFFFFF,) * 4, (0xFFFFFFFF,) * 2, (0x408F276D, 0x41C83B0E, 0xA20BC7C6, 0x6D5451FD)),
           ((0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344), (0xA4093822, 0x299F31D0), (0xD16CFE09, 0x94FDCCEB, 0x5001E420, 0x24126EA1))]
    for ctr, key, want in kat:
        got = O.philox4x32_10(*[np.array([c]) for c in ctr], key[0], key[1])
        assert tuple(int(g[0]) for g in got) == want
    # vectorised over counters = one call per counter
    c0 = np.arange(5)
    many = O.philox4x32_10(c0, np.zeros(5), np.full(5, 7), np.full(5, 9), 123, 456)
    for i in range(5):
        one = O.philox4x32_10(np.array([i]), np.array([0]), np.array([7]), np.array([9]), 123, 456)
        assert [int(w[i]) for w in many] == [int(w[0]) for w in one]


def test_dropout_mask_is_a_function_of_seed_step_site_element():
    n, p = 200_000, 0.1
    m = O.dropout_mask(n, p, seed=5, site=3, step=11)
    assert set(np.unique(m).tolist()) == {0.0, 1.0 / (1.0 - p)}
    dropped = float((m == 0.0).mean())
    assert abs(dropped - p) < 4 * np.sqrt(p * (1 - p) / n)                # binomial, four sigma
    assert abs(m.mean() - 1.0) < 0.01                                     # inverted dropout keeps the expectation
    assert np.array_equal(m, O.dropout_mask(n, p, 5, 3, 11))
    for other in (O.dropout_mask(n, p, 6, 3, 11), O.dropout_mask(n, p, 5, 4, 11), O.dropout_mask(n, p, 5, 3, 12)):
        assert 0.15 < float((other != m).mean()) < 0.21                   # 2 p (1 - p) = 0.18 for independent masks
    assert np.array_equal(O.dropout_mask(1000, p, 5, 3, 11), m[:1000])    # element i does not depend on the tensor's size
    assert np.all(O.dropout_mask(64, 0.0, 5, 3, 11) == 1.0)
    # the threshold is floor(p 2^32) on the element's word: word 0 of the first counter decides element 0
    w = O.philox4x32_10(np.array([0]), np.array([0]), np.array([3]), np.array([11]), 5, 0)
    assert (m[0] == 0.0) == (int(w[0][0]) < int(np.floor(p * 2 ** 32)))


@pytest.mark.parametrize("arch", [0, 1, 2])
def test_fd_with_dropout(arch):
    """With the mask fixed by (seed, step), the loss is a smooth function of the parameters: finite differences
    check the masked backward pass at all three sites (embedding, attention output, feed-forward output)."""
    _fd_check(mini(arch), n_samples=3, drop=(0.25, 77, 3))


@pytest.mark.parametrize("arch", [0, 1, 2])
def test_fd_with_attention_probability_dropout(arch):
    """The same with the attention probabilities dropped as well (their own rate, sites 1000 + block): finite
    differences through o = (softmax o mask) v and its backward pass."""
    _fd_check(mini(arch), n_samples=3, drop=(0.1, 77, 3, 0.3))
    _fd_check(mini(arch), n_samples=2, drop=(0.0, 78, 1, 0.25))


def test_attention_probability_dropout_by_loops_and_its_element_numbering():
    """Attention with a probability mask against plain loops over (batch, head, query, key), forward and backward;
    and the mask the model draws: element ((b H + h) S + q) S' + k of site 1000 + block, S' = S rounded up to 4."""
    rng = np.random.default_rng(9)
    B, S, H, dh = 2, 5, 3, 4
    q, k, v, do = (rng.standard_normal((B, S, H, dh)) for _ in range(4))
    pm = np.where(rng.random((B, H, S, S)) < 0.3, 0.0, 1.0 / 0.7)
    for causal in (False, True):
        o, p = O.attention_fwd(q, k, v, causal, None, pm)
        dq, dk, dv = O.attention_bwd(do, q, k, v, p, pm)
        o_ref, dq_ref, dk_ref, dv_ref = (np.zeros((B, S, H, dh)) for _ in range(4))
        for b in range(B):
            for h in range(H):
                for i in range(S):
                    keys = range(i + 1) if causal else range(S)
                    sc = np.array([q[b, i, h] @ k[b, j, h] / np.sqrt(dh) for j in keys])
                    pr = np.exp(sc - sc.max()); pr /= pr.sum()
                    dp = np.array([(do[b, i, h] @ v[b, j, h]) * pm[b, h, i, j] for j in keys])
                    ds = pr * (dp - (dp * pr).sum())
                    for n, j in enumerate(keys):
                        o_ref[b, i, h] += pr[n] * pm[b, h, i, j] * v[b, j, h]
                        dv_ref[b, j, h] += pr[n] * pm[b, h, i, j] * do[b, i, h]
                        dq_ref[b, i, h] += ds[n] * k[b, j, h] / np.sqrt(dh)
                        dk_ref[b, j, h] += ds[n] * q[b, i, h] / np.sqrt(dh)
        for got, ref in ((o, o_ref), (dq, dq_ref), (dk, dk_ref), (dv, dv_ref)):
            np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-14)
    cfg = mini(0)
    P = params64(cfg)
    tok, lab = batch(cfg)
    _, c = O.forward(cfg, P, tok, lab, None, (0.0, 5, 2, 0.4))
    Bc, Sc = tok.shape
    Hc = cfg.n_heads
    Sp = (Sc + 3) // 4 * 4
    for i in range(cfg.n_blocks):
        m = c["blocks"][i]["pmask"]
        assert m.shape == (Bc, Hc, Sc, Sc) and 0.3 < float((m == 0).mean()) < 0.5
        flat = O.dropout_mask(Bc * Hc * Sc * Sp, 0.4, 5, 1000 + i, 2)
        b, h, qi, kj = 1, Hc - 1, Sc - 1, 2
        assert m[b, h, qi, kj] == flat[((b * Hc + h) * Sc + qi) * Sp + kj]
    assert np.all(c["mask_emb"] == 1.0)                                    # the other rate is its own
    l_plain, _ = O.forward(cfg, P, tok, lab)
    l_none, c0 = O.forward(cfg, P, tok, lab, None, (0.2, 5, 2))            # three-element form: no attention dropout
    assert c0["blocks"][0]["pmask"] is None and l_none != l_plain


def test_dropout_zero_is_the_plain_model_and_the_mask_reaches_every_site():
    cfg = mini(0)
    P = params64(cfg)
    tok, lab = batch(cfg)
    l0, _ = O.forward(cfg, P, tok, lab)
    l1, _ = O.forward(cfg, P, tok, lab, None, (0.0, 1, 0))
    assert l0 == l1
    l2, c2 = O.forward(cfg, P, tok, lab, None, (0.2, 1, 0))
    l3, _ = O.forward(cfg, P, tok, lab, None, (0.2, 1, 1))
    assert l2 != l0 and l3 != l2                                          # another step, another mask
    masks = [c2["mask_emb"]] + [c2["blocks"][i][k] for i in range(cfg.n_blocks) for k in ("mask_a", "mask_f")]
    assert all(np.ndim(m) == 3 and 0.1 < float((m == 0).mean()) < 0.3 for m in masks)
    assert len({m.tobytes() for m in masks}) == len(masks)                # every site draws its own


# ---------------------------------------------------------------- key padding reduces to shorter sequences
def test_key_padding_equals_attention_on_the_unpadded_rows():
    rng = np.random.default_rng(5)
    B, S, H, dh = 3, 7, 2, 4
    q, k, v = (rng.standard_normal((B, S, H, dh)) for _ in range(3))
    lens = [7, 3, 1]
    for causal in (False, True):
        full, _ = O.attention_fwd(q, k, v, causal)
        same, _ = O.attention_fwd(q, k, v, causal, lens=[S] * B)
        assert np.array_equal(full, same)
        o, p = O.attention_fwd(q, k, v, causal, lens=lens)
        for b, l in enumerate(lens):
            ref, _ = O.attention_fwd(q[b:b + 1, :l], k[b:b + 1, :l], v[b:b + 1, :l], causal)
            np.testing.assert_allclose(o[b, :l], ref[0], rtol=1e-13, atol=1e-15)
            assert np.all(p[b, :, :, l:] == 0.0)                       # no weight on padded keys
            np.testing.assert_allclose(p[b].sum(-1), 1.0, rtol=1e-13)
        # no gradient reaches padded keys or values
        do = rng.standard_normal((B, S, H, dh))
        _, dk, dv = O.attention_bwd(do, q, k, v, p)
        for b, l in enumerate(lens):
            assert np.all(dk[b, l:] == 0.0) and np.all(dv[b, l:] == 0.0)


def test_padded_batch_equals_the_sequences_run_alone():
    """Encoder + classifier: the loss of a right-padded batch with the length table is the mean of the losses of
    the unpadded sequences run one by one, whatever the pad token is; and the pad token's embedding gets no gradient."""
    cfg = mini(1, batch=3)
    P = params64(cfg)
    tok, lab = synth.batch_for(cfg, 11, 0, dist="uniform")
    lens = [8, 4, 2]
    pad_id = cfg.vocab - 1
    tok = np.where(tok == pad_id, 0, tok)
    for b, l in enumerate(lens):
        tok[b, l:] = pad_id
    loss, cache = O.forward(cfg, P, tok, lab, lens)
    alone = []
    for b, l in enumerate(lens):
        c1 = cfg.scaled(batch=1, seq=l)
        lb, _ = O.forward(c1, P, tok[b:b + 1, :l], lab[b:b + 1])
        alone.append(lb)
    assert loss == pytest.approx(np.mean(alone), rel=1e-12)
    tok2 = tok.copy()
    tok2[1, 4:] = 7                                                    # other pad content: same loss
    loss2, _ = O.forward(cfg, P, tok2, lab, lens)
    assert loss2 == pytest.approx(loss, rel=1e-13)
    G = O.backward(cfg, P, cache, None)
    assert np.all(G["tok_emb"][pad_id] == 0.0)
    loss_nomask, _ = O.forward(cfg, P, tok, lab)
    assert abs(loss_nomask - loss) > 1e-6                              # the table matters


# ---------------------------------------------------------------- P7: truncated == full restricted
@pytest.mark.parametrize("arch", [0, 1, 2])
def test_truncated_walk_equals_full_backward_bitwise(arch):
    cfg = mini(arch, n_blocks=3, tie_head=1 if arch == 0 else 0)
    P = params64(cfg)
    tok, lab = batch(cfg)
    _, cache = O.forward(cfg, P, tok, lab)
    full = O.backward(cfg, P, cache, None)
    for units in ([0], [1], [2], [3], [4], [1, 2], [3, 4], [0, 1], list(range(5))):
        part = O.backward(cfg, P, cache, units)
        names = [n for u in units for n in O.tensor_names_of_unit(cfg, u)]
        assert sorted(part.keys()) == sorted(names)
        for n in names:
            assert np.array_equal(part[n], full[n]), (units, n)


# ---------------------------------------------------------------- P8: identities
def test_identities_softmax_ce_layernorm_rope_causal():
    rng = np.random.default_rng(1)
    logits = rng.standard_normal((7, 13)) * 3
    labels = np.array([0, 5, -1, 12, 3, 3, 1])
    loss, d = O.cross_entropy(logits, labels)
    assert np.allclose(d.sum(axis=1), 0, atol=1e-15)            # rows of dlogits sum to 0
    assert np.all(d[2] == 0)
    # uniform logits -> loss = ln V
    l0, _ = O.cross_entropy(np.zeros((4, 512)), np.array([1, 2, 3, 4]))
    assert l0 == pytest.approx(math.log(512), rel=1e-14)
    # LayerNorm dX is orthogonal to 1 and to xhat
    x = rng.standard_normal((5, 16))
    g = rng.standard_normal(16)
    y, c = O.layernorm_fwd(x, g, rng.standard_normal(16), 0.0)       # exact only at eps = 0
    dx, _, _ = O.layernorm_bwd(rng.standard_normal((5, 16)), c, g)
    assert np.allclose(dx.sum(-1), 0, atol=1e-13)
    assert np.allclose((dx * c[0]).sum(-1), 0, atol=1e-12)
    # RoPE preserves the norm of each pair and position 0 is the identity; inverse undoes it
    cos, sin = O.rope_tables(8, 16, 10000.0)
    q = rng.standard_normal((2, 8, 3, 16))
    r = O.rope_apply(q, cos, sin)
    assert np.allclose(r[:, 0], q[:, 0])
    n0 = q[..., :8] ** 2 + q[..., 8:] ** 2
    n1 = r[..., :8] ** 2 + r[..., 8:] ** 2
    assert np.allclose(n0, n1, rtol=1e-13)
    assert np.allclose(O.rope_apply(r, cos, sin, inverse=True), q, atol=1e-14)
    # relative-position property: <rope(q)_s, rope(k)_t> depends on s - t only
    qv, kv = rng.standard_normal(16), rng.standard_normal(16)
    qs = O.rope_apply(np.tile(qv, (1, 8, 1, 1)), cos, sin)[0, :, 0]
    ks = O.rope_apply(np.tile(kv, (1, 8, 1, 1)), cos, sin)[0, :, 0]
    assert qs[5] @ ks[3] == pytest.approx(qs[4] @ ks[2], rel=1e-12)
    # causal attention: output at position s does not depend on later tokens
    q, k, v = (rng.standard_normal((1, 6, 2, 4)) for _ in range(3))
    o1, p1 = O.attention_fwd(q, k, v, True)
    k2, v2 = k.copy(), v.copy()
    k2[:, 4:] += 1.0
    v2[:, 4:] -= 2.0
    o2, _ = O.attention_fwd(q, k2, v2, True)
    assert np.array_equal(o1[:, :4], o2[:, :4])
    assert np.allclose(p1.sum(-1), 1.0, atol=1e-15)


def test_initial_loss_near_ln_vocab():
    cfg, _, _ = synth.config_tiny_fp32()
    P = {k: v.astype(np.float64) for k, v in synth.init_params(cfg, 0).items()}
    tok, lab = synth.lm_batch(cfg, 0, 0, dist="uniform")
    loss, _ = O.forward(cfg, P, tok, lab)
    assert abs(loss - math.log(512)) < 0.05


# ---------------------------------------------------------------- P10: brute force
def test_attention_brute_force_loops():
    rng = np.random.default_rng(2)
    B, S, H, dh = 2, 5, 2, 3
    q, k, v = (rng.standard_normal((B, S, H, dh)) for _ in range(3))
    for causal in (True, False):
        o, _ = O.attention_fwd(q, k, v, causal)
        for b in range(B):
            for h in range(H):
                for s in range(S):
                    lim = s + 1 if causal else S
                    sc = [sum(q[b, s, h, e] * k[b, t, h, e] for e in range(dh)) / math.sqrt(dh) for t in range(lim)]
                    mx = max(sc)
                    w = [math.exp(a - mx) for a in sc]
                    z = sum(w)
                    for e in range(dh):
                        ref = sum(w[t] / z * v[b, t, h, e] for t in range(lim))
                        assert o[b, s, h, e] == pytest.approx(ref, rel=1e-12, abs=1e-14)


def test_embedding_gradient_by_token_loops():
    cfg = mini(0, n_blocks=1)
    P = params64(cfg)
    tok, lab = batch(cfg)
    tok[:, :3] = 7                                   # repeated ids must accumulate
    _, cache = O.forward(cfg, P, tok, lab)
    G = O.backward(cfg, P, cache, None)
    # recover d loss / d x0 by back-propagating with only the embedding output perturbed:
    # use the position gradient (sum over batch) and the token gradient (sum over occurrences)
    # and check they describe the same per-token gradient field.
    Gblk = O.backward(cfg, P, cache, [0])
    assert np.array_equal(G["tok_emb"], Gblk["tok_emb"])
    # per-token loops: rows never used have zero gradient; row sums agree with position sums
    used = set(tok.reshape(-1).tolist())
    for r in range(cfg.vocab):
        if r not in used:
            assert not G["tok_emb"][r].any()
    assert np.allclose(G["tok_emb"].sum(axis=0), G["pos_emb"].sum(axis=0), rtol=1e-11, atol=1e-14)
    assert not G["pos_emb"][cfg.seq:].any()


# ---------------------------------------------------------------- library-routine special cases
def test_against_torch_library_routines():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((6, 24))
    g, b = rng.standard_normal(24), rng.standard_normal(24)
    y, _ = O.layernorm_fwd(x, g, b, 1e-5)
    yt = F.layer_norm(torch.tensor(x), (24,), torch.tensor(g), torch.tensor(b), 1e-5).numpy()
    assert np.allclose(y, yt, rtol=1e-12, atol=1e-13)
    yr, _ = O.rmsnorm_fwd(x, g, 1e-6)
    yrt = F.rms_norm(torch.tensor(x), (24,), torch.tensor(g), 1e-6).numpy()
    assert np.allclose(yr, yrt, rtol=1e-12, atol=1e-13)
    a = rng.standard_normal(100) * 3
    assert np.allclose(O.gelu_fwd(a), F.gelu(torch.tensor(a)).numpy(), rtol=1e-12, atol=1e-14)
    at = torch.tensor(a, requires_grad=True)
    F.gelu(at).sum().backward()
    assert np.allclose(O.gelu_bwd(np.ones(100), a), at.grad.numpy(), rtol=1e-11, atol=1e-13)
    gate, up = rng.standard_normal(50) * 3, rng.standard_normal(50)
    assert np.allclose(O.swiglu_fwd(gate, up), (F.silu(torch.tensor(gate)) * torch.tensor(up)).numpy(), rtol=1e-12)
    gt, ut = torch.tensor(gate, requires_grad=True), torch.tensor(up, requires_grad=True)
    (F.silu(gt) * ut).sum().backward()
    dg, du = O.swiglu_bwd(np.ones(50), gate, up)
    assert np.allclose(dg, gt.grad.numpy(), rtol=1e-11, atol=1e-13)
    assert np.allclose(du, ut.grad.numpy(), rtol=1e-11, atol=1e-13)
    logits = rng.standard_normal((9, 17)) * 2
    labels = np.array([1, 2, -1, 4, 16, 0, 0, -1, 3])
    lt = torch.tensor(logits, requires_grad=True)
    loss_t = F.cross_entropy(lt, torch.tensor(labels), ignore_index=-1)
    loss_t.backward()
    loss, d = O.cross_entropy(logits, labels)
    assert loss == pytest.approx(loss_t.item(), rel=1e-13)
    assert np.allclose(d, lt.grad.numpy(), rtol=1e-11, atol=1e-15)
    q, k, v = (rng.standard_normal((2, 7, 3, 8)) for _ in range(3))
    for causal in (True, False):
        o, p = O.attention_fwd(q, k, v, causal)
        qt, kt, vt = (torch.tensor(t.transpose(0, 2, 1, 3), requires_grad=True) for t in (q, k, v))
        ot = F.scaled_dot_product_attention(qt, kt, vt, is_causal=causal)
        assert np.allclose(o, ot.detach().numpy().transpose(0, 2, 1, 3), rtol=1e-11, atol=1e-13)
        do = rng.standard_normal(o.shape)
        ot.backward(torch.tensor(do.transpose(0, 2, 1, 3)))
        dq, dk, dv = O.attention_bwd(do, q, k, v, p)
        for mine, ref in ((dq, qt), (dk, kt), (dv, vt)):
            assert np.allclose(mine, ref.grad.numpy().transpose(0, 2, 1, 3), rtol=1e-10, atol=1e-12)


def test_bf16_round_matches_torch_and_ties_to_even():
    rng = np.random.default_rng(9)
    x = (rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000)).astype(np.float32)
    ref = torch.tensor(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.bf16_round(x), ref)
    # exact ties: 1 + 2^-8 is halfway between 1 and 1+2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert O.bf16_round(np.float32(1 + 2.0 ** -8)) == np.float32(1.0)
    assert O.bf16_round(np.float32(1 + 3 * 2.0 ** -8)) == np.float32(1 + 2.0 ** -6)
