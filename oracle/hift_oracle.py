"""fp64 CPU oracle for the hierarchical fine-tuning (HiFT) training step.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
CUDA library is checked against.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import it; the product path never does, and
this file imports nothing from the CUDA package.

What it computes (paper: Algorithm 1, Eq. 2-3, Section "Memory Analysis"):
  * the unit / group / order bookkeeping of Algorithm 1 (steps c-g), with the
    learning rate advanced once per full cycle of groups (last branch of
    Algorithm 1);
  * a transformer forward pass and ordinary reverse-mode back-propagation in
    fp64, either over every parameter ("full") or walking down only as far as
    the lowest unit of the active group and forming parameter gradients only
    inside it ("truncated", Algorithm 1 step "Backpropagation");
  * textbook AdamW / AdaGrad / SGD-momentum updates applied to the active
    group only, all other numbers untouched (Eq. 2-3: only beta_i o theta moves);
  * the closed-form memory model zeta_fpft = 4 zeta_1, zeta_hift = (k+3)/k zeta_1.

The method is exact with respect to its own definition (back-propagation
restricted to a parameter subset, then a textbook optimizer), so the oracle is
that definition written out.  numpy matmul / scipy erf are used as library
primitives; there is no blocking, fusion or reordering.

Readings taken where the paper is silent are listed in the repository's design
notes; the ones that matter here: units are [embedding(s)], each block, [head
incl. final norm]; groups are a fixed partition in chunks of m (last one short);
"random" shuffles the group order once; a tied LM head matrix belongs to the
embedding unit; Adam bias correction counts the updates the *group* has had;
eps sits outside the square root; decoupled weight decay touches every element
of the group; GELU is the exact erf form; RoPE pairs (j, j + d_h/2).

Parity pins live in tests/test_oracle_*.py (finite differences, closed-form
optimizer steps, frozen-parameter identity, single-group == full step, brute
force attention, library-routine special cases, the paper's printed figures).
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
from scipy.special import erf as _erf

F64 = np.float64

# --------------------------------------------------------------------------
# Number formats
# --------------------------------------------------------------------------
def bf16_round(x) -> np.ndarray:
    """Round fp32 values to the nearest bfloat16 (ties to even); result as fp32.

    bfloat16 is the upper 16 bits of an IEEE binary32; rounding adds
    0x7FFF + (lsb of the kept part) and truncates."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


# --------------------------------------------------------------------------
# Algorithm 1, bookkeeping: units, groups, order, delayed learning rate
# --------------------------------------------------------------------------
def num_groups(n: int, m: int) -> int:
    """k = n/m if m divides n, else floor(n/m)+1 (paper, Notation)."""
    return n // m if n % m == 0 else n // m + 1


def build_groups(n_units: int, m: int, split_emb_head: int = 0, sizes: Sequence[int] = ()) -> List[List[int]]:
    """Fixed partition of unit ids 0..n-1 (0 = embedding, n-1 = head) into
    consecutive chunks of m, last chunk short.  With split_emb_head the
    embedding and the head are groups of their own and only the blocks are
    chunked.  With `sizes` the chunk lengths are the caller's (the paper's
    Notation paragraph groups uniformly; an uneven partition keeps every
    other rule of Algorithm 1: fixed groups, each trained once per cycle)."""
    if len(sizes) > 0:
        if any(int(z) < 1 for z in sizes) or sum(int(z) for z in sizes) != n_units:
            raise ValueError("group sizes must be >= 1 and sum to the number of units")
        out, u = [], 0
        for z in sizes:
            out.append(list(range(u, u + int(z))))
            u += int(z)
        return out
    if m < 1:
        raise ValueError("m must be >= 1")
    if split_emb_head:
        blocks = list(range(1, n_units - 1))
        groups = [[0]]
        groups += [blocks[i:i + m] for i in range(0, len(blocks), m)]
        groups.append([n_units - 1])
        return groups
    ids = list(range(n_units))
    return [ids[i:i + m] for i in range(0, n_units, m)]


_MASK64 = (1 << 64) - 1


def splitmix64(state: int) -> Tuple[int, int]:
    """One step of the SplitMix64 generator (Steele, Lea, Flood 2014)."""
    state = (state + 0x9E3779B97F4A7C15) & _MASK64
    z = state
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    z = z ^ (z >> 31)
    return state, z


def group_order(k: int, order: int, seed: int = 0) -> List[int]:
    """bottom2up: 0..k-1; top2down: k-1..0; random: ONE Fisher-Yates shuffle of
    0..k-1 (SplitMix64 draws, j = draw mod (i+1), i = k-1 .. 1), then fixed."""
    idx = list(range(k))
    if order == 0:
        return idx
    if order == 1:
        return idx[::-1]
    if order == 2:
        s = seed & _MASK64
        for i in range(k - 1, 0, -1):
            s, r = splitmix64(s)
            j = r % (i + 1)
            idx[i], idx[j] = idx[j], idx[i]
        return idx
    raise ValueError("order")


def queue_walk(n_units: int, m: int, order: int, steps: int, seed: int = 0) -> List[List[int]]:
    """Literal queue of Algorithm 1 (steps c, d): Q holds unit ids in strategy
    order (random: the one-time shuffle of the unit ids); each step removes m ids
    from the head and appends them to the tail."""
    q = group_order(n_units, order, seed)
    out = []
    for _ in range(steps):
        e, q = q[:m], q[m:]
        q = q + e
        out.append(e)
    return out


def lr_for_cycle(lr0: float, sched: int, cycle: int, total_cycles: int, warmup_cycles: int = 0) -> float:
    """Delayed learning rate: a function of the completed-cycle count only, so
    it is constant inside a cycle.  const -> lr0; linear -> lr0*max(0, 1-c/C).

    The paper's hyper-parameter tables list a warm-up ratio next to the linear
    schedule (Appendix, hyper-parameter tables: warmup in {0, 0.02, 0.06}).  Read
    as the usual linear warm-up of that schedule, counted in cycles because the
    schedule only moves once per cycle: with W = warmup_cycles,
        c <  W : lr0 * c / W                     (the first cycle runs at 0)
        c >= W : lr0 * max(0, (C - c) / (C - W))
    which is the formula above when W = 0."""
    if sched == 0:
        return lr0
    W, C = int(warmup_cycles), int(total_cycles)
    if cycle < W:
        return lr0 * cycle / float(W)
    return lr0 * max(0.0, (C - cycle) / float(max(1, C - W)))


# --------------------------------------------------------------------------
# Memory model (paper, "Memory Analysis")
# --------------------------------------------------------------------------
def zeta_fpft(zeta1: float) -> float:
    return zeta1 + 2.0 * zeta1 + zeta1


def zeta_hift(zeta1: float, k: int) -> float:
    return zeta1 + 2.0 * zeta1 / k + zeta1 / k


def peak_trainable_fraction(unit_params: Sequence[int], groups: Sequence[Sequence[int]]) -> float:
    tot = float(sum(unit_params))
    return max(sum(unit_params[u] for u in g) for g in groups) / tot


# --------------------------------------------------------------------------
# Layer math, forward and backward, fp64
# --------------------------------------------------------------------------
def layernorm_fwd(x, g, b, eps):
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = (x - mu) * rstd
    return xhat * g + b, (xhat, rstd)


def layernorm_bwd(dy, cache, g):
    xhat, rstd = cache
    dg = (dy * xhat).reshape(-1, xhat.shape[-1]).sum(axis=0)
    db = dy.reshape(-1, xhat.shape[-1]).sum(axis=0)
    dxh = dy * g
    dx = rstd * (dxh - dxh.mean(axis=-1, keepdims=True)
                 - xhat * (dxh * xhat).mean(axis=-1, keepdims=True))
    return dx, dg, db


def rmsnorm_fwd(x, g, eps):
    r = 1.0 / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)
    return x * r * g, (x, r)


def rmsnorm_bwd(dy, cache, g):
    x, r = cache
    dg = (dy * x * r).reshape(-1, x.shape[-1]).sum(axis=0)
    dxh = dy * g
    dx = r * dxh - x * (r ** 3) * (dxh * x).mean(axis=-1, keepdims=True)
    return dx, dg


def gelu_fwd(a):
    return 0.5 * a * (1.0 + _erf(a / math.sqrt(2.0)))


def gelu_bwd(da_out, a):
    cdf = 0.5 * (1.0 + _erf(a / math.sqrt(2.0)))
    pdf = np.exp(-0.5 * a * a) / math.sqrt(2.0 * math.pi)
    return da_out * (cdf + a * pdf)


def swiglu_fwd(gate, up):
    sig = 1.0 / (1.0 + np.exp(-gate))
    return gate * sig * up


def swiglu_bwd(ds, gate, up):
    sig = 1.0 / (1.0 + np.exp(-gate))
    dgate = ds * up * sig * (1.0 + gate * (1.0 - sig))
    dup = ds * gate * sig
    return dgate, dup


def rope_tables(seq: int, d_head: int, base: float):
    half = d_head // 2
    inv = base ** (-2.0 * np.arange(half, dtype=F64) / d_head)
    ang = np.arange(seq, dtype=F64)[:, None] * inv[None, :]
    return np.cos(ang), np.sin(ang)            # [S, half]


def rope_apply(x, cos, sin, inverse=False):
    """x: [B, S, H, d_h]; rotates pair (j, j+half) by +angle (or -angle)."""
    half = x.shape[-1] // 2
    x1, x2 = x[..., :half], x[..., half:]
    c = cos[None, :, None, :]
    s = sin[None, :, None, :]
    if inverse:
        s = -s
    return np.concatenate([x1 * c - x2 * s, x1 * s + x2 * c], axis=-1)


def attention_fwd(q, k, v, causal: bool, lens=None, pmask=None):
    """q,k,v: [B, S, H, d_h] -> o [B, S, H, d_h]; softmax(q k^T / sqrt(d_h) + mask) v.
    pmask (optional, [B, H, S, S]): dropout multipliers of the probabilities (0 or 1 / (1 - p)),
    applied after the softmax: o = (softmax o pmask) v; the returned p is the softmax itself.
    lens (optional, [B] ints in 1..S): batch entry b is a sequence of lens[b] real
    tokens padded on the right; keys at positions >= lens[b] get probability 0
    (the usual key-padding mask of the models the paper fine-tunes; the paper
    itself does not describe batching)."""
    B, S, H, dh = q.shape
    qh, kh, vh = (t.transpose(0, 2, 1, 3) for t in (q, k, v))      # [B,H,S,dh]
    s = np.matmul(qh, kh.transpose(0, 1, 3, 2)) / math.sqrt(dh)
    if causal:
        mask = np.triu(np.ones((S, S), dtype=bool), k=1)
        s = np.where(mask, -np.inf, s)
    if lens is not None:
        pad = np.arange(S)[None, :] >= np.asarray(lens).reshape(B, 1)          # [B, S] True at padded keys
        s = np.where(pad[:, None, None, :], -np.inf, s)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=-1, keepdims=True)
    pd = p if pmask is None else p * pmask
    o = np.matmul(pd, vh).transpose(0, 2, 1, 3)
    return o, p


def attention_bwd(do, q, k, v, p, pmask=None):
    """Backward of attention_fwd; with pmask, o = (p o pmask) v: dv takes the dropped probabilities and the
    gradient of the softmax output is (do v^T) o pmask."""
    B, S, H, dh = q.shape
    qh, kh, vh, doh = (t.transpose(0, 2, 1, 3) for t in (q, k, v, do))
    pd = p if pmask is None else p * pmask
    dv = np.matmul(pd.transpose(0, 1, 3, 2), doh)
    dp = np.matmul(doh, vh.transpose(0, 1, 3, 2))
    if pmask is not None:
        dp = dp * pmask
    ds = p * (dp - (dp * p).sum(axis=-1, keepdims=True))
    dq = np.matmul(ds, kh) / math.sqrt(dh)
    dk = np.matmul(ds.transpose(0, 1, 3, 2), qh) / math.sqrt(dh)
    return tuple(t.transpose(0, 2, 1, 3) for t in (dq, dk, dv))


def cross_entropy(logits, labels):
    """Mean over rows with label >= 0 of -log softmax(logits)[label].
    Returns loss, dlogits."""
    z = logits - logits.max(axis=-1, keepdims=True)
    lse = np.log(np.exp(z).sum(axis=-1, keepdims=True))
    logp = z - lse
    valid = labels >= 0
    nvalid = int(valid.sum())
    rows = np.nonzero(valid)[0]
    loss = -logp[rows, labels[rows]].sum() / nvalid
    d = np.exp(logp)
    d[rows, labels[rows]] -= 1.0
    d[~valid] = 0.0
    return float(loss), d / nvalid


# --------------------------------------------------------------------------
# Dropout masks from a counter-based generator
# --------------------------------------------------------------------------
# The paper's hyper-parameter tables fine-tune with the models' usual dropout; a deterministic parity
# check needs both sides to draw the same mask, so the mask is a pure function of (seed, step, site,
# element): Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
# SC'11), key = the 64-bit seed, counter = (element // 4 as two words, site, step), word element % 4
# of the output.  An element is kept iff its word >= floor(p * 2^32), and kept values are scaled by
# 1 / (1 - p).  Sites: 0 = embedding output; 1 + 2 i = output of block i's attention projection and
# 2 + 2 i = output of its feed-forward network, each before the residual addition; 1000 + i = the
# attention probabilities of block i (after the softmax, before the product with V, as the models'
# usual implementations do it), with their own rate.  The probabilities' elements are numbered
# ((b H + h) S + q) S' + k with S' = S rounded up to a multiple of 4, so that the four words of one
# generator block always belong to one query row.
_PHILOX_M0, _PHILOX_M1, _PHILOX_W0, _PHILOX_W1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Ten rounds of Philox-4x32 on arrays of 32-bit counter words; returns four arrays of 32-bit words."""
    m32 = np.uint64(0xFFFFFFFF)
    c = [np.asarray(x, dtype=np.uint64) & m32 for x in (c0, c1, c2, c3)]
    k0, k1 = np.uint64(k0 & 0xFFFFFFFF), np.uint64(k1 & 0xFFFFFFFF)
    for _ in range(10):
        p0 = np.uint64(_PHILOX_M0) * c[0]
        p1 = np.uint64(_PHILOX_M1) * c[2]
        c = [(p1 >> np.uint64(32)) ^ c[1] ^ k0, p1 & m32, (p0 >> np.uint64(32)) ^ c[3] ^ k1, p0 & m32]
        k0 = (k0 + np.uint64(_PHILOX_W0)) & m32
        k1 = (k1 + np.uint64(_PHILOX_W1)) & m32
    return c


def dropout_mask(numel: int, p: float, seed: int, site: int, step: int) -> np.ndarray:
    """Multiplier of each of `numel` elements (row-major order): 0 where dropped, 1 / (1 - p) where kept."""
    if p <= 0.0:
        return np.ones(numel, dtype=F64)
    idx = np.arange(numel, dtype=np.uint64)
    blk = idx >> np.uint64(2)
    w = philox4x32_10(blk & np.uint64(0xFFFFFFFF), blk >> np.uint64(32), np.full(numel, site, dtype=np.uint64),
                      np.full(numel, step & 0xFFFFFFFF, dtype=np.uint64), seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    word = np.choose((idx & np.uint64(3)).astype(np.int64), w)
    thr = np.uint64(int(math.floor(p * 4294967296.0)))
    return np.where(word >= thr, 1.0 / (1.0 - p), 0.0)


# --------------------------------------------------------------------------
# Model: forward, full backward, truncated backward
# --------------------------------------------------------------------------
def tensor_names_of_unit(cfg, unit: int) -> List[str]:
    """Names of the parameter tensors each unit owns (0 = embedding,
    1..L = blocks, L+1 = head).  A tied LM-head matrix is 'tok_emb' and belongs
    to the embedding unit."""
    L = cfg.n_blocks
    if unit == 0:
        n = ["tok_emb"]
        if cfg.arch in (0, 1):
            n.append("pos_emb")
        if cfg.arch == 1:
            n += ["emb_ln_g", "emb_ln_b"]
        return n
    if unit == L + 1:
        if cfg.arch == 1:
            return ["w_cls", "b_cls"]
        n = ["rmsf_g"] if cfg.arch == 2 else ["lnf_g", "lnf_b"]
        if not cfg.tie_head:
            n.append("w_head")
        return n
    p = f"b{unit - 1}."
    if cfg.arch == 2:
        return [p + s for s in ("rms1_g", "w_qkv", "w_o", "rms2_g", "w_gu", "w_down")]
    return [p + s for s in ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
                            "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")]


def _split_heads(t, H):
    B, S, D = t.shape
    return t.reshape(B, S, H, D // H)


def _merge_heads(t):
    B, S, H, dh = t.shape
    return t.reshape(B, S, H * dh)


def forward(cfg, P: Dict[str, np.ndarray], tokens: np.ndarray, labels: np.ndarray, lens=None, drop=None):
    """Whole-model forward in fp64.  Returns (loss, cache).
    drop = (p, seed, step) or (p, seed, step, p_attn): dropout with the counter-based masks of dropout_mask
    (p at the residual-branch outputs and the embedding output, p_attn on the attention probabilities);
    None: no dropout."""
    B, S = tokens.shape
    d, H = cfg.d_model, cfg.n_heads
    dh = d // H
    causal = bool(cfg.causal)
    eps = cfg.norm_eps
    cache = {"tokens": tokens, "labels": labels, "blocks": []}

    def mask(site):
        if drop is None or drop[0] <= 0.0:
            return 1.0
        return dropout_mask(B * S * d, drop[0], drop[1], site, drop[2]).reshape(B, S, d)

    def pmask(i):
        if drop is None or len(drop) < 4 or drop[3] <= 0.0:
            return None
        Sp = (S + 3) // 4 * 4
        return dropout_mask(B * H * S * Sp, drop[3], drop[1], 1000 + i, drop[2]).reshape(B, H, S, Sp)[..., :S]

    x = P["tok_emb"][tokens]                                   # [B,S,d]
    if cfg.arch in (0, 1):
        x = x + P["pos_emb"][:S][None, :, :]
    if cfg.arch == 1:
        x, cache["emb_ln"] = layernorm_fwd(x, P["emb_ln_g"], P["emb_ln_b"], eps)
    cache["mask_emb"] = mask(0)
    x = x * cache["mask_emb"]
    if cfg.arch == 2:
        cos, sin = rope_tables(S, dh, cfg.rope_base)
        cache["rope"] = (cos, sin)
    for i in range(cfg.n_blocks):
        p = f"b{i}."
        c = {}
        if cfg.arch == 0:          # pre-LN: x += Attn(LN1 x); x += FFN(LN2 x)
            h1, c["ln1"] = layernorm_fwd(x, P[p + "ln1_g"], P[p + "ln1_b"], eps)
            qkv = h1 @ P[p + "w_qkv"].T + P[p + "b_qkv"]
            q, k, v = (_split_heads(t, H) for t in np.split(qkv, 3, axis=-1))
            c["pmask"] = pmask(i)
            o, prob = attention_fwd(q, k, v, causal, lens, c["pmask"])
            om = _merge_heads(o)
            c["mask_a"], c["mask_f"] = mask(1 + 2 * i), mask(2 + 2 * i)
            x2 = x + (om @ P[p + "w_o"].T + P[p + "b_o"]) * c["mask_a"]
            h2, c["ln2"] = layernorm_fwd(x2, P[p + "ln2_g"], P[p + "ln2_b"], eps)
            a = h2 @ P[p + "w_fc1"].T + P[p + "b_fc1"]
            u = gelu_fwd(a)
            x3 = x2 + (u @ P[p + "w_fc2"].T + P[p + "b_fc2"]) * c["mask_f"]
            c.update(h1=h1, q=q, k=k, v=v, p=prob, om=om, h2=h2, a=a, u=u)
            x = x3
        elif cfg.arch == 1:        # post-LN: x = LN1(x + Attn x); x = LN2(x + FFN x)
            qkv = x @ P[p + "w_qkv"].T + P[p + "b_qkv"]
            q, k, v = (_split_heads(t, H) for t in np.split(qkv, 3, axis=-1))
            c["pmask"] = pmask(i)
            o, prob = attention_fwd(q, k, v, causal, lens, c["pmask"])
            om = _merge_heads(o)
            c["mask_a"], c["mask_f"] = mask(1 + 2 * i), mask(2 + 2 * i)
            y = x + (om @ P[p + "w_o"].T + P[p + "b_o"]) * c["mask_a"]
            x1, c["ln1"] = layernorm_fwd(y, P[p + "ln1_g"], P[p + "ln1_b"], eps)
            a = x1 @ P[p + "w_fc1"].T + P[p + "b_fc1"]
            u = gelu_fwd(a)
            z = x1 + (u @ P[p + "w_fc2"].T + P[p + "b_fc2"]) * c["mask_f"]
            xo, c["ln2"] = layernorm_fwd(z, P[p + "ln2_g"], P[p + "ln2_b"], eps)
            c.update(xin=x, q=q, k=k, v=v, p=prob, om=om, x1=x1, a=a, u=u)
            x = xo
        else:                      # LLaMA: RMSNorm, RoPE on q and k, SwiGLU, no biases
            h1, c["rms1"] = rmsnorm_fwd(x, P[p + "rms1_g"], eps)
            qkv = h1 @ P[p + "w_qkv"].T
            q, k, v = (_split_heads(t, H) for t in np.split(qkv, 3, axis=-1))
            q = rope_apply(q, cos, sin)
            k = rope_apply(k, cos, sin)
            c["pmask"] = pmask(i)
            o, prob = attention_fwd(q, k, v, causal, lens, c["pmask"])
            om = _merge_heads(o)
            c["mask_a"], c["mask_f"] = mask(1 + 2 * i), mask(2 + 2 * i)
            x2 = x + (om @ P[p + "w_o"].T) * c["mask_a"]
            h2, c["rms2"] = rmsnorm_fwd(x2, P[p + "rms2_g"], eps)
            gu = h2 @ P[p + "w_gu"].T
            gate, up = np.split(gu, 2, axis=-1)
            s = swiglu_fwd(gate, up)
            x3 = x2 + (s @ P[p + "w_down"].T) * c["mask_f"]
            c.update(h1=h1, q=q, k=k, v=v, p=prob, om=om, h2=h2, gate=gate, up=up, s=s)
            x = x3
        cache["blocks"].append(c)
    # head
    if cfg.arch == 1:
        pooled = x[:, 0, :]
        logits = pooled @ P["w_cls"].T + P["b_cls"]
        loss, dlogits = cross_entropy(logits, labels.reshape(-1))
        cache.update(pooled=pooled, x_shape=x.shape)
    else:
        if cfg.arch == 2:
            xf, cache["normf"] = rmsnorm_fwd(x, P["rmsf_g"], eps)
        else:
            xf, cache["normf"] = layernorm_fwd(x, P["lnf_g"], P["lnf_b"], eps)
        W = P["tok_emb"] if cfg.tie_head else P["w_head"]
        logits = xf.reshape(B * S, d) @ W.T
        loss, dlogits = cross_entropy(logits, labels.reshape(-1))
        cache.update(xf=xf)
    cache["logits"] = logits
    cache["dlogits"] = dlogits
    return loss, cache


def _rows(t):
    return t.reshape(-1, t.shape[-1])


def backward(cfg, P, cache, active_units: Optional[Sequence[int]] = None) -> Dict[str, np.ndarray]:
    """Reverse-mode gradients of the loss.

    active_units = None: ordinary full back-propagation; gradients of every
    parameter tensor are returned.
    active_units = set of unit ids: the walk starts at the loss, forms
    activation gradients through every unit above the lowest active one,
    forms parameter gradients only for tensors owned by active units, and
    stops as soon as nothing below can be needed."""
    L = cfg.n_blocks
    full = active_units is None
    act = set(range(L + 2)) if full else set(active_units)
    lo = min(act)
    H = cfg.n_heads
    causal = bool(cfg.causal)
    G: Dict[str, np.ndarray] = {}
    tokens = cache["tokens"]
    B, S = tokens.shape
    d = cfg.d_model
    dlogits = cache["dlogits"]
    head_on = (L + 1) in act
    # ---- head ----
    if cfg.arch == 1:
        if head_on:
            G["w_cls"] = dlogits.T @ cache["pooled"]
            G["b_cls"] = dlogits.sum(axis=0)
        if lo == L + 1:
            return G
        dx = np.zeros(cache["x_shape"], dtype=F64)
        dx[:, 0, :] = dlogits @ P["w_cls"]
    else:
        W = P["tok_emb"] if cfg.tie_head else P["w_head"]
        xf = cache["xf"]
        if cfg.tie_head:
            if 0 in act:
                G["tok_emb"] = dlogits.T @ _rows(xf)
        elif head_on:
            G["w_head"] = dlogits.T @ _rows(xf)
        need_dx = lo <= L
        if head_on or need_dx:
            dxf = (dlogits @ W).reshape(B, S, d)
            if cfg.arch == 2:
                dx, dg = rmsnorm_bwd(dxf, cache["normf"], P["rmsf_g"])
                if head_on:
                    G["rmsf_g"] = dg
            else:
                dx, dg, db = layernorm_bwd(dxf, cache["normf"], P["lnf_g"])
                if head_on:
                    G["lnf_g"], G["lnf_b"] = dg, db
        if not need_dx:
            return G
    # ---- blocks, top down ----
    for i in range(L - 1, -1, -1):
        unit = i + 1
        if unit < lo:
            return G
        on = unit in act
        need_dx = unit > lo
        c = cache["blocks"][i]
        p = f"b{i}."
        if cfg.arch == 0:
            dfo = dx * c["mask_f"]                               # through the dropout of the feed-forward output
            du = dfo @ P[p + "w_fc2"]
            if on:
                G[p + "w_fc2"] = _rows(dfo).T @ _rows(c["u"])
                G[p + "b_fc2"] = _rows(dfo).sum(axis=0)
            da = gelu_bwd(du, c["a"])
            dh2 = da @ P[p + "w_fc1"]
            if on:
                G[p + "w_fc1"] = _rows(da).T @ _rows(c["h2"])
                G[p + "b_fc1"] = _rows(da).sum(axis=0)
            dn, dg, db = layernorm_bwd(dh2, c["ln2"], P[p + "ln2_g"])
            if on:
                G[p + "ln2_g"], G[p + "ln2_b"] = dg, db
            dx2 = dx + dn
            dao = dx2 * c["mask_a"]                              # through the dropout of the attention output
            dom = dao @ P[p + "w_o"]
            if on:
                G[p + "w_o"] = _rows(dao).T @ _rows(c["om"])
                G[p + "b_o"] = _rows(dao).sum(axis=0)
            dq, dk, dv = attention_bwd(_split_heads(dom, H), c["q"], c["k"], c["v"], c["p"], c.get("pmask"))
            dqkv = np.concatenate([_merge_heads(t) for t in (dq, dk, dv)], axis=-1)
            dh1 = dqkv @ P[p + "w_qkv"]
            if on:
                G[p + "w_qkv"] = _rows(dqkv).T @ _rows(c["h1"])
                G[p + "b_qkv"] = _rows(dqkv).sum(axis=0)
            dn, dg, db = layernorm_bwd(dh1, c["ln1"], P[p + "ln1_g"])
            if on:
                G[p + "ln1_g"], G[p + "ln1_b"] = dg, db
            if not need_dx:
                return G
            dx = dx2 + dn
        elif cfg.arch == 1:
            dz, dg, db = layernorm_bwd(dx, c["ln2"], P[p + "ln2_g"])
            if on:
                G[p + "ln2_g"], G[p + "ln2_b"] = dg, db
            dfo = dz * c["mask_f"]
            du = dfo @ P[p + "w_fc2"]
            if on:
                G[p + "w_fc2"] = _rows(dfo).T @ _rows(c["u"])
                G[p + "b_fc2"] = _rows(dfo).sum(axis=0)
            da = gelu_bwd(du, c["a"])
            dx1 = dz + da @ P[p + "w_fc1"]
            if on:
                G[p + "w_fc1"] = _rows(da).T @ _rows(c["x1"])
                G[p + "b_fc1"] = _rows(da).sum(axis=0)
            dy, dg, db = layernorm_bwd(dx1, c["ln1"], P[p + "ln1_g"])
            if on:
                G[p + "ln1_g"], G[p + "ln1_b"] = dg, db
            dao = dy * c["mask_a"]
            dom = dao @ P[p + "w_o"]
            if on:
                G[p + "w_o"] = _rows(dao).T @ _rows(c["om"])
                G[p + "b_o"] = _rows(dao).sum(axis=0)
            dq, dk, dv = attention_bwd(_split_heads(dom, H), c["q"], c["k"], c["v"], c["p"], c.get("pmask"))
            dqkv = np.concatenate([_merge_heads(t) for t in (dq, dk, dv)], axis=-1)
            if on:
                G[p + "w_qkv"] = _rows(dqkv).T @ _rows(c["xin"])
                G[p + "b_qkv"] = _rows(dqkv).sum(axis=0)
            if not need_dx:
                return G
            dx = dy + dqkv @ P[p + "w_qkv"]
        else:
            cos, sin = cache["rope"]
            dfo = dx * c["mask_f"]
            ds = dfo @ P[p + "w_down"]
            if on:
                G[p + "w_down"] = _rows(dfo).T @ _rows(c["s"])
            dgate, dup = swiglu_bwd(ds, c["gate"], c["up"])
            dgu = np.concatenate([dgate, dup], axis=-1)
            dh2 = dgu @ P[p + "w_gu"]
            if on:
                G[p + "w_gu"] = _rows(dgu).T @ _rows(c["h2"])
            dn, dg = rmsnorm_bwd(dh2, c["rms2"], P[p + "rms2_g"])
            if on:
                G[p + "rms2_g"] = dg
            dx2 = dx + dn
            dao = dx2 * c["mask_a"]
            dom = dao @ P[p + "w_o"]
            if on:
                G[p + "w_o"] = _rows(dao).T @ _rows(c["om"])
            dq, dk, dv = attention_bwd(_split_heads(dom, H), c["q"], c["k"], c["v"], c["p"], c.get("pmask"))
            dq = rope_apply(dq, cos, sin, inverse=True)
            dk = rope_apply(dk, cos, sin, inverse=True)
            dqkv = np.concatenate([_merge_heads(t) for t in (dq, dk, dv)], axis=-1)
            dh1 = dqkv @ P[p + "w_qkv"]
            if on:
                G[p + "w_qkv"] = _rows(dqkv).T @ _rows(c["h1"])
            dn, dg = rmsnorm_bwd(dh1, c["rms1"], P[p + "rms1_g"])
            if on:
                G[p + "rms1_g"] = dg
            if not need_dx:
                return G
            dx = dx2 + dn
    # ---- embedding ----
    if 0 in act:
        dx = dx * cache["mask_emb"]
        if cfg.arch == 1:
            dx, dg, db = layernorm_bwd(dx, cache["emb_ln"], P["emb_ln_g"])
            G["emb_ln_g"], G["emb_ln_b"] = dg, db
        gt = np.zeros_like(P["tok_emb"], dtype=F64)
        np.add.at(gt, tokens.reshape(-1), _rows(dx))
        G["tok_emb"] = G.get("tok_emb", 0.0) + gt
        if cfg.arch in (0, 1):
            gp = np.zeros_like(P["pos_emb"], dtype=F64)
            gp[:S] = dx.sum(axis=0)
            G["pos_emb"] = gp
    return G


# --------------------------------------------------------------------------
# Optimizers (textbook forms; the paper cites them without formulas)
# --------------------------------------------------------------------------
def adamw_update(theta, g, m, v, lr, beta1, beta2, eps, wd, tau):
    """Loshchilov & Hutter AdamW, update count tau >= 1.  Returns theta, m, v."""
    theta = theta * (1.0 - lr * wd)
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** tau)
    vhat = v / (1.0 - beta2 ** tau)
    theta = theta - lr * mhat / (np.sqrt(vhat) + eps)
    return theta, m, v


def adagrad_update(theta, g, acc, lr, eps):
    """Duchi et al. AdaGrad: acc += g^2; theta -= lr g / (sqrt(acc) + eps)."""
    acc = acc + g * g
    theta = theta - lr * g / (np.sqrt(acc) + eps)
    return theta, acc


def sgdm_update(theta, g, buf, lr, mu):
    """Heavy-ball momentum: buf = mu buf + g (buf0 = 0); theta -= lr buf."""
    buf = mu * buf + g
    theta = theta - lr * buf
    return theta, buf


def sgd_update(theta, g, lr):
    """Plain stochastic gradient descent: theta -= lr g (no state; the paper's zero-traffic case)."""
    return theta - lr * g


def adafactor_update(theta, g, s0, s1, lr, eps1, wd, tau, eps2=1e-3, d=1.0, decay=-0.8):
    """Adafactor (Shazeer & Stern 2018, Algorithms 4-5) with relative step size, parameter
    scaling, update clipping and no momentum, in the form torch.optim.Adafactor gives it: eps1
    clamps the factored estimate from below (max(mean(R), eps1), max(V, eps1^2)) instead of being
    added to the squared gradient.  Matrices keep row statistics s0 = R [n] and column
    statistics s1 = C [m]; vectors keep the unfactored second moment in s0.  Returns theta, s0, s1."""
    w = float(tau) ** decay                                   # 1 - beta2_t
    rho = min(lr, 1.0 / math.sqrt(tau))
    alpha = max(eps2, math.sqrt(float((theta * theta).mean()))) * rho
    theta = theta * (1.0 - lr * wd)
    if g.ndim > 1:
        s0 = s0 + w * ((g * g).mean(axis=-1) - s0)
        s1 = s1 + w * ((g * g).mean(axis=-2) - s1)
        vhat = np.outer(s0, s1) / max(float(s0.mean()), eps1)
    else:
        s0 = s0 + w * (g * g - s0)
        vhat = s0
    u = g / np.sqrt(np.maximum(vhat, eps1 * eps1))
    u = u / max(1.0, math.sqrt(float((u * u).mean())) / d)
    return theta - alpha * u, s0, s1


# --------------------------------------------------------------------------
# The training step (Algorithm 1)
# --------------------------------------------------------------------------
class HiFTOracle:
    """Holds fp64 master parameters and optimizer state for every group and
    performs Algorithm 1 one step at a time."""

    def __init__(self, cfg, gcfg, ocfg, params_fp32: Dict[str, np.ndarray]):
        self.cfg, self.gcfg, self.ocfg = cfg, gcfg, ocfg
        self.master = {k: np.array(v, dtype=F64) for k, v in params_fp32.items()}
        self.s0 = {k: np.zeros_like(v) for k, v in self.master.items()}
        self.s1 = {k: np.zeros_like(v) for k, v in self.master.items()}
        self.groups = build_groups(cfg.n_units, gcfg.layers_per_group, gcfg.split_emb_head,
                                   getattr(gcfg, "group_sizes", ()))
        self.k = len(self.groups)
        self.order = group_order(self.k, gcfg.order, gcfg.order_seed)
        self.t = 0
        self.tau = [0] * self.k
        self.last_grads: Dict[str, np.ndarray] = {}
        # Algorithm 1 c-d taken literally: when m does not divide n the sets popped from the queue drift, so the
        # update count (Adam's bias correction) belongs to the unit, and a "group" id is the position in the
        # period of the walk.  k (learning-rate cycle) stays floor(n / m) + 1.
        n, m = cfg.n_units, gcfg.layers_per_group
        self.drifting = bool(getattr(gcfg, "literal_queue", 0)) and not getattr(gcfg, "group_sizes", ()) \
            and not gcfg.split_emb_head and n % m != 0 and m < n
        if self.drifting:
            self.n_sets = n // math.gcd(n, m)
            self.groups = [sorted(e) for e in queue_walk(n, m, gcfg.order, self.n_sets, gcfg.order_seed)]
            self.order = list(range(self.n_sets))
            self.tau = [0] * n                                  # per unit

    def active_group(self) -> int:
        if self.drifting:
            return self.t % self.n_sets
        return self.order[self.t % self.k]

    def current_lr(self) -> float:
        o = self.ocfg
        return lr_for_cycle(o.lr, o.sched, self.t // self.k, o.total_cycles, getattr(o, "warmup_cycles", 0))

    def model_params(self) -> Dict[str, np.ndarray]:
        """What the forward pass reads: the master itself (fp32 configs) or its
        bf16 rounding (mixed-precision configs), as exact fp64 values."""
        if self.cfg.dtype == 1:
            return {k: bf16_round(v.astype(np.float32)).astype(F64) for k, v in self.master.items()}
        return self.master

    def unit_of(self, name: str) -> int:
        for u in range(self.cfg.n_units):
            if name in tensor_names_of_unit(self.cfg, u):
                return u
        raise KeyError(name)

    def tau_of(self, name: str, g: int) -> int:
        """Updates the tensor has had (its unit's count under the drifting queue, else its group's)."""
        return self.tau[self.unit_of(name)] if self.drifting else self.tau[g]

    def group_tensor_names(self, g: int) -> List[str]:
        return [n for u in self.groups[g] for n in tensor_names_of_unit(self.cfg, u)]

    def step(self, tokens: np.ndarray, labels: np.ndarray, lens=None) -> float:
        g = self.active_group()
        lr = self.current_lr()
        P = self.model_params()
        pdrop, padrop = float(getattr(self.cfg, "dropout", 0.0)), float(getattr(self.cfg, "attn_dropout", 0.0))
        drop = (pdrop, int(getattr(self.cfg, "dropout_seed", 0)), self.t, padrop) if max(pdrop, padrop) > 0.0 else None
        loss, cache = forward(self.cfg, P, tokens, labels, lens, drop)
        grads = backward(self.cfg, P, cache, active_units=self.groups[g])
        o = self.ocfg
        if self.drifting:
            for u in self.groups[g]:
                self.tau[u] += 1
        else:
            self.tau[g] += 1
        for name in self.group_tensor_names(g):
            gr = grads[name]
            tau = self.tau[self.unit_of(name)] if self.drifting else self.tau[g]
            if o.kind == 0:
                self.master[name], self.s0[name], self.s1[name] = adamw_update(
                    self.master[name], gr, self.s0[name], self.s1[name],
                    lr, o.beta1, o.beta2, o.eps, o.weight_decay, tau)
            elif o.kind == 1:
                self.master[name], self.s0[name] = adagrad_update(
                    self.master[name], gr, self.s0[name], lr, o.eps)
            elif o.kind == 2:
                self.master[name], self.s0[name] = sgdm_update(
                    self.master[name], gr, self.s0[name], lr, o.momentum)
            elif o.kind == 3:
                self.master[name] = sgd_update(self.master[name], gr, lr)
            else:
                if tau == 1:                                  # factored state has its own shapes
                    m = self.master[name]
                    self.s0[name] = np.zeros(m.shape[0]) if m.ndim > 1 else np.zeros_like(m)
                    self.s1[name] = np.zeros(m.shape[1]) if m.ndim > 1 else np.zeros(0)
                self.master[name], self.s0[name], self.s1[name] = adafactor_update(
                    self.master[name], gr, self.s0[name], self.s1[name], lr, o.eps, o.weight_decay, tau)
        self.last_grads = grads
        self.t += 1
        return loss
