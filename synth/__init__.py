"""Seeded synthetic inputs for the hierarchical fine-tuning (HiFT) step.

This module only *describes and draws inputs*: model shapes, parameter tensor
names and shapes, initial weights, token ids, labels and flat gradients.  It
holds none of the method's arithmetic (no forward, backward, schedule or
optimizer code), so both the CPU oracle and the CUDA library can be fed from it
without sharing any computation.

Workload recipe (stands in for the paper's CoLA / E2E batches, which are used
only for their shapes):
  * token ids: uniform over the vocabulary, or Zipf(s) with P(id = r-1) ~ r^-s,
    r = 1..V, drawn by inverse CDF on an fp64 cumulative table;
  * causal-LM labels: S+1 ids per row, tokens = first S, labels = last S;
  * classifier labels: Bernoulli(0.5);
  * weights N(0, init_std^2), biases 0, norm gains 1;
  * flat gradients N(0, (1e-3)^2).
"""
from __future__ import annotations

from dataclasses import dataclass, asdict, replace
from typing import Dict, List, Tuple

import numpy as np

ARCH_PRELN_GPT = 0      # pre-LayerNorm causal decoder, learned positions, GELU
ARCH_POSTLN_ENC = 1     # post-LayerNorm bidirectional encoder + classifier on token 0
ARCH_LLAMA = 2          # RMSNorm, RoPE, SwiGLU, no biases

DTYPE_FP32 = 0          # fp32 parameters and activations
DTYPE_BF16 = 1          # bf16 parameters/activations with fp32 master weights

OPT_ADAMW, OPT_ADAGRAD, OPT_SGDM, OPT_SGD, OPT_ADAFACTOR = 0, 1, 2, 3, 4
ORDER_BOTTOM2UP, ORDER_TOP2DOWN, ORDER_RANDOM = 0, 1, 2
SCHED_CONST, SCHED_LINEAR = 0, 1


@dataclass(frozen=True)
class ModelCfg:
    arch: int
    n_blocks: int
    d_model: int
    n_heads: int
    d_ffn: int
    vocab: int
    max_pos: int = 0
    n_classes: int = 0
    causal: int = 1
    tie_head: int = 0
    norm_eps: float = 1e-5
    rope_base: float = 10000.0
    init_std: float = 0.02
    dtype: int = DTYPE_BF16
    batch: int = 1
    seq: int = 1
    dropout: float = 0.0               # probability of dropping an element at the residual-branch outputs and the embedding output
    dropout_seed: int = 0
    attn_dropout: float = 0.0          # probability of dropping an attention probability (after the softmax)

    @property
    def n_units(self) -> int:
        return self.n_blocks + 2

    @property
    def tokens_per_step(self) -> int:
        return self.batch * self.seq

    def scaled(self, **kw) -> "ModelCfg":
        return replace(self, **kw)

    def as_dict(self):
        return asdict(self)


@dataclass(frozen=True)
class GroupCfg:
    layers_per_group: int = 1          # m
    split_emb_head: int = 0            # 1: embedding | blocks in chunks of m | head
    order: int = ORDER_BOTTOM2UP
    order_seed: int = 0
    group_sizes: tuple = ()            # non-empty: consecutive units per group, bottom first (overrides m)
    literal_queue: int = 0             # 1: pop m units from a queue per step (sets drift when m does not divide n)


@dataclass(frozen=True)
class OptCfg:
    kind: int = OPT_ADAMW
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.0
    momentum: float = 0.9
    sched: int = SCHED_CONST
    total_cycles: int = 1
    offload_state: int = 1
    prefetch_groups: int = 0
    warmup_cycles: int = 0
    recompute: int = 0
    shard_rank: int = 0                # optimizer state sharded over data-parallel ranks (0 / 1 = off)
    shard_world: int = 0
    grad_bf16: int = 0                 # 1: the active group's gradient is kept in bf16


# --------------------------------------------------------------------------
# Named workloads (shapes only)
# --------------------------------------------------------------------------
def config_tiny_fp32() -> Tuple[ModelCfg, GroupCfg, OptCfg]:
    m = ModelCfg(arch=ARCH_PRELN_GPT, n_blocks=4, d_model=128, n_heads=4, d_ffn=512,
                 vocab=512, max_pos=32, causal=1, tie_head=1, norm_eps=1e-5,
                 dtype=DTYPE_FP32, batch=2, seq=32)
    g = GroupCfg(layers_per_group=1, split_emb_head=0, order=ORDER_BOTTOM2UP)
    o = OptCfg(kind=OPT_ADAMW, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8,
               weight_decay=0.01, sched=SCHED_CONST, total_cycles=1)
    return m, g, o


def config_roberta_base() -> Tuple[ModelCfg, GroupCfg, OptCfg]:
    m = ModelCfg(arch=ARCH_POSTLN_ENC, n_blocks=12, d_model=768, n_heads=12, d_ffn=3072,
                 vocab=50265, max_pos=512, n_classes=2, causal=0, tie_head=0,
                 norm_eps=1e-5, dtype=DTYPE_BF16, batch=16, seq=128)
    g = GroupCfg(layers_per_group=1, split_emb_head=0, order=ORDER_TOP2DOWN)
    o = OptCfg(kind=OPT_ADAMW, lr=2e-5, weight_decay=0.0, sched=SCHED_LINEAR, total_cycles=3)
    return m, g, o


def config_gpt2_large(opt_kind: int = OPT_SGDM) -> Tuple[ModelCfg, GroupCfg, OptCfg]:
    m = ModelCfg(arch=ARCH_PRELN_GPT, n_blocks=36, d_model=1280, n_heads=20, d_ffn=5120,
                 vocab=50257, max_pos=1024, causal=1, tie_head=1, norm_eps=1e-5,
                 dtype=DTYPE_BF16, batch=8, seq=512)
    g = GroupCfg(layers_per_group=2, split_emb_head=1, order=ORDER_RANDOM, order_seed=2401)
    if opt_kind == OPT_SGDM:
        o = OptCfg(kind=OPT_SGDM, lr=1e-3, momentum=0.9)
    else:
        o = OptCfg(kind=OPT_ADAGRAD, lr=1e-2, eps=1e-10)
    return m, g, o


def config_llama_7b() -> Tuple[ModelCfg, GroupCfg, OptCfg]:
    m = ModelCfg(arch=ARCH_LLAMA, n_blocks=32, d_model=4096, n_heads=32, d_ffn=11008,
                 vocab=32000, max_pos=0, causal=1, tie_head=0, norm_eps=1e-6,
                 rope_base=10000.0, dtype=DTYPE_BF16, batch=4, seq=512)
    g = GroupCfg(layers_per_group=1, split_emb_head=0, order=ORDER_BOTTOM2UP)
    o = OptCfg(kind=OPT_ADAMW, lr=1e-5, weight_decay=0.0, offload_state=1)
    return m, g, o


# --------------------------------------------------------------------------
# Parameter tensors: names, shapes and how they are initialised
# --------------------------------------------------------------------------
def unit_tensors(cfg: ModelCfg) -> List[List[Tuple[str, Tuple[int, ...], str]]]:
    """Per unit (embedding, block 0..L-1, head): list of (name, shape, init)."""
    d, f, V = cfg.d_model, cfg.d_ffn, cfg.vocab
    units: List[List[Tuple[str, Tuple[int, ...], str]]] = []
    emb = [("tok_emb", (V, d), "normal")]
    if cfg.arch in (ARCH_PRELN_GPT, ARCH_POSTLN_ENC):
        emb.append(("pos_emb", (cfg.max_pos, d), "normal"))
    if cfg.arch == ARCH_POSTLN_ENC:
        emb += [("emb_ln_g", (d,), "ones"), ("emb_ln_b", (d,), "zeros")]
    units.append(emb)
    for i in range(cfg.n_blocks):
        p = f"b{i}."
        if cfg.arch == ARCH_LLAMA:
            blk = [(p + "rms1_g", (d,), "ones"), (p + "w_qkv", (3 * d, d), "normal"),
                   (p + "w_o", (d, d), "normal"), (p + "rms2_g", (d,), "ones"),
                   (p + "w_gu", (2 * f, d), "normal"), (p + "w_down", (d, f), "normal")]
        else:
            blk = [(p + "ln1_g", (d,), "ones"), (p + "ln1_b", (d,), "zeros"),
                   (p + "w_qkv", (3 * d, d), "normal"), (p + "b_qkv", (3 * d,), "zeros"),
                   (p + "w_o", (d, d), "normal"), (p + "b_o", (d,), "zeros"),
                   (p + "ln2_g", (d,), "ones"), (p + "ln2_b", (d,), "zeros"),
                   (p + "w_fc1", (f, d), "normal"), (p + "b_fc1", (f,), "zeros"),
                   (p + "w_fc2", (d, f), "normal"), (p + "b_fc2", (d,), "zeros")]
        units.append(blk)
    if cfg.arch == ARCH_POSTLN_ENC:
        head = [("w_cls", (cfg.n_classes, d), "normal"), ("b_cls", (cfg.n_classes,), "zeros")]
    elif cfg.arch == ARCH_LLAMA:
        head = [("rmsf_g", (d,), "ones")]
        if not cfg.tie_head:
            head.append(("w_head", (V, d), "normal"))
    else:
        head = [("lnf_g", (d,), "ones"), ("lnf_b", (d,), "zeros")]
        if not cfg.tie_head:
            head.append(("w_head", (V, d), "normal"))
    units.append(head)
    return units


def count_params(cfg: ModelCfg) -> List[int]:
    return [sum(int(np.prod(s)) for _, s, _ in u) for u in unit_tensors(cfg)]


def init_params(cfg: ModelCfg, seed: int, perturb: float = 0.0) -> Dict[str, np.ndarray]:
    """fp32 initial weights.  `perturb` > 0 adds N(0, perturb^2) noise to the
    biases and gains too, so that tests do not sit on the symmetric point
    (bias 0, gain 1) where some mistakes stay hidden."""
    rng = np.random.Generator(np.random.PCG64(seed))
    out: Dict[str, np.ndarray] = {}
    for unit in unit_tensors(cfg):
        for name, shape, kind in unit:
            if kind == "normal":
                a = rng.standard_normal(shape, dtype=np.float32) * np.float32(cfg.init_std)
            elif kind == "ones":
                a = np.ones(shape, dtype=np.float32)
            else:
                a = np.zeros(shape, dtype=np.float32)
            if perturb > 0.0 and kind != "normal":
                a = a + rng.standard_normal(shape, dtype=np.float32) * np.float32(perturb)
            out[name] = np.ascontiguousarray(a, dtype=np.float32)
    return out


# --------------------------------------------------------------------------
# Token ids and labels
# --------------------------------------------------------------------------
def _zipf_cdf(vocab: int, s: float) -> np.ndarray:
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
    c = np.cumsum(w)
    return c / c[-1]


def draw_ids(rng: np.random.Generator, shape, vocab: int, dist: str, s: float = 1.1) -> np.ndarray:
    if dist == "uniform":
        return rng.integers(0, vocab, size=shape, dtype=np.int64).astype(np.int32)
    if dist == "zipf":
        u = rng.random(size=shape)
        ids = np.searchsorted(_zipf_cdf(vocab, s), u, side="left")
        return np.minimum(ids, vocab - 1).astype(np.int32)
    raise ValueError(dist)


def lm_batch(cfg: ModelCfg, seed: int, step: int, dist: str = "zipf") -> Tuple[np.ndarray, np.ndarray]:
    """Next-token batch for step `step`: tokens [B,S] int32, labels [B,S] int32."""
    rng = np.random.Generator(np.random.PCG64([seed, 1000 + step]))
    ids = draw_ids(rng, (cfg.batch, cfg.seq + 1), cfg.vocab, dist)
    return np.ascontiguousarray(ids[:, :-1]), np.ascontiguousarray(ids[:, 1:])


def cls_batch(cfg: ModelCfg, seed: int, step: int, dist: str = "zipf") -> Tuple[np.ndarray, np.ndarray]:
    """Sequence-classification batch: tokens [B,S] int32, labels [B] int32 ~ Bernoulli(0.5)."""
    rng = np.random.Generator(np.random.PCG64([seed, 1000 + step]))
    ids = draw_ids(rng, (cfg.batch, cfg.seq), cfg.vocab, dist)
    labels = rng.integers(0, cfg.n_classes, size=(cfg.batch,), dtype=np.int64).astype(np.int32)
    return ids, labels


def batch_for(cfg: ModelCfg, seed: int, step: int, dist: str = "zipf"):
    if cfg.arch == ARCH_POSTLN_ENC:
        return cls_batch(cfg, seed, step, dist)
    return lm_batch(cfg, seed, step, dist)


# --------------------------------------------------------------------------
# Flat buffers for the optimizer sweep
# --------------------------------------------------------------------------
def flat_optimizer_inputs(n: int, seed: int, warm: bool = False):
    """master ~ N(0, 0.02^2), grad ~ N(0, (1e-3)^2); states zero, or a plausible
    warm state (first moment ~ grad scale, second moment/accumulator >= 0)."""
    rng = np.random.Generator(np.random.PCG64([seed, 77]))
    master = rng.standard_normal(n, dtype=np.float32) * np.float32(0.02)
    grad = rng.standard_normal(n, dtype=np.float32) * np.float32(1e-3)
    if warm:
        s0 = rng.standard_normal(n, dtype=np.float32) * np.float32(1e-3)
        s1 = (rng.standard_normal(n, dtype=np.float32) * np.float32(1e-3)) ** 2
    else:
        s0 = np.zeros(n, dtype=np.float32)
        s1 = np.zeros(n, dtype=np.float32)
    return master, grad, s0, s1
