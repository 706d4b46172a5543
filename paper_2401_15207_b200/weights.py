"""Weight files: the library's own container (read by hift_load_weights) and a converter from
checkpoints in the safetensors layout with the tensor names the public LLaMA, GPT-2 and RoBERTa
checkpoints use.

Host-side file handling only: nothing here touches the GPU or does any of the method's arithmetic.

Container ("HIFTWTS1"): magic[8] | uint32 n | n records of { char name[64] | uint32 dtype (0 fp32,
1 bf16) | uint64 rows | uint64 cols | rows*cols elements }.  Names and shapes are those
hift_tensor_info reports (a vector has rows = 1; linear weights are [out_features, in_features]).
"""
from __future__ import annotations

import json
import struct
from typing import Dict, Tuple

import numpy as np

MAGIC = b"HIFTWTS1"


def write_weights(path: str, tensors: Dict[str, np.ndarray], bf16: bool = False) -> None:
    """tensors: name -> array (1-D arrays are stored as [1, n]).  bf16=True stores the upper 16 bits of
    every value after round-to-nearest-even (half the file size; what a bf16 checkpoint holds)."""
    with open(path, "wb") as f:
        f.write(MAGIC)
        f.write(struct.pack("<I", len(tensors)))
        for name, a in tensors.items():
            a = np.ascontiguousarray(a, dtype=np.float32)
            rows, cols = (1, a.size) if a.ndim == 1 else (a.shape[0], int(np.prod(a.shape[1:])))
            nm = name.encode()
            if len(nm) > 63:
                raise ValueError(f"tensor name too long: {name}")
            f.write(nm.ljust(64, b"\0"))
            f.write(struct.pack("<IQQ", 1 if bf16 else 0, rows, cols))
            if bf16:
                u = a.reshape(-1).view(np.uint32).astype(np.uint64)
                u = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
                f.write(u.tobytes())
            else:
                f.write(a.tobytes())


def read_weights(path: str) -> Dict[str, np.ndarray]:
    out = {}
    with open(path, "rb") as f:
        if f.read(8) != MAGIC:
            raise ValueError("not a HIFTWTS1 file")
        (n,) = struct.unpack("<I", f.read(4))
        for _ in range(n):
            name = f.read(64).split(b"\0")[0].decode()
            dtype, rows, cols = struct.unpack("<IQQ", f.read(20))
            if dtype == 1:
                u = np.frombuffer(f.read(rows * cols * 2), dtype=np.uint16).astype(np.uint32) << 16
                out[name] = u.view(np.float32).reshape(rows, cols)
            else:
                out[name] = np.frombuffer(f.read(rows * cols * 4), dtype=np.float32).reshape(rows, cols)
    return out


_ST_DTYPES = {"F32": (np.float32, 4), "F16": (np.float16, 2), "BF16": (np.uint16, 2), "F64": (np.float64, 8)}


def read_safetensors(path: str) -> Dict[str, np.ndarray]:
    """Minimal reader of the safetensors layout (8-byte little-endian header length, a JSON header
    mapping names to dtype / shape / data_offsets, then the raw data): fp32 arrays out."""
    with open(path, "rb") as f:
        (hlen,) = struct.unpack("<Q", f.read(8))
        header = json.loads(f.read(hlen).decode())
        base = 8 + hlen
        out = {}
        for name, meta in header.items():
            if name == "__metadata__":
                continue
            np_dtype, size = _ST_DTYPES[meta["dtype"]]
            lo, hi = meta["data_offsets"]
            f.seek(base + lo)
            raw = np.frombuffer(f.read(hi - lo), dtype=np_dtype)
            if meta["dtype"] == "BF16":
                raw = (raw.astype(np.uint32) << 16).view(np.float32)
            out[name] = raw.astype(np.float32).reshape(meta["shape"])
    return out


def from_checkpoint_names(arch: int, n_blocks: int, src: Dict[str, np.ndarray], max_pos: int = 0) -> Tuple[Dict[str, np.ndarray], list]:
    """Maps tensors named as in the public checkpoints of the three model families onto this library's
    tensors (fusing q | k | v and gate | up row-wise, transposing GPT-2's [in, out] matrices).
    arch 2: LLaMA names (model.layers.N.self_attn.q_proj.weight ...), rotary pairs (j, j + d_head/2) as stored;
    arch 0: GPT-2 names (h.N.attn.c_attn.weight ..., with or without a 'transformer.' prefix);
    arch 1: RoBERTa encoder names (roberta.encoder.layer.N...; the token-type row is folded into the
            position table, whose first two rows - the padding offset - are dropped).
    Returns (tensors, names of the library's tensors the checkpoint has no counterpart for)."""
    g = lambda k: np.asarray(src[k], dtype=np.float32)
    out: Dict[str, np.ndarray] = {}
    missing = []
    if arch == 2:
        out["tok_emb"] = g("model.embed_tokens.weight")
        for i in range(n_blocks):
            p, q = f"b{i}.", f"model.layers.{i}."
            out[p + "rms1_g"] = g(q + "input_layernorm.weight")
            out[p + "w_qkv"] = np.concatenate([g(q + f"self_attn.{x}_proj.weight") for x in "qkv"], axis=0)
            out[p + "w_o"] = g(q + "self_attn.o_proj.weight")
            out[p + "rms2_g"] = g(q + "post_attention_layernorm.weight")
            out[p + "w_gu"] = np.concatenate([g(q + "mlp.gate_proj.weight"), g(q + "mlp.up_proj.weight")], axis=0)
            out[p + "w_down"] = g(q + "mlp.down_proj.weight")
        out["rmsf_g"] = g("model.norm.weight")
        if "lm_head.weight" in src:
            out["w_head"] = g("lm_head.weight")
        else:
            missing.append("w_head")
    elif arch == 0:
        pre = "transformer." if any(k.startswith("transformer.") for k in src) else ""
        out["tok_emb"] = g(pre + "wte.weight")
        out["pos_emb"] = g(pre + "wpe.weight")
        for i in range(n_blocks):
            p, q = f"b{i}.", f"{pre}h.{i}."
            out[p + "ln1_g"], out[p + "ln1_b"] = g(q + "ln_1.weight"), g(q + "ln_1.bias")
            out[p + "w_qkv"], out[p + "b_qkv"] = g(q + "attn.c_attn.weight").T, g(q + "attn.c_attn.bias")
            out[p + "w_o"], out[p + "b_o"] = g(q + "attn.c_proj.weight").T, g(q + "attn.c_proj.bias")
            out[p + "ln2_g"], out[p + "ln2_b"] = g(q + "ln_2.weight"), g(q + "ln_2.bias")
            out[p + "w_fc1"], out[p + "b_fc1"] = g(q + "mlp.c_fc.weight").T, g(q + "mlp.c_fc.bias")
            out[p + "w_fc2"], out[p + "b_fc2"] = g(q + "mlp.c_proj.weight").T, g(q + "mlp.c_proj.bias")
        out["lnf_g"], out["lnf_b"] = g(pre + "ln_f.weight"), g(pre + "ln_f.bias")
    elif arch == 1:
        e = "roberta.embeddings."
        out["tok_emb"] = g(e + "word_embeddings.weight")
        pos = g(e + "position_embeddings.weight")[2:]
        if e + "token_type_embeddings.weight" in src:
            pos = pos + g(e + "token_type_embeddings.weight")[0][None, :]
        out["pos_emb"] = pos[:max_pos] if max_pos else pos
        out["emb_ln_g"], out["emb_ln_b"] = g(e + "LayerNorm.weight"), g(e + "LayerNorm.bias")
        for i in range(n_blocks):
            p, q = f"b{i}.", f"roberta.encoder.layer.{i}."
            a = q + "attention.self."
            out[p + "w_qkv"] = np.concatenate([g(a + f"{x}.weight") for x in ("query", "key", "value")], axis=0)
            out[p + "b_qkv"] = np.concatenate([g(a + f"{x}.bias") for x in ("query", "key", "value")], axis=0)
            out[p + "w_o"], out[p + "b_o"] = g(q + "attention.output.dense.weight"), g(q + "attention.output.dense.bias")
            out[p + "ln1_g"], out[p + "ln1_b"] = g(q + "attention.output.LayerNorm.weight"), g(q + "attention.output.LayerNorm.bias")
            out[p + "w_fc1"], out[p + "b_fc1"] = g(q + "intermediate.dense.weight"), g(q + "intermediate.dense.bias")
            out[p + "w_fc2"], out[p + "b_fc2"] = g(q + "output.dense.weight"), g(q + "output.dense.bias")
            out[p + "ln2_g"], out[p + "ln2_b"] = g(q + "output.LayerNorm.weight"), g(q + "output.LayerNorm.bias")
        missing += ["w_cls", "b_cls"]       # the checkpoints' two-layer classification head has no counterpart here
    else:
        raise ValueError("arch must be 0, 1 or 2")
    return {k: np.ascontiguousarray(v, dtype=np.float32) for k, v in out.items()}, missing


def convert_safetensors(src_path: str, dst_path: str, arch: int, n_blocks: int, max_pos: int = 0, bf16: bool = False) -> list:
    """safetensors checkpoint -> HIFTWTS1 container.  Returns the tensors left for the caller to initialise."""
    tensors, missing = from_checkpoint_names(arch, n_blocks, read_safetensors(src_path), max_pos)
    write_weights(dst_path, tensors, bf16=bf16)
    return missing
