"""Weight files: the container hift_load_weights reads, and the converter from checkpoints that use the
public LLaMA / GPT-2 / RoBERTa tensor names (safetensors layout, written here by hand: json header + raw data)."""
import json
import struct

import numpy as np
import pytest

import synth
from paper_2401_15207_b200 import weights as W


def _write_safetensors(path, tensors, dtype="F32"):
    header, blobs, off = {}, [], 0
    for name, a in tensors.items():
        a = np.ascontiguousarray(a, dtype=np.float32)
        if dtype == "BF16":
            raw = (a.reshape(-1).view(np.uint32) >> 16).astype(np.uint16).tobytes()
        else:
            raw = a.tobytes()
        header[name] = {"dtype": dtype, "shape": list(a.shape), "data_offsets": [off, off + len(raw)]}
        blobs.append(raw)
        off += len(raw)
    h = json.dumps(header).encode()
    with open(path, "wb") as f:
        f.write(struct.pack("<Q", len(h)))
        f.write(h)
        for b in blobs:
            f.write(b)


def _llama_checkpoint(cfg, p):
    d, f = cfg.d_model, cfg.d_ffn
    src = {"model.embed_tokens.weight": p["tok_emb"], "model.norm.weight": p["rmsf_g"], "lm_head.weight": p["w_head"]}
    for i in range(cfg.n_blocks):
        q, b = f"model.layers.{i}.", f"b{i}."
        src[q + "input_layernorm.weight"] = p[b + "rms1_g"]
        for j, x in enumerate("qkv"):
            src[q + f"self_attn.{x}_proj.weight"] = p[b + "w_qkv"][j * d:(j + 1) * d]
        src[q + "self_attn.o_proj.weight"] = p[b + "w_o"]
        src[q + "post_attention_layernorm.weight"] = p[b + "rms2_g"]
        src[q + "mlp.gate_proj.weight"], src[q + "mlp.up_proj.weight"] = p[b + "w_gu"][:f], p[b + "w_gu"][f:]
        src[q + "mlp.down_proj.weight"] = p[b + "w_down"]
    return src


def _gpt2_checkpoint(cfg, p):
    src = {"wte.weight": p["tok_emb"], "wpe.weight": p["pos_emb"], "ln_f.weight": p["lnf_g"], "ln_f.bias": p["lnf_b"]}
    for i in range(cfg.n_blocks):
        q, b = f"h.{i}.", f"b{i}."
        src[q + "ln_1.weight"], src[q + "ln_1.bias"] = p[b + "ln1_g"], p[b + "ln1_b"]
        src[q + "attn.c_attn.weight"], src[q + "attn.c_attn.bias"] = p[b + "w_qkv"].T, p[b + "b_qkv"]     # [in, out] on file
        src[q + "attn.c_proj.weight"], src[q + "attn.c_proj.bias"] = p[b + "w_o"].T, p[b + "b_o"]
        src[q + "ln_2.weight"], src[q + "ln_2.bias"] = p[b + "ln2_g"], p[b + "ln2_b"]
        src[q + "mlp.c_fc.weight"], src[q + "mlp.c_fc.bias"] = p[b + "w_fc1"].T, p[b + "b_fc1"]
        src[q + "mlp.c_proj.weight"], src[q + "mlp.c_proj.bias"] = p[b + "w_fc2"].T, p[b + "b_fc2"]
    return src


def _mini(arch):
    return synth.ModelCfg(arch=arch, n_blocks=2, d_model=64, n_heads=4, d_ffn=128, vocab=203, max_pos=48,
                          causal=1, tie_head=1 if arch == 0 else 0, norm_eps=1e-6 if arch == 2 else 1e-5,
                          dtype=synth.DTYPE_BF16, batch=2, seq=40, init_std=0.08)


@pytest.mark.parametrize("arch", [0, 2])
def test_checkpoint_names_map_onto_the_fused_tensors(arch, tmp_path):
    cfg = _mini(arch)
    p = synth.init_params(cfg, 3, perturb=0.1)
    src = (_llama_checkpoint if arch == 2 else _gpt2_checkpoint)(cfg, p)
    st, out = str(tmp_path / "m.safetensors"), str(tmp_path / "m.hift")
    _write_safetensors(st, src)
    missing = W.convert_safetensors(st, out, arch, cfg.n_blocks)
    assert missing == []
    back = W.read_weights(out)
    assert sorted(back) == sorted(p)
    for n in p:
        assert np.array_equal(back[n].reshape(p[n].shape), p[n]), n


def test_roberta_names_fold_token_type_and_drop_the_padding_offset():
    cfg = synth.ModelCfg(arch=1, n_blocks=1, d_model=16, n_heads=2, d_ffn=32, vocab=50, max_pos=8, n_classes=2, causal=0,
                         dtype=synth.DTYPE_BF16, batch=1, seq=8)
    p = synth.init_params(cfg, 1, perturb=0.1)
    rng = np.random.default_rng(0)
    tt = rng.standard_normal((1, 16)).astype(np.float32)
    pos_file = np.concatenate([rng.standard_normal((2, 16)).astype(np.float32), p["pos_emb"] - tt], axis=0)
    e, q, b = "roberta.embeddings.", "roberta.encoder.layer.0.", "b0."
    src = {e + "word_embeddings.weight": p["tok_emb"], e + "position_embeddings.weight": pos_file,
           e + "token_type_embeddings.weight": tt, e + "LayerNorm.weight": p["emb_ln_g"], e + "LayerNorm.bias": p["emb_ln_b"],
           q + "attention.output.dense.weight": p[b + "w_o"], q + "attention.output.dense.bias": p[b + "b_o"],
           q + "attention.output.LayerNorm.weight": p[b + "ln1_g"], q + "attention.output.LayerNorm.bias": p[b + "ln1_b"],
           q + "intermediate.dense.weight": p[b + "w_fc1"], q + "intermediate.dense.bias": p[b + "b_fc1"],
           q + "output.dense.weight": p[b + "w_fc2"], q + "output.dense.bias": p[b + "b_fc2"],
           q + "output.LayerNorm.weight": p[b + "ln2_g"], q + "output.LayerNorm.bias": p[b + "ln2_b"]}
    for j, x in enumerate(("query", "key", "value")):
        src[q + f"attention.self.{x}.weight"] = p[b + "w_qkv"][j * 16:(j + 1) * 16]
        src[q + f"attention.self.{x}.bias"] = p[b + "b_qkv"][j * 16:(j + 1) * 16]
    out, missing = W.from_checkpoint_names(1, 1, src, max_pos=8)
    assert missing == ["w_cls", "b_cls"]
    for n in out:
        assert np.allclose(out[n].reshape(p[n].shape), p[n], atol=1e-6), n


def test_bf16_container_rounds_to_nearest_even(tmp_path):
    a = np.array([1.0, 1.00390625, 1.01171875, -3.0e-5, 65504.0], dtype=np.float32)     # 1 + 2^-8 is a tie: stays 1.0
    path = str(tmp_path / "b.hift")
    W.write_weights(path, {"v": a}, bf16=True)
    from oracle import hift_oracle as O
    assert np.array_equal(W.read_weights(path)["v"].reshape(-1), O.bf16_round(a))


@pytest.mark.gpu
@pytest.mark.parametrize("arch,bf16", [(2, False), (0, False), (2, True)])
def test_load_weights_sets_master_and_model_copy(arch, bf16, tmp_path):
    import torch
    from paper_2401_15207_b200 import HiFT, HiftError
    cfg = _mini(arch)
    p = synth.init_params(cfg, 3, perturb=0.1)
    path = str(tmp_path / "w.hift")
    W.write_weights(path, p, bf16=bf16)
    gc, oc = synth.GroupCfg(1), synth.OptCfg(kind=0, lr=1e-3, offload_state=1, prefetch_groups=2)
    a, b = HiFT(cfg, gc, oc), HiFT(cfg, gc, oc)
    try:
        from oracle import hift_oracle as O
        expect = {n: (O.bf16_round(v) if bf16 else v) for n, v in p.items()}
        a.set_params(expect)
        assert b.load_weights(path) == len(p)
        for n in p:
            assert np.array_equal(a.get_param(n), b.get_param(n)), n
            assert np.array_equal(a.get_model_param(n), b.get_model_param(n)), n
        tok, lab = synth.lm_batch(cfg, 1, 0)
        tt, ll = torch.from_numpy(tok).cuda(), torch.from_numpy(lab).cuda()
        assert a.step(tt, ll) == b.step(tt, ll)
        # a file that lacks a tensor: fine unless strict; a foreign tensor or shape: refused
        part = {n: v for n, v in p.items() if n != "b0.w_o"}
        W.write_weights(path, part)
        assert b.load_weights(path, strict=False) == len(part)
        with pytest.raises(HiftError) as e:
            b.load_weights(path, strict=True)
        assert e.value.status == 4
        W.write_weights(path, {"b0.w_o": p["b0.w_o"][:, :-8]})
        with pytest.raises(HiftError):
            b.load_weights(path, strict=False)
        W.write_weights(path, {"no_such_tensor": np.zeros(4, np.float32)})
        with pytest.raises(HiftError):
            b.load_weights(path, strict=False)
        with pytest.raises(HiftError):
            b.load_weights(str(tmp_path / "missing.hift"))
    finally:
        a.close()
        b.close()
