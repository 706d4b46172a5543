"""ctypes binding of include/hift.h: same names, argument marshalling only.

torch is used for device memory (tensors whose data_ptr() is handed to the
library) and for the CUDA stream; nothing is computed in Python.  There is no
CPU fallback: if libhift.so is missing or no CUDA device is present the calls
raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libhift.so")
_lib = None

KERNEL_CLASSES = ["gemm_fwd", "gemm_dx", "gemm_dw", "attn_fwd", "attn_bwd", "norm", "elementwise",
                  "cross_entropy", "embedding", "optimizer", "reduce"]

STATUS_NAMES = {0: "HIFT_OK", 1: "HIFT_ERR_CFG", 2: "HIFT_ERR_OOM_DEVICE", 3: "HIFT_ERR_OOM_PINNED",
                4: "HIFT_ERR_INPUT", 5: "HIFT_ERR_NONFINITE", 6: "HIFT_ERR_TIMEOUT", 7: "HIFT_ERR_CUDA",
                8: "HIFT_ERR_CAPACITY"}
STATIC_SCRATCH_MAX_COLS = 8192


class HiftError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().hift_strerror(status).decode() if _lib is not None else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({msg})")


class ModelCfgC(C.Structure):
    _fields_ = [("arch", C.c_int32), ("n_blocks", C.c_int32), ("d_model", C.c_int32),
                ("n_heads", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32),
                ("max_pos", C.c_int32), ("n_classes", C.c_int32), ("causal", C.c_int32),
                ("tie_head", C.c_int32), ("dtype", C.c_int32), ("batch", C.c_int32),
                ("seq", C.c_int32), ("norm_eps", C.c_double), ("rope_base", C.c_double),
                ("dropout", C.c_double), ("dropout_seed", C.c_uint64), ("attn_dropout", C.c_double)]


class GroupCfgC(C.Structure):
    _fields_ = [("layers_per_group", C.c_int32), ("split_emb_head", C.c_int32),
                ("order", C.c_int32), ("order_seed", C.c_uint64),
                ("group_sizes", C.POINTER(C.c_int32)), ("n_group_sizes", C.c_int32),
                ("literal_queue", C.c_int32)]


class OptCfgC(C.Structure):
    _fields_ = [("kind", C.c_int32), ("sched", C.c_int32), ("total_cycles", C.c_int32),
                ("offload_state", C.c_int32), ("prefetch_groups", C.c_int32), ("recompute", C.c_int32), ("warmup_cycles", C.c_int32),
                ("shard_rank", C.c_int32), ("shard_world", C.c_int32), ("grad_bf16", C.c_int32),
                ("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double),
                ("eps", C.c_double), ("weight_decay", C.c_double), ("momentum", C.c_double)]


# name -> (restype, argtypes); mirrors include/hift.h one to one
def _prototypes():
    vp, i32, i64, f64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_double, C.c_size_t
    pf = C.POINTER(C.c_float)
    return {
        "hift_strerror": (C.c_char_p, [C.c_int]),
        "hift_create": (C.c_int, [C.POINTER(ModelCfgC), C.POINTER(GroupCfgC), C.POINTER(OptCfgC), vp, C.POINTER(vp)]),
        "hift_destroy": (None, [vp]),
        "hift_step": (C.c_int, [vp, vp, vp, pf]),
        "hift_step_host": (C.c_int, [vp, vp, vp, pf]),
        "hift_set_key_lengths": (C.c_int, [vp, vp]),
        "hift_step_begin": (C.c_int, [vp, vp, vp, pf]),
        "hift_grad_view": (C.c_int, [vp, C.POINTER(vp), C.POINTER(sz)]),
        "hift_grad_elem_bytes": (i32, [vp]),
        "hift_step_end": (C.c_int, [vp]),
        "hift_step_abort": (C.c_int, [vp]),
        "hift_step_begin_async": (C.c_int, [vp, vp, vp]),
        "hift_grad_num_chunks": (i32, [vp]),
        "hift_grad_chunk": (C.c_int, [vp, i32, C.POINTER(sz), C.POINTER(sz)]),
        "hift_grad_chunk_wait": (C.c_int, [vp, i32, vp]),
        "hift_gate_view": (C.c_int, [vp, C.POINTER(vp)]),
        "hift_set_grad_chunk_bytes": (C.c_int, [vp, sz]),
        "hift_shard_range": (C.c_int, [vp, i32, i32, C.POINTER(sz), C.POINTER(sz)]),
        "hift_param_view": (C.c_int, [vp, C.POINTER(vp), C.POINTER(sz), C.POINTER(i32)]),
        "hift_step_finish": (C.c_int, [vp, pf]),
        "hift_plan_grad_chunks": (i32, [vp, vp, i32, sz, vp, i32, sz, vp, vp, vp, i32]),
        "hift_active_group": (i32, [vp]),
        "hift_num_groups": (i32, [vp]),
        "hift_num_sets": (i32, [vp]),
        "hift_set_units": (C.c_int, [vp, i32, C.POINTER(i32), i32, C.POINTER(i32)]),
        "hift_step_count": (i64, [vp]),
        "hift_current_lr": (f64, [vp]),
        "hift_group_units": (C.c_int, [vp, i32, C.POINTER(i32), C.POINTER(i32)]),
        "hift_force_group": (C.c_int, [vp, i32]),
        "hift_force_sequence": (C.c_int, [vp, vp, i32]),
        "hift_peak_hbm_bytes": (sz, [vp]),
        "hift_pinned_host_bytes": (sz, [vp]),
        "hift_num_tensors": (i32, [vp]),
        "hift_tensor_info": (C.c_int, [vp, i32, C.c_char_p, C.POINTER(i32), C.POINTER(i64), C.POINTER(i64)]),
        "hift_set_param": (C.c_int, [vp, i32, vp, sz]),
        "hift_get_param": (C.c_int, [vp, i32, vp, sz]),
        "hift_get_model_param": (C.c_int, [vp, i32, vp, sz]),
        "hift_get_grad": (C.c_int, [vp, i32, vp, sz]),
        "hift_get_state": (C.c_int, [vp, i32, i32, vp, sz]),
        "hift_get_factored_state": (C.c_int, [vp, i32, i32, vp, sz]),
        "hift_adafactor_step": (C.c_int, [i64, i64, vp, vp, vp, vp, vp, f64, f64, f64, i64, vp]),
        "hift_init_synthetic": (C.c_int, [vp, C.c_uint64, f64]),
        "hift_load_weights": (C.c_int, [vp, C.c_char_p, i32, C.POINTER(i32)]),
        "hift_save": (C.c_int, [vp, C.c_char_p]),
        "hift_load": (C.c_int, [vp, C.c_char_p]),
        "hift_profile_enable": (C.c_int, [vp, i32]),
        "hift_profile": (C.c_int, [vp, i32, C.POINTER(i64), C.POINTER(f64), C.POINTER(f64)]),
        "hift_last_step_launches": (i64, [vp]),
        "hift_last_step_paging": (C.c_int, [vp, C.POINTER(sz), C.POINTER(sz)]),
        "hift_last_step_timeline": (C.c_int, [vp, C.POINTER(f64)]),
        "hift_tc_error_flag": (i32, [i32]),
        "hift_test_switch": (i32, [i32, i32]),
        "hift_check_arena": (i64, [vp]),
        "hift_arena_guard_count": (i64, [vp]),
        "hift_opt_step": (C.c_int, [i32, sz, vp, vp, vp, vp, vp, f64, f64, f64, f64, f64, f64, i64, vp]),
        "hift_k_linear": (C.c_int, [i32, i32, i32, i64, i64, i64, vp, vp, vp, vp, vp, vp]),
        "hift_k_attention_fwd": (C.c_int, [i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp]),
        "hift_k_attention_bwd": (C.c_int, [i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]),
        "hift_k_attention_fwd_drop": (C.c_int, [i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, f64, C.c_uint64, i32, i64, vp]),
        "hift_k_attention_bwd_drop": (C.c_int, [i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, f64, C.c_uint64, i32, i64, vp]),
        "hift_k_linear_rope": (C.c_int, [i64, i64, i64, vp, vp, vp, vp, vp, i32, i32, i64, vp]),
        "hift_k_linear_swiglu": (C.c_int, [i64, i64, i64, vp, vp, vp, vp, vp, vp]),
        "hift_k_linear_dx_swiglu_bwd": (C.c_int, [i64, i64, i64, vp, vp, vp, vp, vp]),
        "hift_k_linear_gelu": (C.c_int, [i64, i64, i64, vp, vp, vp, vp, vp, vp]),
        "hift_k_linear_dx_gelu_bwd": (C.c_int, [i64, i64, i64, vp, vp, vp, vp, vp]),
        "hift_k_norm_fwd": (C.c_int, [i32, i32, i64, i64, f64, vp, vp, vp, vp, vp, vp]),
        "hift_k_norm_bwd": (C.c_int, [i32, i32, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]),
        "hift_k_norm_bwd_static": (C.c_int, [i32, i32, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp]),
        "hift_k_cross_entropy": (C.c_int, [i32, i64, i64, i64, vp, vp, vp, vp, vp]),
    }


def load_library(path: Optional[str] = None):
    """dlopen libhift.so and declare the prototypes of include/hift.h."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(f"{p} not found: build it with `python -m paper_2401_15207_b200.build`")
    L = C.CDLL(p)
    for name, (res, args) in _prototypes().items():
        f = getattr(L, name)
        f.restype = res
        f.argtypes = args
    if path is None:
        _lib = L
    return L


def lib():
    return load_library()


def _check(status: int, where: str):
    if status != 0:
        raise HiftError(status, where)


def _stream_ptr() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


class HiFT:
    """One model on one GPU; mirrors hift_create / hift_step / getters."""

    def __init__(self, model, groups, opt, stream: Optional[int] = None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("HiFT needs a CUDA device; there is no CPU fallback")
        self.model, self.groups_cfg, self.opt = model, groups, opt
        m = ModelCfgC(model.arch, model.n_blocks, model.d_model, model.n_heads, model.d_ffn,
                      model.vocab, model.max_pos, model.n_classes, model.causal, model.tie_head,
                      model.dtype, model.batch, model.seq, model.norm_eps, model.rope_base,
                      float(getattr(model, "dropout", 0.0)), int(getattr(model, "dropout_seed", 0)),
                      float(getattr(model, "attn_dropout", 0.0)))
        sizes = tuple(getattr(groups, "group_sizes", None) or ())
        arr = (C.c_int32 * len(sizes))(*sizes) if sizes else None
        g = GroupCfgC(groups.layers_per_group, groups.split_emb_head, groups.order, groups.order_seed,
                      C.cast(arr, C.POINTER(C.c_int32)) if sizes else None, len(sizes), int(getattr(groups, "literal_queue", 0)))
        o = OptCfgC(opt.kind, opt.sched, opt.total_cycles, opt.offload_state, opt.prefetch_groups,
                    getattr(opt, "recompute", 0), getattr(opt, "warmup_cycles", 0),
                    getattr(opt, "shard_rank", 0), getattr(opt, "shard_world", 0), getattr(opt, "grad_bf16", 0), opt.lr, opt.beta1, opt.beta2, opt.eps, opt.weight_decay, opt.momentum)
        self._h = C.c_void_p()
        self._stream = _stream_ptr() if stream is None else stream
        _check(lib().hift_create(C.byref(m), C.byref(g), C.byref(o), self._stream, C.byref(self._h)), "hift_create")
        self._names: Dict[str, int] = {}
        self._info: List[Tuple[str, int, int, int]] = []
        buf = C.create_string_buffer(64)
        for i in range(lib().hift_num_tensors(self._h)):
            u, r, c = C.c_int32(), C.c_int64(), C.c_int64()
            _check(lib().hift_tensor_info(self._h, i, buf, C.byref(u), C.byref(r), C.byref(c)), "hift_tensor_info")
            name = buf.value.decode()
            self._names[name] = i
            self._info.append((name, u.value, r.value, c.value))

    # -- lifetime
    def close(self):
        if self._h:
            lib().hift_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the step
    def step(self, tokens, labels) -> float:
        """tokens/labels: int32 CUDA tensors.  Returns the loss (before the update)."""
        loss = C.c_float()
        st = lib().hift_step(self._h, tokens.data_ptr(), labels.data_ptr(), C.byref(loss))
        _check(st, "hift_step")
        return loss.value

    def set_key_lengths(self, lens) -> None:
        """lens: batch ints in [1, seq] (real tokens per right-padded batch entry), or None for no padding."""
        if lens is None:
            _check(lib().hift_set_key_lengths(self._h, None), "hift_set_key_lengths")
            return
        a = np.ascontiguousarray(lens, dtype=np.int32)
        if a.shape != (self.model.batch,):
            raise ValueError("one length per batch entry")
        _check(lib().hift_set_key_lengths(self._h, a.ctypes.data), "hift_set_key_lengths")

    def step_host(self, tokens: np.ndarray, labels: np.ndarray) -> float:
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        labels = np.ascontiguousarray(labels, dtype=np.int32)
        loss = C.c_float()
        st = lib().hift_step_host(self._h, tokens.ctypes.data, labels.ctypes.data, C.byref(loss))
        _check(st, "hift_step_host")
        return loss.value

    def step_begin(self, tokens, labels) -> float:
        """Forward + truncated backward; the group's gradient stays on the device (see grad_view)."""
        loss = C.c_float()
        _check(lib().hift_step_begin(self._h, tokens.data_ptr(), labels.data_ptr(), C.byref(loss)), "hift_step_begin")
        return loss.value

    def grad_view(self):
        """The active group's flat gradient (fp32, or bf16 with grad_bf16) as a torch CUDA tensor sharing the
        library's memory."""
        import torch
        ptr, n = C.c_void_p(), C.c_size_t()
        _check(lib().hift_grad_view(self._h, C.byref(ptr), C.byref(n)), "hift_grad_view")
        half = lib().hift_grad_elem_bytes(self._h) == 2

        class _View:
            __cuda_array_interface__ = {"shape": (n.value,), "typestr": "<i2" if half else "<f4", "data": (ptr.value, False), "version": 3}
        t = torch.as_tensor(_View(), device="cuda")
        return t.view(torch.bfloat16) if half else t

    def step_end(self):
        _check(lib().hift_step_end(self._h), "hift_step_end")

    def step_abort(self):
        _check(lib().hift_step_abort(self._h), "hift_step_abort")

    def step_begin_async(self, tokens, labels) -> None:
        """Enqueues forward + truncated backward and returns; see grad_chunks / step_finish."""
        _check(lib().hift_step_begin_async(self._h, tokens.data_ptr(), labels.data_ptr()), "hift_step_begin_async")

    def grad_chunks(self) -> List[Tuple[int, int]]:
        """(offset, length) of the chunks of grad_view() in the order the backward pass completes them."""
        out = []
        for i in range(lib().hift_grad_num_chunks(self._h)):
            o, n = C.c_size_t(), C.c_size_t()
            _check(lib().hift_grad_chunk(self._h, i, C.byref(o), C.byref(n)), "hift_grad_chunk")
            out.append((o.value, n.value))
        return out

    def grad_chunk_wait(self, i: int, stream: int) -> None:
        _check(lib().hift_grad_chunk_wait(self._h, i, stream), "hift_grad_chunk_wait")

    def gate_view(self):
        """The step's gate word as a one-element int32 CUDA tensor sharing the library's memory."""
        import torch
        ptr = C.c_void_p()
        _check(lib().hift_gate_view(self._h, C.byref(ptr)), "hift_gate_view")

        class _View:
            __cuda_array_interface__ = {"shape": (1,), "typestr": "<i4", "data": (ptr.value, False), "version": 3}
        return torch.as_tensor(_View(), device="cuda")

    def shard_range(self, g: int, rank: int) -> Tuple[int, int]:
        lo, n = C.c_size_t(), C.c_size_t()
        _check(lib().hift_shard_range(self._h, g, rank, C.byref(lo), C.byref(n)), "hift_shard_range")
        return lo.value, n.value

    def param_view(self):
        """Parameters of the group in flight (bf16 or fp32, as the forward pass reads them) as a torch CUDA tensor
        sharing the library's memory."""
        import torch
        ptr, n, eb = C.c_void_p(), C.c_size_t(), C.c_int32()
        _check(lib().hift_param_view(self._h, C.byref(ptr), C.byref(n), C.byref(eb)), "hift_param_view")
        if eb.value == 4:
            class _View:
                __cuda_array_interface__ = {"shape": (n.value,), "typestr": "<f4", "data": (ptr.value, False), "version": 3}
            return torch.as_tensor(_View(), device="cuda")

        class _View16:                                       # bf16 has no array-interface code: view the bits, reinterpret
            __cuda_array_interface__ = {"shape": (n.value,), "typestr": "<i2", "data": (ptr.value, False), "version": 3}
        return torch.as_tensor(_View16(), device="cuda").view(torch.bfloat16)

    def set_grad_chunk_bytes(self, nbytes: int) -> None:
        _check(lib().hift_set_grad_chunk_bytes(self._h, nbytes), "hift_set_grad_chunk_bytes")

    def step_finish(self) -> float:
        loss = C.c_float()
        _check(lib().hift_step_finish(self._h, C.byref(loss)), "hift_step_finish")
        return loss.value

    # -- getters
    def active_group(self) -> int:
        return lib().hift_active_group(self._h)

    def num_groups(self) -> int:
        return lib().hift_num_groups(self._h)

    def num_sets(self) -> int:
        return lib().hift_num_sets(self._h)

    def set_units(self, set_id: int) -> List[int]:
        cap = self.model.n_blocks + 2
        arr, n = (C.c_int32 * cap)(), C.c_int32()
        _check(lib().hift_set_units(self._h, set_id, arr, cap, C.byref(n)), "hift_set_units")
        return list(arr[:n.value])

    def step_count(self) -> int:
        return lib().hift_step_count(self._h)

    def current_lr(self) -> float:
        return lib().hift_current_lr(self._h)

    def group_units(self, g: int) -> Tuple[int, int]:
        lo, hi = C.c_int32(), C.c_int32()
        _check(lib().hift_group_units(self._h, g, C.byref(lo), C.byref(hi)), "hift_group_units")
        return lo.value, hi.value

    def force_group(self, g: int):
        _check(lib().hift_force_group(self._h, g), "hift_force_group")

    def force_sequence(self, groups):
        """The next steps train groups[0], groups[1], ... cyclically; an empty list restores the schedule."""
        a = np.ascontiguousarray(list(groups), dtype=np.int32)
        _check(lib().hift_force_sequence(self._h, a.ctypes.data if a.size else None, int(a.size)), "hift_force_sequence")

    def peak_hbm_bytes(self) -> int:
        return lib().hift_peak_hbm_bytes(self._h)

    def pinned_host_bytes(self) -> int:
        return lib().hift_pinned_host_bytes(self._h)

    def tensor_names(self) -> List[str]:
        return [n for n, _, _, _ in self._info]

    def tensor_info(self, name: str) -> Tuple[int, Tuple[int, int]]:
        n, u, r, c = self._info[self._names[name]]
        return u, (r, c)

    def _numel(self, name: str) -> int:
        _, _, r, c = self._info[self._names[name]]
        return r * c

    def set_param(self, name: str, value: np.ndarray):
        a = np.ascontiguousarray(value, dtype=np.float32)
        _check(lib().hift_set_param(self._h, self._names[name], a.ctypes.data, a.size), "hift_set_param")

    def set_params(self, params: Dict[str, np.ndarray]):
        for k, v in params.items():
            self.set_param(k, v)

    def _get(self, fn, where: str, name: str, *extra) -> np.ndarray:
        n = self._numel(name)
        out = np.empty(n, dtype=np.float32)
        _check(fn(self._h, self._names[name], *extra, out.ctypes.data, n), where)
        _, _, r, c = self._info[self._names[name]]
        return out.reshape(r, c)

    def get_param(self, name: str) -> np.ndarray:
        return self._get(lib().hift_get_param, "hift_get_param", name)

    def get_model_param(self, name: str) -> np.ndarray:
        return self._get(lib().hift_get_model_param, "hift_get_model_param", name)

    def get_grad(self, name: str) -> np.ndarray:
        return self._get(lib().hift_get_grad, "hift_get_grad", name)

    def get_state(self, name: str, which: int) -> np.ndarray:
        return self._get(lib().hift_get_state, "hift_get_state", name, which)

    def get_factored_state(self, name: str, which: int) -> np.ndarray:
        _, _, r, c = self._info[self._names[name]]
        n = c if (r == 1 or which == 1) else r
        out = np.empty(n, dtype=np.float32)
        _check(lib().hift_get_factored_state(self._h, self._names[name], which, out.ctypes.data, n),
               "hift_get_factored_state")
        return out

    def init_synthetic(self, seed: int, std: float = 0.02):
        _check(lib().hift_init_synthetic(self._h, seed, std), "hift_init_synthetic")

    def load_weights(self, path: str, strict: bool = True) -> int:
        """Sets parameters from a HIFTWTS1 file (see weights.py); returns the number of tensors set."""
        n = C.c_int32()
        _check(lib().hift_load_weights(self._h, path.encode(), 1 if strict else 0, C.byref(n)), "hift_load_weights")
        return n.value

    def save(self, path: str):
        _check(lib().hift_save(self._h, path.encode()), "hift_save")

    def load(self, path: str):
        _check(lib().hift_load(self._h, path.encode()), "hift_load")

    # -- instrumentation
    def profile_enable(self, on: bool):
        _check(lib().hift_profile_enable(self._h, 1 if on else 0), "hift_profile_enable")

    def profile(self) -> Dict[str, Dict[str, float]]:
        out = {}
        for i, name in enumerate(KERNEL_CLASSES):
            n, ms, w = C.c_int64(), C.c_double(), C.c_double()
            _check(lib().hift_profile(self._h, i, C.byref(n), C.byref(ms), C.byref(w)), "hift_profile")
            out[name] = {"launches": n.value, "ms": ms.value, "work": w.value}
        return out

    def check_arena(self) -> int:
        """Checked mode: number of arena guard regions the last step overwrote (-1: not in checked mode)."""
        return lib().hift_check_arena(self._h)

    def arena_guard_count(self) -> int:
        return lib().hift_arena_guard_count(self._h)

    def last_step_launches(self) -> int:
        return lib().hift_last_step_launches(self._h)

    def last_step_paging(self) -> Tuple[int, int]:
        a, b = C.c_size_t(), C.c_size_t()
        _check(lib().hift_last_step_paging(self._h, C.byref(a), C.byref(b)), "hift_last_step_paging")
        return a.value, b.value


    def last_step_timeline(self) -> List[float]:
        arr = (C.c_double * 6)()
        _check(lib().hift_last_step_timeline(self._h, arr), "hift_last_step_timeline")
        return list(arr)


# ---------------------------------------------------------------- free functions
def _st(stream):
    return _stream_ptr() if stream is None else stream


def opt_step(kind, n, param_bf16, master, grad, s0, s1, lr, beta1=0.9, beta2=0.999, eps=1e-8,
             weight_decay=0.0, momentum=0.9, tau=1, stream=None):
    _check(lib().hift_opt_step(kind, n, _ptr(param_bf16), _ptr(master), _ptr(grad), _ptr(s0), _ptr(s1),
                               lr, beta1, beta2, eps, weight_decay, momentum, tau, _st(stream)), "hift_opt_step")


def adafactor_step(rows, cols, param_bf16, master, grad, state, scratch, lr, eps1=1e-30, weight_decay=0.0, tau=1,
                   stream=None):
    _check(lib().hift_adafactor_step(rows, cols, _ptr(param_bf16), _ptr(master), _ptr(grad), _ptr(state),
                                     _ptr(scratch), lr, eps1, weight_decay, tau, _st(stream)), "hift_adafactor_step")


def plan_grad_chunks(offsets, sizes, span_elems, completion_order, min_chunk_elems):
    """Host-only chunk plan (hift_plan_grad_chunks): returns [(offset, length, after)]."""
    off = np.ascontiguousarray(offsets, dtype=np.uint64)
    siz = np.ascontiguousarray(sizes, dtype=np.uint64)
    order = np.ascontiguousarray(completion_order, dtype=np.int32)
    cap = len(off) + 1
    co, cn, ca = np.zeros(cap, np.uint64), np.zeros(cap, np.uint64), np.zeros(cap, np.int32)
    n = lib().hift_plan_grad_chunks(off.ctypes.data, siz.ctypes.data, len(off), int(span_elems), order.ctypes.data,
                                    len(order), int(min_chunk_elems), co.ctypes.data, cn.ctypes.data, ca.ctypes.data, cap)
    if n < 0:
        raise ValueError("hift_plan_grad_chunks: bad arguments")
    return [(int(co[i]), int(cn[i]), int(ca[i])) for i in range(n)]


def tc_error_flag(set_value: int = -1) -> int:
    return lib().hift_tc_error_flag(set_value)


SWITCH_GEMM_PAIR, SWITCH_PDL, SWITCH_ATTN_FWD_TC, SWITCH_ATTN_BWD_TC, SWITCH_FAIL_PINNED, SWITCH_CHECKED_ARENA = 0, 1, 2, 3, 4, 5


def code_path_switch(which: int, value: int = -1) -> int:
    """Sets (value >= 0) or reads a code-path switch of the library; returns the previous value."""
    return lib().hift_test_switch(which, value)


def k_linear(form, dtype, M, N, K, a, b, out, bias=None, residual=None, path=0, stream=None):
    _check(lib().hift_k_linear(form, dtype, path, M, N, K, _ptr(a), _ptr(b), _ptr(out), _ptr(bias),
                               _ptr(residual), _st(stream)), "hift_k_linear")


def k_attention_fwd(dtype, B, S, H, dh, causal, qkv, o, lse, stream=None, key_lens=None):
    _check(lib().hift_k_attention_fwd(dtype, B, S, H, dh, causal, _ptr(qkv), _ptr(o), _ptr(lse), _ptr(key_lens),
                                      _st(stream)), "hift_k_attention_fwd")


def k_attention_bwd(dtype, B, S, H, dh, causal, qkv, o, lse, dout, dqkv, dsum, stream=None, key_lens=None):
    _check(lib().hift_k_attention_bwd(dtype, B, S, H, dh, causal, _ptr(qkv), _ptr(o), _ptr(lse), _ptr(dout),
                                      _ptr(dqkv), _ptr(dsum), _ptr(key_lens), _st(stream)), "hift_k_attention_bwd")


def k_attention_fwd_drop(dtype, B, S, H, dh, causal, qkv, o, lse, p, seed, site, step, stream=None, key_lens=None):
    _check(lib().hift_k_attention_fwd_drop(dtype, B, S, H, dh, causal, _ptr(qkv), _ptr(o), _ptr(lse), _ptr(key_lens),
                                           float(p), int(seed), int(site), int(step), _st(stream)),
           "hift_k_attention_fwd_drop")


def k_attention_bwd_drop(dtype, B, S, H, dh, causal, qkv, o, lse, dout, dqkv, dsum, p, seed, site, step, stream=None,
                         key_lens=None):
    _check(lib().hift_k_attention_bwd_drop(dtype, B, S, H, dh, causal, _ptr(qkv), _ptr(o), _ptr(lse), _ptr(dout),
                                           _ptr(dqkv), _ptr(dsum), _ptr(key_lens), float(p), int(seed),
                                           int(site), int(step), _st(stream)), "hift_k_attention_bwd_drop")


def k_linear_rope(M, N, K, a, b, out, bias, cs, seq, d_head, rope_cols, stream=None):
    _check(lib().hift_k_linear_rope(M, N, K, _ptr(a), _ptr(b), _ptr(out), _ptr(bias), _ptr(cs), seq, d_head, rope_cols,
                                    _st(stream)), "hift_k_linear_rope")


def k_linear_swiglu(M, f, K, a, b, gu, s, bias=None, stream=None):
    _check(lib().hift_k_linear_swiglu(M, f, K, _ptr(a), _ptr(b), _ptr(gu), _ptr(s), _ptr(bias), _st(stream)),
           "hift_k_linear_swiglu")


def k_linear_dx_swiglu_bwd(M, N, f, dy, w, gu, dgu, stream=None):
    _check(lib().hift_k_linear_dx_swiglu_bwd(M, N, f, _ptr(dy), _ptr(w), _ptr(gu), _ptr(dgu), _st(stream)),
           "hift_k_linear_dx_swiglu_bwd")


def k_linear_gelu(M, N, K, a, b, pre, act, bias=None, stream=None):
    _check(lib().hift_k_linear_gelu(M, N, K, _ptr(a), _ptr(b), _ptr(pre), _ptr(act), _ptr(bias), _st(stream)),
           "hift_k_linear_gelu")


def k_linear_dx_gelu_bwd(M, N, f, dy, w, pre, da, stream=None):
    _check(lib().hift_k_linear_dx_gelu_bwd(M, N, f, _ptr(dy), _ptr(w), _ptr(pre), _ptr(da), _st(stream)),
           "hift_k_linear_dx_gelu_bwd")


def k_norm_fwd(dtype, kind, rows, cols, eps, x, gain, bias, y, stats, stream=None):
    _check(lib().hift_k_norm_fwd(dtype, kind, rows, cols, eps, _ptr(x), _ptr(gain), _ptr(bias), _ptr(y),
                                 _ptr(stats), _st(stream)), "hift_k_norm_fwd")


def k_norm_bwd(dtype, kind, rows, cols, dy, x, stats, gain, add, dx, dgain, dbias, partial, stream=None):
    _check(lib().hift_k_norm_bwd(dtype, kind, rows, cols, _ptr(dy), _ptr(x), _ptr(stats), _ptr(gain), _ptr(add),
                                 _ptr(dx), _ptr(dgain), _ptr(dbias), _ptr(partial), _st(stream)), "hift_k_norm_bwd")


def k_norm_bwd_static(dtype, kind, rows, cols, dy, x, stats, gain, add, dx, dgain, dbias, stream=None):
    """hift_k_norm_bwd without the caller-provided scratch and without any allocation: for
    callers that may not allocate.  cols <= STATIC_SCRATCH_MAX_COLS; calls on one GPU must not
    overlap (they share one built-in scratch array)."""
    _check(lib().hift_k_norm_bwd_static(dtype, kind, rows, cols, _ptr(dy), _ptr(x), _ptr(stats), _ptr(gain),
                                        _ptr(add), _ptr(dx), _ptr(dgain), _ptr(dbias), _st(stream)),
           "hift_k_norm_bwd_static")


def k_cross_entropy(dtype, rows, vocab, ld, logits, labels, rowloss, loss, stream=None):
    _check(lib().hift_k_cross_entropy(dtype, rows, vocab, ld, _ptr(logits), _ptr(labels), _ptr(rowloss),
                                      _ptr(loss), _st(stream)), "hift_k_cross_entropy")
