"""ctypes access to the CPU oracle (`qwen3_oracle.c`).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's cpu-baseline leg import this package; nothing under the
product package does.  `build()` compiles two variants of the same file with gcc: fp32 accumulation (the
reference precision) and double accumulation (its error bar).  Tensors are torch CPU tensors used purely as
memory: bf16 for weights and cache contents, float32 for activations, int32 for tokens.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qwen3_oracle.c")
_LIBS = {}


def lib_path(double_acc: bool = False) -> str:
    return os.path.join(_HERE, "liboracle_f64.so" if double_acc else "liboracle_f32.so")


def build(force: bool = False) -> None:
    for dbl in (False, True):
        out = lib_path(dbl)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
            continue
        cmd = ["gcc", "-O2", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", out, _SRC, "-lm"]
        if dbl:
            cmd.insert(1, "-DORC_ACC_DOUBLE")
        subprocess.check_call(cmd)


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim",
                                         "intermediate", "vocab", "max_seq")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_double)]


_LAYER_FIELDS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "g_in", "g_post", "g_q", "g_k")


class _Layer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _LAYER_FIELDS]


def load(double_acc: bool = False) -> C.CDLL:
    if double_acc not in _LIBS:
        build()
        L = C.CDLL(lib_path(double_acc))
        L.orc_bf16_to_f32.restype = C.c_float
        L.orc_bf16_to_f32.argtypes = [C.c_uint16]
        L.orc_f32_to_bf16.restype = C.c_uint16
        L.orc_f32_to_bf16.argtypes = [C.c_float]
        L.orc_silu.restype = C.c_float
        L.orc_silu.argtypes = [C.c_float]
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.POINTER(_Config), C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(_Layer)]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_reset.argtypes = [C.c_void_p]
        L.orc_length.argtypes = [C.c_void_p]
        L.orc_rope_ptr.restype = C.c_void_p
        L.orc_rope_ptr.argtypes = [C.c_void_p]
        L.orc_kv_import.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int]
        L.orc_kv_export.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int]
        L.orc_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_layer_decode.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_float, C.c_void_p]
        L.orc_rope_table.argtypes = [C.c_int, C.c_int, C.c_double, C.c_void_p]
        L.orc_rope_apply.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
        L.orc_matmul.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]
        L.orc_softmax.argtypes = [C.c_void_p, C.c_int]
        L.orc_attend.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_size_t,
                                 C.c_void_p, C.c_void_p]
        L.orc_e4m3_to_f32.restype = C.c_float
        L.orc_e4m3_to_f32.argtypes = [C.c_uint8]
        L.orc_f32_to_e4m3.restype = C.c_uint8
        L.orc_f32_to_e4m3.argtypes = [C.c_float]
        L.orc_quantise_rows_e4m3.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_dequantise_rows_e4m3.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        L.orc_argmax_margin.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        _LIBS[double_acc] = L
    return _LIBS[double_acc]


def _f32(t: torch.Tensor) -> torch.Tensor:
    assert t.dtype == torch.float32 and t.device.type == "cpu" and t.is_contiguous()
    return t


def _bf16(t: torch.Tensor) -> torch.Tensor:
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu" and t.is_contiguous()
    return t


# ---- thin function wrappers (used by the pin tests) --------------------------------------------------

def rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float, double_acc=False) -> torch.Tensor:
    y = torch.empty_like(_f32(x))
    load(double_acc).orc_rmsnorm(x.data_ptr(), _bf16(gain).data_ptr(), x.numel(), eps, y.data_ptr())
    return y


def rope_table(n_pos: int, d: int, theta: float) -> torch.Tensor:
    t = torch.empty(n_pos, d // 2, 2, dtype=torch.float32)
    load().orc_rope_table(n_pos, d, theta, t.data_ptr())
    return t


def rope_apply(x: torch.Tensor, row: torch.Tensor) -> torch.Tensor:
    y = _f32(x).clone()
    load().orc_rope_apply(y.data_ptr(), y.numel(), _f32(row).data_ptr())
    return y


def matmul(W: torch.Tensor, X: torch.Tensor, double_acc=False) -> torch.Tensor:
    n_out, n_in = W.shape
    T = X.shape[0]
    Y = torch.empty(T, n_out, dtype=torch.float32)
    load(double_acc).orc_matmul(_bf16(W).data_ptr(), _f32(X).data_ptr(), T, n_out, n_in, Y.data_ptr())
    return Y


def softmax(s: torch.Tensor, double_acc=False) -> torch.Tensor:
    y = _f32(s).clone()
    load(double_acc).orc_softmax(y.data_ptr(), y.numel())
    return y


def silu(z: float) -> float:
    return load().orc_silu(z)


def attend(q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, double_acc=False) -> torch.Tensor:
    n, d = K.shape
    o = torch.empty(d, dtype=torch.float32)
    scratch = torch.empty(n, dtype=torch.float32)
    load(double_acc).orc_attend(_f32(q).data_ptr(), _bf16(K).data_ptr(), _bf16(V).data_ptr(), n, d, d,
                                scratch.data_ptr(), o.data_ptr())
    return o


def argmax_margin(v: torch.Tensor):
    idx, margin = C.c_int32(), C.c_float()
    load().orc_argmax_margin(_f32(v).data_ptr(), v.numel(), C.byref(idx), C.byref(margin))
    if idx.value < 0:
        raise ValueError("argmax_margin: the logits hold a NaN or an infinity")
    return idx.value, margin.value


def e4m3_to_f32(code: int) -> float:
    return load().orc_e4m3_to_f32(code)


def f32_to_e4m3(x: float) -> int:
    return load().orc_f32_to_e4m3(x)


def quantise_rows_e4m3(W: torch.Tensor):
    """bf16 [n_out][n_in] -> (codes uint8 [n_out][n_in], exps int8 [n_out]): E4M3 codes of W / 2^exp per row."""
    n_out, n_in = W.shape
    codes = torch.empty(n_out, n_in, dtype=torch.uint8)
    exps = torch.empty(n_out, dtype=torch.int8)
    load().orc_quantise_rows_e4m3(_bf16(W).data_ptr(), n_out, n_in, codes.data_ptr(), exps.data_ptr())
    return codes, exps


def dequantise_rows_e4m3(codes: torch.Tensor, exps: torch.Tensor) -> torch.Tensor:
    """(codes, exps) -> bf16 [n_out][n_in] holding e4m3(code) * 2^exp exactly."""
    n_out, n_in = codes.shape
    assert codes.dtype == torch.uint8 and exps.dtype == torch.int8 and codes.is_contiguous() and exps.is_contiguous()
    W = torch.empty(n_out, n_in, dtype=torch.bfloat16)
    load().orc_dequantise_rows_e4m3(codes.data_ptr(), exps.data_ptr(), n_out, n_in, W.data_ptr())
    return W


def f32_to_bf16_bits(f: float) -> int:
    return load().orc_f32_to_bf16(f)


# ---- model ---------------------------------------------------------------------------------------------

class Oracle:
    """One sequence of the oracle model.  `shape` needs the attributes of a model shape (n_layers, hidden,
    n_q_heads, n_kv_heads, head_dim, intermediate, vocab, tie_embeddings, rms_eps, rope_theta); `weights` is
    a dict {embed, lm_head|None, g_final, layers: [{wq, ..., g_k}]} of CPU bf16 tensors."""

    def __init__(self, shape, weights: dict, max_seq: int, double_acc: bool = False):
        self.L = load(double_acc)
        self.shape, self.max_seq = shape, max_seq
        self._keep = weights
        cfg = _Config(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                      shape.intermediate, shape.vocab, max_seq, shape.rms_eps, shape.rope_theta)
        layers = (_Layer * shape.n_layers)()
        for l, lw in enumerate(weights["layers"]):
            for n in _LAYER_FIELDS:
                setattr(layers[l], n, _bf16(lw[n]).data_ptr())
        lm = weights.get("lm_head")
        self.h = self.L.orc_create(C.byref(cfg), _bf16(weights["embed"]).data_ptr(),
                                   _bf16(lm).data_ptr() if lm is not None else None,
                                   _bf16(weights["g_final"]).data_ptr(), layers)
        if not self.h:
            raise ValueError("oracle rejected the configuration")

    def close(self):
        if self.h:
            self.L.orc_destroy(self.h)
            self.h = None

    __del__ = close

    @property
    def length(self) -> int:
        return self.L.orc_length(self.h)

    def reset(self):
        self.L.orc_reset(self.h)

    def rope(self) -> torch.Tensor:
        d = self.shape.head_dim
        buf = (C.c_float * (self.max_seq * d)).from_address(self.L.orc_rope_ptr(self.h))
        return torch.frombuffer(buf, dtype=torch.float32).view(self.max_seq, d // 2, 2).clone()

    def kv_import(self, layer: int, k: torch.Tensor, v: torch.Tensor):
        assert k.shape == v.shape and k.shape[0] == self.shape.n_kv_heads
        if self.L.orc_kv_import(self.h, layer, _bf16(k).data_ptr(), _bf16(v).data_ptr(), k.shape[1]):
            raise ValueError("kv_import out of range")

    def kv_export(self, layer: int, n_pos: int):
        s = self.shape
        k = torch.empty(s.n_kv_heads, n_pos, s.head_dim, dtype=torch.bfloat16)
        v = torch.empty_like(k)
        if self.L.orc_kv_export(self.h, layer, k.data_ptr(), v.data_ptr(), n_pos):
            raise ValueError("kv_export out of range")
        return k, v

    def forward(self, tokens: torch.Tensor, all_positions: bool = False, want_taps: bool = False):
        """Returns (logits, taps): logits [T][V] or [V]; taps [L+1][T][H] or None."""
        tokens = tokens.to(torch.int32).contiguous()
        T, s = tokens.numel(), self.shape
        logits = torch.empty((T, s.vocab) if all_positions else (s.vocab,), dtype=torch.float32)
        taps = torch.empty(s.n_layers + 1, T, s.hidden, dtype=torch.float32) if want_taps else None
        rc = self.L.orc_forward(self.h, tokens.data_ptr(), T, logits.data_ptr(), int(all_positions),
                                taps.data_ptr() if want_taps else None)
        if rc:
            raise ValueError("oracle forward failed (cache overflow or token out of range)")
        return logits, taps

    def layer_decode(self, layer: int, x: torch.Tensor) -> torch.Tensor:
        y = torch.empty_like(_f32(x))
        if self.L.orc_layer_decode(self.h, layer, x.data_ptr(), y.data_ptr()):
            raise ValueError("oracle layer_decode failed")
        return y
