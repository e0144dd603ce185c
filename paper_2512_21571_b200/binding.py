"""ctypes binding of libnnc.so: same names as the C ABI (include/nnc.h), argument marshalling only.

PyTorch is used for device memory and the CUDA stream; every step of the forward pass runs inside the library's
kernels.  Importing this module loads the shared library and raises if it has not been built -- there is no
fallback path of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("NNC_LIBRARY") or os.path.join(_HERE, "libnnc.so")   # NNC_LIBRARY: another build of the same ABI

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_21571_b200.build` "
                      "(or __graft_entry__.build()); there is no fallback implementation")
lib = C.CDLL(LIB_PATH)


class nnc_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "intermediate",
                                         "vocab", "max_seq", "max_batch", "max_tokens", "tie_embeddings")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("tc_operands", C.c_int32),
                ("weight_format", C.c_int32), ("serial_launches", C.c_int32)]


LAYER_FIELDS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "g_in", "g_post", "g_q", "g_k")


class nnc_layer_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in LAYER_FIELDS]


class nnc_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("g_final", C.c_void_p),
                ("layers", C.POINTER(nnc_layer_weights))]


EXPORTS = {
    "nnc_workspace_bytes": (C.c_size_t, [C.POINTER(nnc_config)]),
    "nnc_model_create": (C.c_int, [C.POINTER(nnc_config), C.POINTER(nnc_weights), C.c_void_p, C.c_size_t, C.c_void_p,
                                   C.POINTER(C.c_void_p)]),
    "nnc_model_destroy": (None, [C.c_void_p]),
    "nnc_prefill": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32]),
    "nnc_decode_step": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "nnc_decode_step_host": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "nnc_prefill_host": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32]),
    "nnc_kv_import": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32]),
    "nnc_kv_export": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32]),
    "nnc_set_length": (C.c_int, [C.c_void_p, C.c_int32]),
    "nnc_get_length": (C.c_int32, [C.c_void_p]),
    "nnc_set_hidden_tap": (C.c_int, [C.c_void_p, C.c_void_p]),
    "nnc_layer_decode": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "nnc_unrepack": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]),
    "nnc_device_status": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32)]),
    "nnc_launch_count": (C.c_int64, [C.c_void_p]),
    "nnc_bounds_check_report": (C.c_int, [C.POINTER(C.c_int32), C.POINTER(C.c_int32)]),
    "nnc_bounds_check_selftest": (C.c_int, [C.c_int32, C.c_void_p]),
    "nnc_last_error": (C.c_char_p, [C.c_void_p]),
    "nnc_status_string": (C.c_char_p, [C.c_int]),
    "nnc_op_gemm": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                              C.c_int32, C.c_void_p]),
    "nnc_op_gemm_swiglu": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                     C.c_int32, C.c_void_p]),
    "nnc_op_gemm_splitk": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                     C.c_int32, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]),
    "nnc_op_gemm_f16": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                  C.c_void_p]),
    "nnc_op_gemm_swiglu_f16": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                         C.c_void_p]),
    "nnc_op_to_f16_scaled": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p]),
    "nnc_op_status": (C.c_int, [C.POINTER(C.c_int32)]),
    "nnc_op_gemv": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_float, C.c_int32,
                              C.c_void_p]),
    "nnc_op_quantise_rows_e4m3": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]),
    "nnc_op_gemv_fp8": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_float,
                                  C.c_int32, C.c_void_p]),
    "nnc_attn_scratch_bytes": (C.c_size_t, [C.c_int32, C.c_int32, C.c_int32]),
    "nnc_op_attn_decode": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                     C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]),
    "nnc_op_attn_prefill": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                      C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]),
    "nnc_op_attn_prefill_f16": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                          C.c_int32, C.c_int32, C.c_int32, C.c_void_p]),
    "nnc_op_attn_decode_static": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                            C.c_int32, C.c_int32, C.c_int32, C.c_void_p]),
}
for _name, (_res, _args) in EXPORTS.items():
    _fn = getattr(lib, _name)
    _fn.restype, _fn.argtypes = _res, _args


class NncError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        super().__init__(f"nnc status {status} ({lib.nnc_status_string(status).decode()}): {detail}")


def _stream_ptr() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype) -> int:
    assert t.is_cuda and t.dtype == dtype and t.is_contiguous(), (t.device, t.dtype, t.is_contiguous())
    return t.data_ptr()


class Model:
    """nnc_model_create / nnc_prefill / nnc_decode_step and the auxiliary calls, one method per C function."""

    def __init__(self, shape, weights: dict, max_seq: int, max_batch: int = 1, max_tokens: Optional[int] = None,
                 tc_operands: int = 0, serial_launches: bool = False,
                 weight_format: int = 0):
        self.shape = shape
        self.cfg = nnc_config(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                              shape.intermediate, shape.vocab, max_seq, max_batch,
                              max_tokens if max_tokens is not None else max(max_batch, 1),
                              int(shape.tie_embeddings), shape.rms_eps, shape.rope_theta,
                              int(tc_operands), int(weight_format), int(serial_launches))
        self.handle = C.c_void_p()
        nbytes = lib.nnc_workspace_bytes(C.byref(self.cfg))
        if nbytes == 0:
            raise NncError(-1, "configuration rejected by nnc_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        layers = (nnc_layer_weights * shape.n_layers)()
        for l, lw in enumerate(weights["layers"]):
            for n in LAYER_FIELDS:
                setattr(layers[l], n, _dev(lw[n], torch.bfloat16))
        lm = weights.get("lm_head")
        w = nnc_weights(_dev(weights["embed"], torch.bfloat16), _dev(lm, torch.bfloat16) if lm is not None else None,
                        _dev(weights["g_final"], torch.bfloat16), layers)
        self.stream = _stream_ptr()
        rc = lib.nnc_model_create(C.byref(self.cfg), C.byref(w), self.workspace.data_ptr(), nbytes, self.stream,
                                  C.byref(self.handle))
        if rc:
            self.handle = C.c_void_p()
            raise NncError(rc, "nnc_model_create")
        self._tap = None

    def _check(self, rc: int):
        if rc:
            raise NncError(rc, lib.nnc_last_error(self.handle).decode())

    def close(self):
        if getattr(self, "handle", None):
            lib.nnc_model_destroy(self.handle)
            self.handle = C.c_void_p()
            self.workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the three calls ----
    def prefill(self, tokens: torch.Tensor, logits: Optional[torch.Tensor] = None, all_positions: bool = False,
                want_logits: bool = True) -> Optional[torch.Tensor]:
        batch, n = tokens.shape
        if want_logits and logits is None:
            shape = (batch, n, self.shape.vocab) if all_positions else (batch, self.shape.vocab)
            logits = torch.empty(shape, dtype=torch.float32, device="cuda")
        self._check(lib.nnc_prefill(self.handle, _dev(tokens, torch.int32), batch, n,
                                    _dev(logits, torch.float32) if want_logits else None, int(all_positions)))
        return logits

    def decode_step(self, tokens: torch.Tensor, logits: torch.Tensor, argmax: Optional[torch.Tensor] = None):
        self._check(lib.nnc_decode_step(self.handle, _dev(tokens, torch.int32), tokens.numel(),
                                        _dev(logits, torch.float32),
                                        _dev(argmax, torch.int32) if argmax is not None else None))

    def decode_step_host(self, tokens_host: torch.Tensor, logits_host: Optional[torch.Tensor],
                         argmax_host: Optional[torch.Tensor] = None):
        assert not tokens_host.is_cuda and tokens_host.dtype == torch.int32
        self._check(lib.nnc_decode_step_host(
            self.handle, tokens_host.data_ptr(), tokens_host.numel(),
            logits_host.data_ptr() if logits_host is not None else None,
            argmax_host.data_ptr() if argmax_host is not None else None))

    def prefill_host(self, tokens_host: torch.Tensor, logits_host: Optional[torch.Tensor], all_positions=False):
        assert not tokens_host.is_cuda and tokens_host.dtype == torch.int32
        batch, n = tokens_host.shape
        self._check(lib.nnc_prefill_host(self.handle, tokens_host.data_ptr(), batch, n,
                                         logits_host.data_ptr() if logits_host is not None else None,
                                         int(all_positions)))

    # ---- auxiliaries ----
    def kv_import(self, layer: int, batch_index: int, k: torch.Tensor, v: torch.Tensor):
        self._check(lib.nnc_kv_import(self.handle, layer, batch_index, _dev(k, torch.bfloat16),
                                      _dev(v, torch.bfloat16), k.shape[1]))

    def kv_export(self, layer: int, batch_index: int, n_pos: int):
        s = self.shape
        k = torch.empty(s.n_kv_heads, n_pos, s.head_dim, dtype=torch.bfloat16, device="cuda")
        v = torch.empty_like(k)
        self._check(lib.nnc_kv_export(self.handle, layer, batch_index, k.data_ptr(), v.data_ptr(), n_pos))
        return k, v

    def set_length(self, n: int):
        self._check(lib.nnc_set_length(self.handle, n))

    @property
    def length(self) -> int:
        return lib.nnc_get_length(self.handle)

    def set_hidden_tap(self, taps: Optional[torch.Tensor]):
        self._tap = taps
        self._check(lib.nnc_set_hidden_tap(self.handle, _dev(taps, torch.float32) if taps is not None else None))

    def layer_decode(self, layer: int, x: torch.Tensor) -> torch.Tensor:
        y = torch.empty_like(x)
        self._check(lib.nnc_layer_decode(self.handle, layer, _dev(x, torch.float32), y.data_ptr()))
        return y

    def unrepack(self, layer: int, which: int, like: torch.Tensor) -> torch.Tensor:
        out = torch.empty_like(like)
        self._check(lib.nnc_unrepack(self.handle, layer, which, out.data_ptr()))
        return out

    def device_status(self) -> int:
        st = C.c_int32(0)
        lib.nnc_device_status(self.handle, C.byref(st))
        return st.value

    @property
    def launch_count(self) -> int:
        return lib.nnc_launch_count(self.handle)


# ---- single operations -----------------------------------------------------------------------------------

def _ok(rc: int, what: str):
    if rc:
        raise NncError(rc, what)


def op_gemm(X: torch.Tensor, W: torch.Tensor, out_f32: bool = True, accumulate_into: Optional[torch.Tensor] = None,
            X_lo: Optional[torch.Tensor] = None):
    T, K = X.shape
    N = W.shape[0]
    if accumulate_into is not None:
        Y = accumulate_into
    else:
        Y = torch.empty(T, N, dtype=torch.float32 if out_f32 else torch.bfloat16, device="cuda")
    _ok(lib.nnc_op_gemm(_dev(X, torch.bfloat16), _dev(X_lo, torch.bfloat16) if X_lo is not None else None,
                        _dev(W, torch.bfloat16), Y.data_ptr(), T, N, K, int(out_f32),
                        int(accumulate_into is not None), _stream_ptr()), "nnc_op_gemm")
    return Y


def op_gemm_swiglu(X: torch.Tensor, W: torch.Tensor, X_lo: Optional[torch.Tensor] = None, want_lo: bool = False):
    T, K = X.shape
    N = W.shape[0]
    Y = torch.empty(T, N // 2, dtype=torch.bfloat16, device="cuda")
    Y_lo = torch.empty_like(Y) if want_lo else None
    _ok(lib.nnc_op_gemm_swiglu(_dev(X, torch.bfloat16), _dev(X_lo, torch.bfloat16) if X_lo is not None else None,
                               _dev(W, torch.bfloat16), Y.data_ptr(), Y_lo.data_ptr() if want_lo else None, T, N, K,
                               _stream_ptr()), "nnc_op_gemm_swiglu")
    return (Y, Y_lo) if want_lo else Y


def op_to_f16_scaled(W: torch.Tensor):
    """nnc_op_to_f16_scaled: (fp16 copy of W * 2^e, scales tensor {2^e, 2^-e} on the device)."""
    out = torch.empty(W.shape, dtype=torch.float16, device="cuda")
    scales = torch.zeros(2, dtype=torch.float32, device="cuda")
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    _ok(lib.nnc_op_to_f16_scaled(_dev(W, torch.bfloat16), out.data_ptr(), W.numel(), scales.data_ptr(), word.data_ptr(),
                                 _stream_ptr()), "nnc_op_to_f16_scaled")
    return out, scales


def op_gemm_f16(X: torch.Tensor, W: torch.Tensor, out_scale: Optional[torch.Tensor] = None,
                accumulate_into: Optional[torch.Tensor] = None):
    T, K = X.shape
    N = W.shape[0]
    Y = accumulate_into if accumulate_into is not None else torch.empty(T, N, dtype=torch.float32, device="cuda")
    _ok(lib.nnc_op_gemm_f16(_dev(X, torch.float16), _dev(W, torch.float16), _dev(Y, torch.float32), T, N, K,
                            int(accumulate_into is not None), out_scale.data_ptr() if out_scale is not None else None,
                            _stream_ptr()), "nnc_op_gemm_f16")
    return Y


def op_gemm_swiglu_f16(X: torch.Tensor, W: torch.Tensor, out_scale: Optional[torch.Tensor] = None):
    T, K = X.shape
    N = W.shape[0]
    Y = torch.empty(T, N // 2, dtype=torch.float16, device="cuda")
    _ok(lib.nnc_op_gemm_swiglu_f16(_dev(X, torch.float16), _dev(W, torch.float16), Y.data_ptr(), T, N, K,
                                   out_scale.data_ptr() if out_scale is not None else None, _stream_ptr()),
        "nnc_op_gemm_swiglu_f16")
    return Y


def bounds_check_report():
    """(misses, first code) since the last call; misses == -1 in a library built without -DNNC_BOUNDS_CHECK."""
    n, code = C.c_int32(0), C.c_int32(0)
    _ok(lib.nnc_bounds_check_report(C.byref(n), C.byref(code)), "nnc_bounds_check_report")
    return n.value, code.value


def op_status() -> int:
    st = C.c_int32(0)
    lib.nnc_op_status(C.byref(st))
    return st.value


GEMV_CHAINED = 0x100


def op_gemv(W: torch.Tensor, x: torch.Tensor, mode: int = 0, gain: Optional[torch.Tensor] = None, eps: float = 1e-6,
            y: Optional[torch.Tensor] = None, chained: bool = False):
    N, K = W.shape
    if y is None:
        y = torch.empty(N // 2 if (mode & 0xff) == 2 else N, dtype=torch.float32, device="cuda")
    _ok(lib.nnc_op_gemv(_dev(W, torch.bfloat16), _dev(x, torch.float32), _dev(y, torch.float32), N, K,
                        _dev(gain, torch.bfloat16) if gain is not None else None, eps,
                        mode | (GEMV_CHAINED if chained else 0), _stream_ptr()), "nnc_op_gemv")
    return y


def op_quantise_rows_e4m3(W: torch.Tensor, want_dequant: bool = True):
    """nnc_op_quantise_rows_e4m3: (codes uint8, scales fp32 [n_out], dequantised bf16 or None)."""
    n_out, n_in = W.shape
    codes = torch.empty(n_out, n_in, dtype=torch.uint8, device="cuda")
    scales = torch.empty(n_out, dtype=torch.float32, device="cuda")
    dq = torch.empty_like(W) if want_dequant else None
    _ok(lib.nnc_op_quantise_rows_e4m3(_dev(W, torch.bfloat16), codes.data_ptr(), scales.data_ptr(),
                                      dq.data_ptr() if want_dequant else None, n_out, n_in, _stream_ptr()),
        "nnc_op_quantise_rows_e4m3")
    return codes, scales, dq


def op_gemv_fp8(codes: torch.Tensor, scales: torch.Tensor, x: torch.Tensor, mode: int = 0,
                gain: Optional[torch.Tensor] = None, eps: float = 1e-6, y: Optional[torch.Tensor] = None,
                chained: bool = False):
    N, K = codes.shape
    if y is None:
        y = torch.empty(N // 2 if (mode & 0xff) == 2 else N, dtype=torch.float32, device="cuda")
    _ok(lib.nnc_op_gemv_fp8(_dev(codes, torch.uint8), _dev(scales, torch.float32), _dev(x, torch.float32),
                            _dev(y, torch.float32), N, K, _dev(gain, torch.bfloat16) if gain is not None else None, eps,
                            mode | (GEMV_CHAINED if chained else 0), _stream_ptr()), "nnc_op_gemv_fp8")
    return y


def op_attn_decode(q: torch.Tensor, kcache: torch.Tensor, vcache: torch.Tensor, n_ctx: int,
                   scratch: Optional[torch.Tensor] = None):
    batch, nq, d = q.shape
    _, nkv, max_seq, _ = kcache.shape
    if scratch is None:
        scratch = torch.empty(lib.nnc_attn_scratch_bytes(batch, nq, n_ctx), dtype=torch.uint8, device="cuda")
    out = torch.empty_like(q)
    _ok(lib.nnc_op_attn_decode(_dev(q, torch.float32), _dev(kcache, torch.bfloat16), _dev(vcache, torch.bfloat16),
                               out.data_ptr(), batch, nq, nkv, max_seq, n_ctx, scratch.data_ptr(), _stream_ptr()),
        "nnc_op_attn_decode")
    return out


def op_attn_decode_static(q: torch.Tensor, kcache: torch.Tensor, vcache: torch.Tensor, n_ctx: int):
    """nnc_op_attn_decode_static: as op_attn_decode, with the scratch in the library's built-in array (for callers
    that cannot allocate).  The output tensor is the only buffer this wrapper creates."""
    batch, nq, d = q.shape
    _, nkv, max_seq, _ = kcache.shape
    out = torch.empty_like(q)
    _ok(lib.nnc_op_attn_decode_static(_dev(q, torch.float32), _dev(kcache, torch.bfloat16), _dev(vcache, torch.bfloat16),
                                      out.data_ptr(), batch, nq, nkv, max_seq, n_ctx, _stream_ptr()),
        "nnc_op_attn_decode_static")
    return out


def op_gemm_splitk(X: torch.Tensor, W: torch.Tensor, scratch: torch.Tensor, out_f32: bool = True,
                   accumulate_into: Optional[torch.Tensor] = None, X_lo: Optional[torch.Tensor] = None):
    """nnc_op_gemm_splitk; `scratch` is a uint8 CUDA tensor whose first 16 KiB are zero."""
    T, K = X.shape
    N = W.shape[0]
    Y = accumulate_into if accumulate_into is not None else \
        torch.empty(T, N, dtype=torch.float32 if out_f32 else torch.bfloat16, device="cuda")
    _ok(lib.nnc_op_gemm_splitk(_dev(X, torch.bfloat16), _dev(X_lo, torch.bfloat16) if X_lo is not None else None,
                               _dev(W, torch.bfloat16), Y.data_ptr(), T, N, K, int(out_f32),
                               int(accumulate_into is not None), scratch.data_ptr(), scratch.numel(), _stream_ptr()),
        "nnc_op_gemm_splitk")
    return Y


def op_attn_prefill(qkv: torch.Tensor, kcache: torch.Tensor, vcache: torch.Tensor, T: int, n_q_heads: int, n_past: int):
    """nnc_op_attn_prefill; returns (out, out_lo), bf16 [batch * T][n_q_heads * 128]."""
    batch, nkv, max_seq, _ = kcache.shape
    out = torch.empty(batch * T, n_q_heads * 128, dtype=torch.bfloat16, device="cuda")
    out_lo = torch.empty_like(out)
    _ok(lib.nnc_op_attn_prefill(_dev(qkv, torch.float32), _dev(kcache, torch.bfloat16), _dev(vcache, torch.bfloat16),
                                out.data_ptr(), out_lo.data_ptr(), batch, T, n_q_heads, nkv, max_seq, n_past,
                                _stream_ptr()), "nnc_op_attn_prefill")
    return out, out_lo


def op_attn_prefill_f16(qkv: torch.Tensor, k16: torch.Tensor, v16: torch.Tensor, T: int, n_q_heads: int, n_past: int):
    """nnc_op_attn_prefill_f16; k16, v16 fp16 [batch][n_kv_heads][max_seq][128]; returns fp16 [batch * T][n_q_heads * 128]."""
    batch, nkv, max_seq, _ = k16.shape
    out = torch.empty(batch * T, n_q_heads * 128, dtype=torch.float16, device="cuda")
    _ok(lib.nnc_op_attn_prefill_f16(_dev(qkv, torch.float32), _dev(k16, torch.float16), _dev(v16, torch.float16), out.data_ptr(),
                                    batch, T, n_q_heads, nkv, max_seq, n_past, _stream_ptr()), "nnc_op_attn_prefill_f16")
    return out
