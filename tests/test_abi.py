"""The C-ABI library loads without a GPU, exports every symbol include/nnc.h declares, and its host-only
entry points (workspace sizing, argument validation, status strings) behave."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2512_21571_b200 import build
    build.build()
    from paper_2512_21571_b200 import binding as b
    return b


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "nnc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nnc_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    names = declared_symbols()
    assert "nnc_model_create" in names and "nnc_prefill" in names and "nnc_decode_step" in names
    for n in names:
        assert hasattr(binding.lib, n), f"{n} declared in nnc.h but not exported"
    assert set(names) == set(binding.EXPORTS), "binding and header disagree on the entry points"


def _cfg(binding, **kw):
    base = dict(n_layers=36, hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, intermediate=12288, vocab=151936,
                max_seq=4352, max_batch=1, max_tokens=1, tie_embeddings=0, rms_eps=1e-6, rope_theta=1e6,
                tc_operands=0, serial_launches=0)
    base.update(kw)
    return binding.nnc_config(**base)


def test_workspace_bytes_is_host_arithmetic(binding):
    c = _cfg(binding)
    n = binding.lib.nnc_workspace_bytes(C.byref(c))
    weights = 2 * (36 * ((4096 + 2048) * 4096 + 4096 * 4096 + 3 * 12288 * 4096) + 2 * 151936 * 4096)
    kv = 2 * 36 * 8 * 128 * 4352 * 2
    assert weights + kv < n < weights + kv + (1 << 28)
    assert n % 256 == 0
    # more cache -> more bytes, exactly
    n2 = binding.lib.nnc_workspace_bytes(C.byref(_cfg(binding, max_seq=8704)))
    assert n2 - n >= kv
    tied = binding.lib.nnc_workspace_bytes(C.byref(_cfg(binding, tie_embeddings=1)))
    assert n - tied == 151936 * 4096 * 2
    # prompt-phase capacity beyond 128 tokens adds, in operand mode 0 only, the fp16 copies of Wo, Wgate/up, Wdown and
    # the fp16 image of one layer's K and V rows
    big0 = binding.lib.nnc_workspace_bytes(C.byref(_cfg(binding, max_tokens=8192)))
    big1 = binding.lib.nnc_workspace_bytes(C.byref(_cfg(binding, max_tokens=8192, tc_operands=1)))
    assert big0 - big1 == 2 * 36 * (4096 * 4096 + 3 * 12288 * 4096) + 2 * (8 * 128 * 4352 * 2)


@pytest.mark.parametrize("bad", [dict(head_dim=64), dict(n_q_heads=30), dict(hidden=1000), dict(max_seq=0),
                                 dict(n_kv_heads=2), dict(max_tokens=0), dict(rms_eps=0.0), dict(vocab=-1),
                                 dict(tc_operands=3)])
def test_invalid_configs_are_rejected(binding, bad):
    assert binding.lib.nnc_workspace_bytes(C.byref(_cfg(binding, **bad))) == 0


def test_null_arguments_and_status_strings(binding):
    out = C.c_void_p()
    assert binding.lib.nnc_model_create(None, None, None, 0, None, C.byref(out)) == -1
    assert binding.lib.nnc_workspace_bytes(None) == 0
    assert binding.lib.nnc_get_length(None) == -1
    assert binding.lib.nnc_status_string(0) == b"ok"
    assert b"capacity" in binding.lib.nnc_status_string(-3)
    assert binding.lib.nnc_op_gemm(None, None, None, None, 1, 8, 64, 1, 0, None) == -1
    binding.lib.nnc_model_destroy(None)
