"""The allocation-free flash-decode entry point, nnc_op_attn_decode_static, through the C ABI.

It exists for callers that cannot allocate device memory (a plug-in that only receives its inputs and outputs,
a process whose memory pool belongs to another runtime): the split-K scratch lives in a fixed array inside the
library.  Its result must equal the caller-scratch entry point's, also on a second call that finds the first
call's leftovers in the shared array.  Collected last on purpose (file name), so a failure here cannot hide
the outcome of any other test in a run that stops at the first failure.
"""
import ctypes as C

import pytest
import torch

from paper_2512_21571_b200 import synth


@pytest.mark.gpu
def test_static_scratch_variant_matches_caller_scratch_variant_twice():
    from paper_2512_21571_b200 import binding as nnc
    cases = [(1, 32, 8, 4097, 4224, 21), (2, 16, 8, 333, 512, 22)]   # second call: other shape, other data
    for batch, nq, nkv, n_ctx, max_seq, seed in cases:
        q = synth.normal(seed, 1, (batch, nq, 128), 1.0, torch.float32, "cuda")
        kc = synth.normal(seed, 2, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
        vc = synth.normal(seed, 3, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
        want = nnc.op_attn_decode(q, kc, vc, n_ctx)
        got = nnc.op_attn_decode_static(q, kc, vc, n_ctx)
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        assert torch.allclose(got, want, rtol=1e-4, atol=2e-5), (batch, nq, n_ctx)
    # and once more on the first shape, now that the array holds the second call's partials
    batch, nq, nkv, n_ctx, max_seq, seed = cases[0]
    q = synth.normal(seed, 1, (batch, nq, 128), 1.0, torch.float32, "cuda")
    kc = synth.normal(seed, 2, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    vc = synth.normal(seed, 3, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    assert torch.allclose(nnc.op_attn_decode_static(q, kc, vc, n_ctx), nnc.op_attn_decode(q, kc, vc, n_ctx),
                          rtol=1e-4, atol=2e-5)


def test_static_scratch_variant_refuses_oversized_problems_on_the_host():
    """The size check comes before any CUDA call, so it runs without a GPU: dummy non-null pointers are never
    dereferenced."""
    from paper_2512_21571_b200 import build
    build.build()
    from paper_2512_21571_b200 import binding as nnc
    dummy = C.c_void_p(256)
    too_big = nnc.lib.nnc_op_attn_decode_static(dummy, dummy, dummy, dummy, 64, 32, 8, 128, 64, None)
    assert too_big == -3   # NNC_ERR_CAPACITY
    assert nnc.lib.nnc_op_attn_decode_static(dummy, dummy, dummy, dummy, 1, 30, 8, 128, 64, None) == -1
    assert nnc.lib.nnc_op_attn_decode_static(None, dummy, dummy, dummy, 1, 32, 8, 128, 64, None) == -1
