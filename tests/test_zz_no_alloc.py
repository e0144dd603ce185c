"""The allocation-free flash-decode entry point, nnc_op_attn_decode_static, through the C ABI.

It exists for callers that cannot allocate device memory (a plug-in that only receives its inputs and outputs,
a process whose memory pool belongs to another runtime): the split-K scratch lives in a fixed array inside the
library.  Its result must equal the CPU oracle's attention (and the caller-scratch entry point's), also on a
second call that finds the first call's leftovers in the shared array, and the call itself must leave the
device's free memory untouched.  Collected last on purpose (file name), so a failure here cannot hide the outcome
of any other test in a run that stops at the first failure.
"""
import ctypes as C

import pytest
import torch

from paper_2512_21571_b200 import synth


def _oracle_attention(oracle_mod, q, kc, vc, n_ctx):
    """out[b][h] = oracle.attend(q[b][h], K, V of KV head h // G), positions [0, n_ctx)."""
    batch, nq, _ = q.shape
    G = nq // kc.shape[1]
    qc, kcc, vcc = q.cpu(), kc.cpu(), vc.cpu()
    out = torch.empty_like(qc)
    for b in range(batch):
        for h in range(nq):
            out[b, h] = oracle_mod.attend(qc[b, h].contiguous(), kcc[b, h // G, :n_ctx].contiguous(),
                                          vcc[b, h // G, :n_ctx].contiguous())
    return out


@pytest.mark.gpu
def test_static_scratch_variant_matches_the_oracle_and_the_caller_scratch_variant_twice(oracle_mod):
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
        assert torch.allclose(got.cpu(), _oracle_attention(oracle_mod, q, kc, vc, n_ctx), rtol=1e-4, atol=2e-5), \
            (batch, nq, n_ctx)
    # and once more on the first shape, now that the array holds the second call's partials
    batch, nq, nkv, n_ctx, max_seq, seed = cases[0]
    q = synth.normal(seed, 1, (batch, nq, 128), 1.0, torch.float32, "cuda")
    kc = synth.normal(seed, 2, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    vc = synth.normal(seed, 3, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    assert torch.allclose(nnc.op_attn_decode_static(q, kc, vc, n_ctx), nnc.op_attn_decode(q, kc, vc, n_ctx),
                          rtol=1e-4, atol=2e-5)


@pytest.mark.gpu
def test_static_scratch_call_allocates_nothing_and_covers_its_stated_capacity(oracle_mod):
    """The C entry point is called directly on tensors that exist beforehand: the device's free memory must read
    the same before and after.  The largest batch * n_q_heads the built-in array holds still works (checked against
    the oracle on one sequence), the next size up is refused."""
    from paper_2512_21571_b200 import binding as nnc
    nq, nkv, n_ctx, max_seq = 32, 8, 777, 1024
    cap = nnc.lib.nnc_attn_scratch_bytes
    limit = 4 << 20
    batch = 1
    while cap(batch + 1, nq, n_ctx) <= limit:
        batch += 1
    assert cap(batch, nq, n_ctx) <= limit < cap(batch + 1, nq, n_ctx)
    q = synth.normal(31, 1, (batch + 1, nq, 128), 1.0, torch.float32, "cuda")
    kc = synth.normal(31, 2, (batch + 1, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    vc = synth.normal(31, 3, (batch + 1, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    out = torch.zeros_like(q)
    stream = torch.cuda.current_stream().cuda_stream

    def call(b):
        return nnc.lib.nnc_op_attn_decode_static(q.data_ptr(), kc.data_ptr(), vc.data_ptr(), out.data_ptr(), b, nq, nkv,
                                                 max_seq, n_ctx, stream)

    assert call(batch) == 0          # first call on this device: looks up the array's address
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    assert call(batch) == 0
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    for b in (0, batch - 1):
        want = _oracle_attention(oracle_mod, q[b:b + 1], kc[b:b + 1], vc[b:b + 1], n_ctx)
        assert torch.allclose(out[b:b + 1].cpu(), want, rtol=1e-4, atol=2e-5), b
    assert call(batch + 1) == -3     # NNC_ERR_CAPACITY: one sequence more than the array holds


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
