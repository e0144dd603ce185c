"""Kernel-level parity: each CUDA operation, called through the C ABI, against the oracle's matching function
on the same seeded inputs.  Sizes span several tiles and ragged tails."""
import math

import pytest
import torch

from gpu_util import split_bf16
from paper_2512_21571_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nnc():
    from paper_2512_21571_b200 import binding
    return binding


def _w(seed, stream, shape, sigma=0.02):
    return synth.normal(seed, stream, shape, sigma, torch.bfloat16, "cuda")


@pytest.mark.parametrize("n_out,n_in", [(8, 64), (1000, 384), (4096, 1024), (6144, 4096), (1024, 3072), (2050, 640)])
def test_gemv_store_and_residual(nnc, oracle_mod, n_out, n_in):
    W = _w(1, 1, (n_out, n_in))
    x = synth.normal(1, 2, (n_in,), 1.0, torch.float32, "cuda")
    want = oracle_mod.matmul(W.cpu(), x.cpu().view(1, -1))[0]
    y = nnc.op_gemv(W, x, mode=0)
    assert torch.allclose(y.cpu(), want, rtol=1e-4, atol=2e-5 * math.sqrt(n_in))
    base = synth.normal(1, 3, (n_out,), 1.0, torch.float32, "cuda")
    y2 = nnc.op_gemv(W, x, mode=1, y=base.clone())
    assert torch.allclose(y2.cpu(), base.cpu() + want, rtol=1e-4, atol=2e-5 * math.sqrt(n_in))


@pytest.mark.parametrize("n_out,n_in", [(1024, 256), (6144, 1024), (24576, 4096), (1280, 384)])
def test_gemv_norm_prologue_and_swiglu(nnc, oracle_mod, n_out, n_in):
    W = _w(2, 1, (n_out, n_in))
    x = synth.normal(2, 2, (n_in,), 3.0, torch.float32, "cuda")
    gain = (1.0 + synth.normal(2, 3, (n_in,), 0.1, torch.float32, "cuda")).to(torch.bfloat16)
    h = oracle_mod.rmsnorm(x.cpu(), gain.cpu(), 1e-6)
    # rows interleaved gate/up
    full = oracle_mod.matmul(W.cpu(), h.view(1, -1))[0]
    y = nnc.op_gemv(W, x, mode=0, gain=gain, eps=1e-6)
    assert torch.allclose(y.cpu(), full, rtol=1e-4, atol=1e-4)
    want = torch.tensor([oracle_mod.silu(float(g)) * float(u) for g, u in zip(full[0::2], full[1::2])])
    a = nnc.op_gemv(W, x, mode=2, gain=gain, eps=1e-6)
    assert a.shape == (n_out // 2,)
    assert torch.allclose(a.cpu(), want, rtol=1e-4, atol=1e-5)


def test_gemv_identity_and_one_hot(nnc):
    n = 256
    eye = torch.eye(n, dtype=torch.bfloat16, device="cuda")
    x = synth.normal(3, 1, (n,), 1.0, torch.float32, "cuda")
    assert torch.equal(nnc.op_gemv(eye, x), x)
    W = _w(3, 2, (512, n))
    e = torch.zeros(n, device="cuda"); e[37] = 1.0
    assert torch.equal(nnc.op_gemv(W, e), W[:, 37].float())


@pytest.mark.parametrize("T,N,K", [(1, 256, 64), (7, 384, 256), (32, 1024, 256), (33, 1000, 640), (64, 512, 128),
                                   (100, 2048, 1024), (128, 256, 64), (129, 1280, 384), (300, 6144, 1024),
                                   (1000, 1000, 512), (513, 24576, 256)])
def test_gemm_tensor_core_against_oracle_matmul(nnc, oracle_mod, T, N, K):
    X = synth.normal(4, 1, (T, K), 1.0, torch.bfloat16, "cuda")
    W = _w(4, 2, (N, K))
    Y = nnc.op_gemm(X, W, out_f32=True)
    torch.cuda.synchronize()
    assert nnc.op_status() == 0
    rows = sorted(set([0, T - 1, T // 2] + list(range(0, T, max(1, T // 5)))))
    want = oracle_mod.matmul(W.cpu(), X[rows].float().cpu())
    assert torch.allclose(Y[rows].cpu(), want, rtol=1e-4, atol=2e-5 * math.sqrt(K))
    # every element against a float64 product on the device (same operands), to catch misplaced tiles
    ref = (X.double() @ W.double().T)
    assert (Y.double() - ref).abs().max().item() < 2e-5 * math.sqrt(K)
    Yb = nnc.op_gemm(X, W, out_f32=False)
    assert torch.allclose(Yb.float(), ref.float(), rtol=1e-2, atol=1e-3)
    acc = synth.normal(4, 3, (T, N), 1.0, torch.float32, "cuda")
    Y2 = nnc.op_gemm(X, W, accumulate_into=acc.clone())
    assert (Y2.double() - (acc.double() + ref)).abs().max().item() < 1e-4 * math.sqrt(K)
    assert nnc.op_status() == 0


@pytest.mark.parametrize("T,N,K", [(5, 512, 256), (64, 1024, 128), (130, 1280, 384), (400, 6144, 1024)])
def test_gemm_swiglu_epilogue(nnc, oracle_mod, T, N, K):
    X = synth.normal(5, 1, (T, K), 1.0, torch.bfloat16, "cuda")
    W = _w(5, 2, (N, K), sigma=0.1)
    A = nnc.op_gemm_swiglu(X, W)
    rows = [0, T - 1, T // 3]
    full = oracle_mod.matmul(W.cpu(), X[rows].float().cpu())
    g, u = full[:, 0::2], full[:, 1::2]
    want = g / (1 + torch.exp(-g)) * u
    assert A.shape == (T, N // 2)
    assert torch.allclose(A[rows].float().cpu(), want, rtol=1e-2, atol=2e-3)
    ref = X.double() @ W.double().T
    refa = (ref[:, 0::2] / (1 + torch.exp(-ref[:, 0::2])) * ref[:, 1::2]).float()
    assert torch.allclose(A.float(), refa, rtol=1e-2, atol=2e-3)
    assert nnc.op_status() == 0


@pytest.mark.parametrize("batch,nq,nkv,n_ctx,max_seq", [(1, 2, 1, 1, 8), (1, 16, 8, 129, 256), (2, 4, 4, 17, 64),
                                                         (1, 32, 8, 4097, 4224), (3, 8, 1, 1000, 1024),
                                                         (1, 16, 8, 777, 8192)])
def test_attn_decode_against_oracle(nnc, oracle_mod, batch, nq, nkv, n_ctx, max_seq):
    q = synth.normal(6, 1, (batch, nq, 128), 1.0, torch.float32, "cuda")
    kc = synth.normal(6, 2, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    vc = synth.normal(6, 3, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    # positions beyond n_ctx hold NaN bit patterns: they must never be read into the result
    kc[:, :, n_ctx:] = float("nan"); vc[:, :, n_ctx:] = float("nan")
    out = nnc.op_attn_decode(q, kc, vc, n_ctx)
    out2 = nnc.op_attn_decode(q, kc, vc, n_ctx)
    assert torch.equal(out, out2), "split-K combine must not depend on arrival order"
    G = nq // nkv
    qc, kcc, vcc = q.cpu(), kc.cpu(), vc.cpu()
    for b in range(batch):
        for i in sorted(set([0, nq - 1, nq // 2])):
            want = oracle_mod.attend(qc[b, i], kcc[b, i // G, :n_ctx].contiguous(), vcc[b, i // G, :n_ctx].contiguous())
            assert torch.allclose(out[b, i].cpu(), want, rtol=1e-4, atol=2e-5), (b, i)
    assert torch.isfinite(out).all()


@pytest.mark.parametrize("T,N,K", [(9, 512, 256), (64, 1024, 128), (100, 384, 640), (300, 2048, 1024), (1000, 1000, 512)])
def test_gemm_split_activations_recover_fp32_inputs(nnc, oracle_mod, T, N, K):
    """Feeding value + rounding residual as two bf16 operands reproduces the product of the fp32 activations
    (the oracle's matmul on the unrounded X) to ~2^-16, on both operand assignments (T <= 128 and T > 128)."""
    X = synth.normal(7, 1, (T, K), 1.0, torch.float32, "cuda")
    W = _w(7, 2, (N, K))
    hi, lo = split_bf16(X)
    Y = nnc.op_gemm(hi, W, X_lo=lo)
    rows = sorted(set([0, T - 1, T // 2]))
    want = oracle_mod.matmul(W.cpu(), X[rows].cpu())
    assert torch.allclose(Y[rows].cpu(), want, rtol=1e-4, atol=3e-5 * math.sqrt(K) * 0.02 * 50)
    ref = X.double() @ W.double().T
    err_split = (Y.double() - ref).abs().max().item()
    err_plain = (nnc.op_gemm(hi, W).double() - ref).abs().max().item()
    assert err_split < 2e-5 * math.sqrt(K) and err_split < err_plain / 20
    # SwiGLU epilogue with residual output (an output pitch that would misalign 16-byte stores is refused)
    if N % 16:
        with pytest.raises(nnc.NncError):
            nnc.op_gemm_swiglu(hi, W, X_lo=lo, want_lo=True)
        return
    A, A_lo = nnc.op_gemm_swiglu(hi, W, X_lo=lo, want_lo=True)
    refa = ref[:, 0::2] / (1 + torch.exp(-ref[:, 0::2])) * ref[:, 1::2]
    assert (A.double() + A_lo.double() - refa).abs().max().item() < 1e-4
    assert nnc.op_status() == 0


@pytest.mark.parametrize("T,N,K", [(32, 4096, 4096), (7, 384, 640), (128, 1024, 2048), (33, 1000, 1024), (32, 4096, 12288),
                                   (1, 128, 256), (64, 6144, 4096), (100, 24576, 1024), (32, 151936, 256), (17, 136, 8192)])
def test_gemm_split_k_for_few_tokens(nnc, oracle_mod, T, N, K):
    """Few tokens: the (output tile, K stage) list is cut into one contiguous range per CTA; tiles that straddle a
    cut are finished from fp32 partial tiles added in K order.  Covers a single tile with a single stage (one CTA),
    fewer tiles than SMs (every tile shared by several CTAs), more tiles than SMs (most tiles whole), ragged N and
    K that is not a multiple of the 4-slab stage.  Same result as the oracle's matmul, bit-identical from run to
    run, scratch flags left at zero."""
    X = synth.normal(8, 1, (T, K), 1.0, torch.float32, "cuda")
    W = _w(8, 2, (N, K))
    hi, lo = split_bf16(X)
    scratch = torch.zeros(16384 + (32 << 20), dtype=torch.uint8, device="cuda")
    Y = nnc.op_gemm_splitk(hi, W, scratch, X_lo=lo)
    Y2 = nnc.op_gemm_splitk(hi, W, scratch, X_lo=lo)
    torch.cuda.synchronize()
    assert nnc.op_status() == 0
    assert torch.equal(Y, Y2)
    assert int(scratch[:16384].max()) == 0
    rows = sorted(set([0, T - 1, T // 2]))
    want = oracle_mod.matmul(W.cpu(), X[rows].cpu())
    assert torch.allclose(Y[rows].cpu(), want, rtol=1e-4, atol=3e-5 * math.sqrt(K))
    ref = X.double() @ W.double().T
    assert (Y.double() - ref).abs().max().item() < 2e-5 * math.sqrt(K)
    acc = synth.normal(8, 3, (T, N), 1.0, torch.float32, "cuda")
    Y3 = nnc.op_gemm_splitk(hi, W, scratch, X_lo=lo, accumulate_into=acc.clone())
    assert (Y3.double() - (acc.double() + ref)).abs().max().item() < 1e-4 * math.sqrt(K)
    Yb = nnc.op_gemm_splitk(hi, W, scratch, out_f32=False)
    assert torch.allclose(Yb.float(), ref.float(), rtol=2e-2, atol=2e-2)


def test_quantise_rows_e4m3_matches_the_oracle_bit_for_bit(nnc, oracle_mod):
    """Codes, row exponents and dequantised values of the device quantiser equal the oracle's (integer / byte work:
    bit-exact), on random rows and on rows that sit on the rule's edges."""
    W = _w(51, 1, (300, 512))
    W[0] = 0                                  # all-zero row
    W[1, 7] = 448.0; W[2, 7] = 450.0          # a maximum that just fits / just does not
    W[3] = W[3] * 1e-30                       # tiny row: large negative exponent
    W[4, :16] = torch.tensor([1.0625, 1.1875, -1.0625, 2.0 ** -10, 3 * 2.0 ** -10, 7.5 * 2.0 ** -9, 1.9999, 0.0,
                              448.0, -448.0, 224.0, 0.4375, 0.001953125, -0.001953125, 1.0, 8.0])   # ties, subnormals
    W[5] = W[5] * 3e4                         # large row: positive exponent
    codes, scales, dq = nnc.op_quantise_rows_e4m3(W)
    torch.cuda.synchronize()
    oc, oe = oracle_mod.quantise_rows_e4m3(W.cpu())
    assert torch.equal(scales.cpu(), torch.exp2(oe.float()))
    assert torch.equal(codes.cpu(), oc)
    assert torch.equal(dq.cpu().view(torch.int16), oracle_mod.dequantise_rows_e4m3(oc, oe).view(torch.int16))
    # in place: the dequantised values may overwrite the input
    W2 = W.clone()
    import ctypes as C
    assert nnc.lib.nnc_op_quantise_rows_e4m3(W2.data_ptr(), codes.data_ptr(), scales.data_ptr(), W2.data_ptr(), 300, 512,
                                             torch.cuda.current_stream().cuda_stream) == 0
    torch.cuda.synchronize()
    assert torch.equal(W2, dq) and torch.equal(codes.cpu(), oc)


@pytest.mark.parametrize("n_out,n_in", [(16, 128), (1000, 384), (4096, 1024), (6144, 4096), (4096, 12288), (2050, 640)])
def test_gemv_fp8_against_oracle(nnc, oracle_mod, n_out, n_in):
    """Streaming GEMV on FP8 codes with row scales = the oracle's matmul on the dequantised matrix (store, residual,
    norm prologue); SwiGLU on interleaved rows."""
    W = _w(52, 1, (n_out, n_in))
    W[n_out // 2, 3] = 0.75                   # one row with an outlier: its scale differs from its neighbours'
    x = synth.normal(52, 2, (n_in,), 1.0, torch.float32, "cuda")
    codes, scales, dq = nnc.op_quantise_rows_e4m3(W)
    oc, oe = oracle_mod.quantise_rows_e4m3(W.cpu())
    D = oracle_mod.dequantise_rows_e4m3(oc, oe)
    assert torch.equal(codes.cpu(), oc)
    want = oracle_mod.matmul(D, x.cpu().view(1, -1))[0]
    tol = dict(rtol=1e-4, atol=2e-5 * math.sqrt(n_in))
    y = nnc.op_gemv_fp8(codes, scales, x, mode=0)
    assert torch.allclose(y.cpu(), want, **tol)
    base = synth.normal(52, 3, (n_out,), 1.0, torch.float32, "cuda")
    y1 = nnc.op_gemv_fp8(codes, scales, x, mode=1, y=base.clone())
    assert torch.allclose(y1.cpu(), base.cpu() + want, **tol)
    gain = (1.0 + synth.normal(52, 4, (n_in,), 0.1, torch.float32, "cuda")).to(torch.bfloat16)
    h = oracle_mod.rmsnorm(x.cpu(), gain.cpu(), 1e-6)
    want_n = oracle_mod.matmul(D, h.view(1, -1))[0]
    yn = nnc.op_gemv_fp8(codes, scales, x, mode=0, gain=gain)
    assert torch.allclose(yn.cpu(), want_n, **tol)
    if n_out % 2 == 0:
        g, u = want_n[0::2].double(), want_n[1::2].double()
        ya = nnc.op_gemv_fp8(codes, scales, x, mode=2, gain=gain)
        assert torch.allclose(ya.double().cpu(), g / (1 + torch.exp(-g)) * u, rtol=1e-4, atol=1e-4)


def test_f16_scaled_weight_copy_is_exact(nnc):
    """The fp16 copy holds W * 2^e exactly: dividing by the scale gives the bf16 values back, bit for bit -- also for
    a matrix whose columns are spread over 12 more binades and for one with a large outlier."""
    W = _w(31, 1, (512, 256))
    for case in range(3):
        M = W.clone()
        if case == 1:
            M[3, 5] = 96.0                                   # an outlier sets the scale
        if case == 2:
            M = (M.float() * torch.exp2(-torch.arange(256, device="cuda").float() % 12)).to(torch.bfloat16)
        h, scales = nnc.op_to_f16_scaled(M)
        torch.cuda.synchronize()
        sc, inv = scales.tolist()
        assert sc * inv == 1.0 and math.log2(sc) == int(math.log2(sc))
        amax = M.float().abs().max().item() * sc
        assert 2.0 ** 14 <= amax < 2.0 ** 15
        assert torch.equal(h.float() * inv, M.float())


@pytest.mark.parametrize("T,N,K", [(129, 256, 64), (300, 1000, 384), (1024, 512, 1024), (515, 264, 2048)])
def test_gemm_f16_against_oracle(nnc, oracle_mod, T, N, K):
    """One-term fp16 GEMM (the prompt-phase form): fp16 activations, scaled fp16 weight copy, scale undone in the
    epilogue.  The oracle multiplies the same values (fp16 activations are exact in fp32, weights are bf16)."""
    W = _w(32, 1, (N, K))
    X = synth.normal(32, 2, (T, K), 1.0, torch.float32, "cuda").to(torch.float16)
    W16, scales = nnc.op_to_f16_scaled(W)
    want = oracle_mod.matmul(W.cpu(), X.float().cpu())
    Y = nnc.op_gemm_f16(X, W16, out_scale=scales[1:])
    assert nnc.op_status() == 0
    assert torch.allclose(Y.cpu(), want, rtol=1e-4, atol=2e-5 * math.sqrt(K))
    acc = synth.normal(32, 3, (T, N), 1.0, torch.float32, "cuda")
    Y2 = nnc.op_gemm_f16(X, W16, out_scale=scales[1:], accumulate_into=acc.clone())
    assert torch.allclose(Y2.cpu(), acc.cpu() + want, rtol=1e-4, atol=2e-5 * math.sqrt(K))
    if N % 16 == 0:
        A = nnc.op_gemm_swiglu_f16(X, W16, out_scale=scales[1:])
        g, u = want[:, 0::2].double(), want[:, 1::2].double()
        ref = g / (1 + torch.exp(-g)) * u
        # one fp16 rounding of the result (2^-11 relative) on top of the fp32 accumulation noise
        assert torch.allclose(A.double().cpu(), ref, rtol=1e-3, atol=1e-4 * math.sqrt(K) * 0.02 + 1e-6)
    assert nnc.op_status() == 0


@pytest.mark.parametrize("batch,T,nq,nkv,n_past,growth", [
    (1, 19, 2, 1, 0, 0.0), (2, 130, 4, 2, 7, 0.0), (1, 300, 8, 2, 0, 0.0), (1, 64, 16, 8, 200, 0.0),
    (1, 128, 1, 1, 0, 0.0), (1, 129, 2, 2, 127, 0.0),            # exactly one tile; one row past a tile boundary
    (1, 2048, 4, 1, 100, 0.0),                                    # the prompt length of the batched workload, with a past
    (1, 700, 2, 1, 60, 0.15), (1, 400, 2, 2, 0, 1.0),             # keys that grow along the sequence: the running maximum moves
    (1, 65, 2, 1, 63, 0.0), (2, 200, 4, 2, 33, 0.5)])             # pasts that end inside a 64-position step; two sequences, growing keys
def test_attn_prefill_against_oracle(nnc, oracle_mod, batch, T, nq, nkv, n_past, growth):
    """Causal prompt-phase attention: query s sees cache positions 0 .. n_past + s.  Rows are checked against the
    oracle's single-query attention over the matching cache prefix (sampled rows, all heads of those rows).  With
    `growth` the keys of each further block of 128 positions are larger, so a later tile's score maximum exceeds the
    running one by a little (0.15) or by far (1.0) and the accumulator is rescaled on the way."""
    max_seq = n_past + T + 5
    heads = nq + 2 * nkv
    qkv = synth.normal(9, 1, (batch * T, heads * 128), 1.0, torch.float32, "cuda")
    kc = synth.normal(9, 2, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    vc = synth.normal(9, 3, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    if growth:
        blk = (torch.arange(max_seq, device="cuda") // 128).float()
        kc = (kc.float() * (1.0 + growth * blk).view(1, 1, -1, 1)).to(torch.bfloat16).contiguous()
    kc[:, :, n_past + T:] = float("nan"); vc[:, :, n_past + T:] = float("nan")   # never to be read into a result
    out, out_lo = nnc.op_attn_prefill(qkv, kc, vc, T, nq, n_past)
    # the one-term fp16 form on the fp16 image of the same cache (bf16 values of this size are exact in fp16)
    out16 = nnc.op_attn_prefill_f16(qkv, kc.to(torch.float16), vc.to(torch.float16), T, nq, n_past)
    torch.cuda.synchronize()
    got = (out.float() + out_lo.float()).cpu().view(batch, T, nq, 128)
    got16 = out16.float().cpu().view(batch, T, nq, 128)
    assert torch.isfinite(got).all() and torch.isfinite(got16).all()
    G = nq // nkv
    qc, kcc, vcc = qkv.cpu().view(batch, T, heads, 128), kc.cpu(), vc.cpu()
    for b in range(batch):
        for s in sorted(set([0, 1, T // 2, T - 1, min(T - 1, 127), min(T - 1, 128), min(T - 1, 255), (2 * T) // 3])):
            n = n_past + s + 1
            for h in range(nq):
                want = oracle_mod.attend(qc[b, s, h].contiguous(), kcc[b, h // G, :n].contiguous(), vcc[b, h // G, :n].contiguous())
                assert torch.allclose(got[b, s, h], want, rtol=1e-3, atol=1e-4), (b, s, h)
                # one fp16 rounding of q (2^-11 on a score of size ~|q||k|/sqrt(d)), of p and of the output
                assert torch.allclose(got16[b, s, h], want, rtol=1e-2, atol=1e-2 * (1.0 + growth * 8)), (b, s, h, "f16")
