"""Pins for the CPU oracle: closed forms, invariants, textbook special cases and an independent unfused
float64 numpy forward.  Nothing here compares the oracle with itself through the same formula, and nothing
touches the CUDA path."""
import dataclasses
import math

import numpy as np
import pytest
import torch

import ref_numpy
from paper_2512_21571_b200 import synth

SMALL = synth.ModelShape(n_layers=2, hidden=16, n_q_heads=4, n_kv_heads=2, head_dim=8, intermediate=24,
                         vocab=32, tie_embeddings=True)
SMALL_UNTIED = dataclasses.replace(SMALL, n_layers=3, tie_embeddings=False, vocab=40)


def _weights(shape, seed, sigma=0.3, gains=True):
    w = synth.make_weights(shape, seed, sigma=sigma)
    if gains:
        synth.random_gains(w, seed + 1)
    return w


# ------------------------------------------------------------------------------------------------ bf16
def test_bf16_rounding_is_nearest_even(oracle_mod):
    L = oracle_mod.load()
    x = torch.cat([torch.randn(20000, generator=torch.Generator().manual_seed(0)) * 3,
                   torch.tensor([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, -2.5])])
    # exact ties: 1 + 2^-8 lies halfway between 1 and 1 + 2^-7 -> even mantissa (1.0)
    want = x.to(torch.bfloat16).view(torch.int16).numpy().astype(np.uint16)
    got = np.array([L.orc_f32_to_bf16(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)
    assert L.orc_f32_to_bf16(1.00390625) == 0x3F80 and L.orc_f32_to_bf16(1.01171875) == 0x3F82
    assert L.orc_bf16_to_f32(0x3FC0) == 1.5


# --------------------------------------------------------------------------------------------- RMSNorm
def test_rmsnorm_constant_vector_closed_form(oracle_mod):
    for c in (3.0, -0.25, 1e-3):
        n, eps = 64, 1e-6
        y = oracle_mod.rmsnorm(torch.full((n,), c), torch.ones(n, dtype=torch.bfloat16), eps)
        want = c / math.sqrt(c * c + eps)
        assert torch.allclose(y, torch.full((n,), want), rtol=1e-6, atol=0)


def test_rmsnorm_unit_rms_scale_invariance_and_gain(oracle_mod):
    g = torch.Generator().manual_seed(1)
    x = torch.randn(1024, generator=g)
    ones = torch.ones(1024, dtype=torch.bfloat16)
    y = oracle_mod.rmsnorm(x, ones, 1e-6)
    assert abs(y.double().pow(2).mean().sqrt().item() - 1.0) < 1e-5
    assert torch.allclose(oracle_mod.rmsnorm(x * 37.0, ones, 1e-6), y, rtol=1e-5, atol=1e-6)
    # no mean subtraction: a shifted vector keeps its mean direction
    assert oracle_mod.rmsnorm(x + 10.0, ones, 1e-6).mean().item() > 0.9
    gain = (torch.rand(1024, generator=g) + 0.5).to(torch.bfloat16)
    assert torch.allclose(oracle_mod.rmsnorm(x, gain, 1e-6), y * gain.float(), rtol=1e-6, atol=1e-7)
    # eps sits inside the root: a zero vector maps to zero, a tiny one is damped by sqrt(eps)
    tiny = torch.full((8,), 1e-4)
    assert torch.allclose(oracle_mod.rmsnorm(tiny, torch.ones(8, dtype=torch.bfloat16), 1e-6),
                          tiny / math.sqrt(1e-8 + 1e-6), rtol=1e-5)


# ------------------------------------------------------------------------------------------------ RoPE
def test_rope_table_values(oracle_mod):
    d, theta = 128, 1e6
    t = oracle_mod.rope_table(2049, d, theta)
    assert torch.equal(t[0, :, 0], torch.ones(64)) and torch.equal(t[0, :, 1], torch.zeros(64))
    # pair 0 has inverse frequency 1: position p rotates it by p radians
    assert t[1, 0, 0].item() == np.float32(math.cos(1.0)) and t[1, 0, 1].item() == np.float32(math.sin(1.0))
    assert abs(t[2048, 0, 1].item() - math.sin(2048.0)) < 1e-6
    # pair 32 has inverse frequency theta^-0.5 = 1e-3: position 1000 rotates it by one radian
    assert abs(t[1000, 32, 0].item() - math.cos(1.0)) < 1e-6
    # last pair: theta^(-126/128)
    assert abs(t[500, 63, 1].item() - math.sin(500 * theta ** (-126 / 128))) < 1e-7


def test_rope_pairing_norm_and_relative_property(oracle_mod):
    d = 128
    t = oracle_mod.rope_table(300, d, 1e6)
    e0 = torch.zeros(d); e0[0] = 1.0
    y = oracle_mod.rope_apply(e0, t[1])
    # half-split pairing: element 0 rotates into element d/2, by +1 radian
    want = torch.zeros(d); want[0] = math.cos(1.0); want[64] = math.sin(1.0)
    assert torch.allclose(y, want, atol=1e-7)
    e64 = torch.zeros(d); e64[64] = 1.0
    y = oracle_mod.rope_apply(e64, t[1])
    want = torch.zeros(d); want[0] = -math.sin(1.0); want[64] = math.cos(1.0)
    assert torch.allclose(y, want, atol=1e-7)
    g = torch.Generator().manual_seed(2)
    q, k = torch.randn(d, generator=g), torch.randn(d, generator=g)
    assert torch.equal(oracle_mod.rope_apply(q, t[0]), q)
    assert abs(oracle_mod.rope_apply(q, t[77]).norm().item() - q.norm().item()) < 1e-4
    a = torch.dot(oracle_mod.rope_apply(q, t[10]), oracle_mod.rope_apply(k, t[3]))
    b = torch.dot(oracle_mod.rope_apply(q, t[210]), oracle_mod.rope_apply(k, t[203]))
    assert abs(a.item() - b.item()) < 2e-4


# ------------------------------------------------------------------------------------- softmax, attention
def test_softmax_rows_sum_to_one_and_shift_invariant(oracle_mod):
    g = torch.Generator().manual_seed(3)
    s = torch.randn(777, generator=g) * 4
    p = oracle_mod.softmax(s)
    assert abs(p.double().sum().item() - 1.0) < 1e-6 and torch.all(p >= 0)
    assert torch.allclose(oracle_mod.softmax(s + 50.0), p, rtol=2e-5, atol=1e-9)
    assert torch.allclose(p, torch.softmax(s.double(), 0).float(), rtol=1e-5, atol=1e-9)
    # large scores do not overflow (maximum is subtracted)
    assert torch.isfinite(oracle_mod.softmax(torch.tensor([1000.0, 999.0]))).all()
    two = oracle_mod.softmax(torch.tensor([math.log(3.0), 0.0]))
    assert torch.allclose(two, torch.tensor([0.75, 0.25]), atol=1e-6)


def test_attention_special_cases(oracle_mod):
    d = 128
    g = torch.Generator().manual_seed(4)
    q = torch.randn(d, generator=g)
    K = torch.randn(9, d, generator=g).to(torch.bfloat16)
    V = torch.randn(9, d, generator=g).to(torch.bfloat16)
    # one cached token: the output is that token's V exactly
    assert torch.equal(oracle_mod.attend(q, K[:1].contiguous(), V[:1].contiguous()), V[0].float())
    # identical keys: uniform weights, output = mean of V
    Ksame = K[:1].repeat(9, 1).contiguous()
    assert torch.allclose(oracle_mod.attend(q, Ksame, V), V.float().mean(0), atol=1e-6)
    # the 1/sqrt(d) scale: q = sqrt(d) ln3 e_0 against keys e_0 and 0 gives weights 3/4, 1/4
    q2 = torch.zeros(d); q2[0] = math.sqrt(d) * math.log(3.0)
    K2 = torch.zeros(2, d); K2[0, 0] = 1.0
    V2 = torch.zeros(2, d); V2[0, 5] = 1.0; V2[1, 5] = -1.0
    o = oracle_mod.attend(q2, K2.to(torch.bfloat16), V2.to(torch.bfloat16))
    assert abs(o[5].item() - 0.5) < 1e-6
    # general case against float64 numpy
    s = (K.double() @ q.double()) / math.sqrt(d)
    want = torch.softmax(s, 0) @ V.double()
    assert torch.allclose(oracle_mod.attend(q, K, V).double(), want, atol=1e-5)


def test_silu_and_argmax(oracle_mod):
    assert oracle_mod.silu(0.0) == 0.0
    assert abs(oracle_mod.silu(1.0) - 0.7310585786) < 1e-7
    assert abs(oracle_mod.silu(-1.0) + 0.2689414214) < 1e-7
    assert abs(oracle_mod.silu(30.0) - 30.0) < 1e-5 and abs(oracle_mod.silu(-30.0)) < 1e-10
    idx, margin = oracle_mod.argmax_margin(torch.tensor([0.5, 2.0, -1.0, 2.0, 1.5]))
    assert idx == 1 and margin == 0.0
    idx, margin = oracle_mod.argmax_margin(torch.tensor([0.5, 2.0, -1.0, 2.25, 1.5]))
    assert idx == 3 and margin == 0.25
    # non-finite logits are an error, never a rank
    for bad in (float("nan"), float("inf"), float("-inf")):
        with pytest.raises(ValueError):
            oracle_mod.argmax_margin(torch.tensor([0.5, bad, 1.0]))


# ----------------------------------------------------------------------------------------------- matmul
def test_matmul_identity_onehot_and_bruteforce(oracle_mod):
    n = 48
    eye = torch.eye(n).to(torch.bfloat16)
    g = torch.Generator().manual_seed(5)
    X = torch.randn(3, n, generator=g)
    assert torch.equal(oracle_mod.matmul(eye, X), X)
    W = (torch.randn(20, n, generator=g) * 0.1).to(torch.bfloat16)
    onehot = torch.zeros(1, n); onehot[0, 7] = 1.0
    assert torch.equal(oracle_mod.matmul(W, onehot)[0], W[:, 7].float())   # a weight COLUMN: y = W x
    want = np.zeros((3, 20))
    Wd, Xd = W.double().numpy(), X.double().numpy()
    for t in range(3):
        for o in range(20):
            for k in range(n):
                want[t, o] += Wd[o, k] * Xd[t, k]
    assert np.allclose(oracle_mod.matmul(W, X).numpy(), want, atol=1e-5)


# ------------------------------------------------------------------------------------------ whole model
@pytest.mark.parametrize("shape,seed", [(SMALL, 11), (SMALL_UNTIED, 12)])
def test_model_matches_unfused_numpy_forward(oracle_mod, shape, seed):
    w = _weights(shape, seed)
    toks = synth.prompt_tokens(shape, seed, 7)
    want_logits, want_taps, ks, vs = ref_numpy.forward(shape, w, toks.tolist())
    for dbl in (False, True):
        m = oracle_mod.Oracle(shape, w, max_seq=16, double_acc=dbl)
        logits, taps = m.forward(toks, all_positions=True, want_taps=True)
        tol = 1e-9 if dbl else 3e-5
        # (bf16 cache rounding can flip on a 1-ulp fp32 difference, so the fp64 build is the sharp check
        #  only up to such flips; none occur for these seeds)
        assert np.abs(taps.double().numpy() - want_taps).max() < max(tol, 2e-6) * np.abs(want_taps).max()
        assert np.abs(logits.double().numpy() - want_logits).max() < 5e-5
        k0, v0 = m.kv_export(0, 7)
        assert np.array_equal(k0.double().numpy(), ks[0]) and np.array_equal(v0.double().numpy(), vs[0])
        m.close()


def test_prefill_equals_stepwise_decode(oracle_mod):
    shape, seed = SMALL_UNTIED, 21
    w = _weights(shape, seed)
    toks = synth.prompt_tokens(shape, seed, 9)
    a = oracle_mod.Oracle(shape, w, max_seq=16)
    la, ta = a.forward(toks, all_positions=True, want_taps=True)
    b = oracle_mod.Oracle(shape, w, max_seq=16)
    for i in range(9):
        lb, tb = b.forward(toks[i:i + 1], want_taps=True)
        assert torch.allclose(lb, la[i], atol=1e-5)
        assert torch.allclose(tb[:, 0], ta[:, i], atol=1e-5)
    assert b.length == 9
    for l in range(shape.n_layers):
        ka, va = a.kv_export(l, 9)
        kb, vb = b.kv_export(l, 9)
        assert torch.equal(ka, kb) and torch.equal(va, vb)
    # split in two calls as well: 4 tokens, then 5
    c = oracle_mod.Oracle(shape, w, max_seq=16)
    c.forward(toks[:4])
    lc, _ = c.forward(toks[4:], all_positions=True)
    assert torch.allclose(lc, la[4:], atol=1e-5)


def test_kv_import_continues_like_numpy_with_past(oracle_mod):
    shape, seed = SMALL, 31
    w = _weights(shape, seed)
    P = 5
    past = [synth.kv_fill(shape, seed, l, P) for l in range(shape.n_layers)]
    m = oracle_mod.Oracle(shape, w, max_seq=16)
    for l, (k, v) in enumerate(past):
        m.kv_import(l, k, v)
    toks = synth.prompt_tokens(shape, seed, 3)
    logits, taps = m.forward(toks, all_positions=True, want_taps=True)
    want_logits, want_taps, _, _ = ref_numpy.forward(
        shape, w, toks.tolist(), [k.double().numpy() for k, _ in past], [v.double().numpy() for _, v in past])
    assert np.abs(logits.double().numpy() - want_logits).max() < 5e-5
    assert np.abs(taps.double().numpy() - want_taps).max() < 5e-5 * np.abs(want_taps).max()
    assert m.length == P + 3


def test_layer_decode_matches_numpy_layer(oracle_mod):
    """One layer, one step on a given hidden vector (the single-layer workload): position = cache length."""
    shape = dataclasses.replace(SMALL, n_layers=1)
    w = _weights(shape, 41)
    P = 6
    k, v = synth.kv_fill(shape, 41, 0, P)
    m = oracle_mod.Oracle(shape, w, max_seq=8)
    m.kv_import(0, k, v)
    x = synth.hidden_state(shape, 41)
    y = m.layer_decode(0, x)
    assert m.length == P + 1
    # numpy: feed x through a fake one-row embedding
    w2 = dict(w); w2["embed"] = x.view(1, -1)  # fp32 tensor, _f64 handles it
    _, taps, _, _ = ref_numpy.forward(shape, w2, [0], [k.double().numpy()], [v.double().numpy()])
    assert np.abs(y.double().numpy() - taps[1, 0]).max() < 5e-5 * np.abs(taps[1]).max()


def test_gqa_equals_mha_with_replicated_kv_heads(oracle_mod):
    shape, seed = SMALL, 51
    w = _weights(shape, seed)
    toks = synth.prompt_tokens(shape, seed, 6)
    a, _ = oracle_mod.Oracle(shape, w, 8).forward(toks, all_positions=True)
    G, d = shape.n_q_heads // shape.n_kv_heads, shape.head_dim
    mha = dataclasses.replace(shape, n_kv_heads=shape.n_q_heads)
    w2 = dict(w); w2["layers"] = []
    for lw in w["layers"]:
        lw2 = dict(lw)
        for n in ("wk", "wv"):
            lw2[n] = lw[n].view(shape.n_kv_heads, d, -1).repeat_interleave(G, dim=0).reshape(-1, shape.hidden).contiguous()
        w2["layers"].append(lw2)
    b, _ = oracle_mod.Oracle(mha, w2, 8).forward(toks, all_positions=True)
    assert torch.allclose(a, b, atol=1e-6)


def test_zero_layers_closed_form_and_vocab_permutation(oracle_mod):
    shape, seed = SMALL, 61
    w = _weights(shape, seed)
    for lw in w["layers"]:
        for n in ("wo", "w_down"):
            lw[n] = torch.zeros_like(lw[n])
    toks = synth.prompt_tokens(shape, seed, 4)
    logits, _ = oracle_mod.Oracle(shape, w, 8).forward(toks, all_positions=True)
    E = w["embed"].double().numpy()
    x = E[toks.numpy()]
    want = ref_numpy.rmsnorm(x, w["g_final"].double().numpy(), shape.rms_eps) @ E.T
    assert np.abs(logits.double().numpy() - want).max() < 1e-5
    # permuting lm_head rows permutes the logits (untied head)
    shape2 = SMALL_UNTIED
    w2 = _weights(shape2, seed)
    toks2 = synth.prompt_tokens(shape2, seed, 4)
    base, _ = oracle_mod.Oracle(shape2, w2, 8).forward(toks2)
    perm = torch.randperm(shape2.vocab, generator=torch.Generator().manual_seed(0))
    w3 = dict(w2); w3["lm_head"] = w2["lm_head"][perm].contiguous()
    out, _ = oracle_mod.Oracle(shape2, w3, 8).forward(toks2)
    assert torch.equal(out, base[perm])


def test_fp32_and_fp64_accumulation_agree(oracle_mod):
    """The oracle's own rounding-order error bar on a library-sized shape, far below the parity tolerances."""
    shape = synth.SHAPES["tiny"]
    w = synth.make_weights(shape, 71)
    toks = synth.prompt_tokens(shape, 71, 12)
    a, ta = oracle_mod.Oracle(shape, w, 16).forward(toks, all_positions=True, want_taps=True)
    b, tb = oracle_mod.Oracle(shape, w, 16, double_acc=True).forward(toks, all_positions=True, want_taps=True)
    rel = ((ta - tb).double().norm(dim=-1) / tb.double().norm(dim=-1)).max().item()
    assert rel < 1e-4 and (a - b).abs().max().item() < 1e-3


def test_errors(oracle_mod):
    shape = SMALL
    w = _weights(shape, 81)
    m = oracle_mod.Oracle(shape, w, max_seq=4)
    with pytest.raises(ValueError):
        m.forward(torch.tensor([1, 2, 3, 4, 5], dtype=torch.int32))
    with pytest.raises(ValueError):
        m.forward(torch.tensor([shape.vocab], dtype=torch.int32))
    assert m.length == 0
