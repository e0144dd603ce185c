"""The seeded input generators: distribution, determinism, independence of chunking and of the device."""
import torch

from paper_2512_21571_b200 import synth


def test_table_is_monotone_symmetric_and_scaled():
    t = synth.normal_table(1.0, torch.float32).double()
    assert torch.all(t[1:] >= t[:-1])
    assert torch.allclose(t, -t.flip(0), atol=1e-6)
    # the median bins sit next to zero, the 84.13th percentile at one sigma
    assert abs(t[32768].item()) < 1e-4 and abs(t[int(0.841345 * 65536)].item() - 1.0) < 1e-3
    assert abs(t.std().item() - 1.0) < 2e-3
    t2 = synth.normal_table(0.02, torch.bfloat16)
    assert t2.dtype == torch.bfloat16 and abs(t2.float().std().item() - 0.02) < 1e-4


def test_normal_moments_and_determinism():
    x = synth.normal(7, 3, (1 << 22,), 0.02, torch.bfloat16).float()
    assert abs(x.mean().item()) < 5e-5 and abs(x.std().item() - 0.02) < 5e-5
    y = synth.normal(7, 3, (1 << 22,), 0.02, torch.bfloat16).float()
    assert torch.equal(x, y)
    z = synth.normal(8, 3, (1 << 22,), 0.02, torch.bfloat16).float()
    assert not torch.equal(x, z)
    # different streams are uncorrelated
    w = synth.normal(7, 4, (1 << 22,), 0.02, torch.bfloat16).float()
    assert abs((x * w).mean().item() / 0.02 ** 2) < 5e-3


def test_elements_do_not_depend_on_chunking(monkeypatch):
    a = synth.normal(1, 9, (3, 1000), 1.0, torch.float32)
    monkeypatch.setattr(synth, "_CHUNK", 257)
    b = synth.normal(1, 9, (3, 1000), 1.0, torch.float32)
    assert torch.equal(a, b)


def test_tokens_uniform_in_range():
    t = synth.tokens(5, 1, 200000, 151936)
    assert t.dtype == torch.int32 and int(t.min()) >= 0 and int(t.max()) < 151936
    assert int(t.max()) > 151000 and int(t.min()) < 1000
    hist = torch.bincount((t.long() * 16) // 151936, minlength=16).double()
    assert (hist / hist.sum() - 1 / 16).abs().max() < 3e-3


def test_weight_set_shapes_and_bytes():
    s = synth.SHAPES["tiny-untied"]
    w = synth.make_weights(s, 1)
    assert w["embed"].shape == (s.vocab, s.hidden) and w["lm_head"].shape == (s.vocab, s.hidden)
    lw = w["layers"][2]
    assert lw["wq"].shape == (s.q_dim, s.hidden) and lw["w_down"].shape == (s.hidden, s.intermediate)
    assert torch.all(lw["g_q"] == 1)
    assert not torch.equal(w["layers"][0]["wk"], w["layers"][0]["wv"])
    # bytes/step of the 8B shape: 15.137 GB of weights, 147456 B of cache per position
    big = synth.SHAPES["qwen3-8b"]
    assert abs(big.weight_bytes_per_decode_step() / 1e9 - 15.137) < 0.01
    assert big.kv_bytes_per_position() == 147456
