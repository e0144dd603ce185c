"""Seeded synthetic inputs for the Qwen3 forward pass: weights, KV-cache fill, hidden states, token ids.

This module serves both the CUDA path and the CPU oracle (through the tests and the bench) and contains
none of the model's arithmetic: it only turns (seed, stream, index) into numbers.  Every element is a pure
function of its index, so a tensor has the same bits whether it is produced on the CPU or on the GPU, in one
piece or in chunks.

Recipe (the paper evaluates trained Qwen3-0.6B / 1.7B checkpoints with an 8-token prompt, Section 4; those
are not available offline, so random-init tensors of the same shapes stand in for them):

  u      = splitmix64(seed * GOLDEN + stream * STREAM_MUL + index)         (64-bit counter hash)
  normal = TABLE_sigma[u >> 48],  TABLE_sigma[i] = sigma * Phi^-1((i + 0.5) / 65536)   (inverse-CDF table)
  token  = ((u >> 32) * vocab) >> 32                                      (uniform on [0, vocab))

The normal table is built once on the host in float64 and rounded to the target dtype, so a bf16 tensor holds
exact bf16 values and no later rounding step can differ between consumers.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List

import torch

_GOLDEN = -7046029254386353131          # 0x9E3779B97F4A7C15 as int64
_MUL1 = -4658895280553007687            # 0xBF58476D1CE4E5B9 as int64
_MUL2 = -7723592293110705685            # 0x94D049BB133111EB as int64
_STREAM_MUL = -3335678366873096957      # 0xD1B54A32D192ED03 as int64
_CHUNK = 1 << 24

_tables: Dict[tuple, torch.Tensor] = {}


def _wrap64(v: int) -> int:
    v &= (1 << 64) - 1
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(z: torch.Tensor, n: int) -> torch.Tensor:
    """Logical shift right of the 64-bit pattern held in an int64 tensor."""
    return (z >> n) & ((1 << (64 - n)) - 1)


def _splitmix64(z: torch.Tensor) -> torch.Tensor:
    z = z + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def _bits(seed: int, stream: int, start: int, count: int, device) -> torch.Tensor:
    base = _wrap64(seed * (_GOLDEN & ((1 << 64) - 1)) + stream * (_STREAM_MUL & ((1 << 64) - 1)) + start)
    idx = torch.arange(count, dtype=torch.int64, device=device) + base
    return _splitmix64(idx)


def normal_table(sigma: float, dtype: torch.dtype) -> torch.Tensor:
    """65536-entry inverse-CDF table of N(0, sigma^2), float64 on the host, rounded once to `dtype`."""
    key = (float(sigma), dtype)
    if key not in _tables:
        p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        _tables[key] = (torch.special.ndtri(p) * sigma).to(dtype)
    return _tables[key]


def normal(seed: int, stream: int, shape, sigma: float, dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """Tensor of `shape` with N(0, sigma^2) entries (table-quantised to 65536 levels)."""
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=dtype, device=device)
    table = normal_table(sigma, dtype).to(device)
    for start in range(0, n, _CHUNK):
        cnt = min(_CHUNK, n - start)
        u = _bits(seed, stream, start, cnt, device)
        out[start:start + cnt] = table[_lsr(u, 48)]
    return out.view(*shape)


def tokens(seed: int, stream: int, n: int, vocab: int, device="cpu") -> torch.Tensor:
    """`n` token ids uniform on [0, vocab), int32."""
    u = _lsr(_bits(seed, stream, 0, n, device), 32)
    return ((u * vocab) >> 32).to(torch.int32)


# ---------------------------------------------------------------------------------------------------------
# Model shapes (the public Qwen3 shapes the workloads use) and random-init weight sets.
# ---------------------------------------------------------------------------------------------------------

@dataclasses.dataclass(frozen=True)
class ModelShape:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    intermediate: int
    vocab: int
    tie_embeddings: bool
    rms_eps: float = 1e-6
    rope_theta: float = 1e6

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def weight_bytes_per_decode_step(self) -> int:
        """bf16 bytes of every matrix a decode step streams once (embedding row and gains excluded)."""
        per_layer = (self.q_dim + 2 * self.kv_dim) * self.hidden + self.hidden * self.q_dim \
            + 3 * self.intermediate * self.hidden
        return 2 * (self.n_layers * per_layer + self.vocab * self.hidden)

    def kv_bytes_per_position(self) -> int:
        return 2 * 2 * self.kv_dim * self.n_layers


SHAPES: Dict[str, ModelShape] = {
    # smallest shape the CUDA library accepts (head_dim is fixed at 128); used by fast tests
    "tiny": ModelShape(2, 256, 2, 1, 128, 512, 1024, True),
    "tiny-untied": ModelShape(3, 384, 4, 2, 128, 640, 1000, False),
    "qwen3-0.6b": ModelShape(28, 1024, 16, 8, 128, 3072, 151936, True),
    "qwen3-0.6b-1layer": ModelShape(1, 1024, 16, 8, 128, 3072, 151936, True),
    "qwen3-1.7b": ModelShape(28, 2048, 16, 8, 128, 6144, 151936, True),
    "qwen3-8b": ModelShape(36, 4096, 32, 8, 128, 12288, 151936, False),
}

# stream ids: fixed enumeration, layer-major
_PER_LAYER = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")
_S_EMBED, _S_LMHEAD, _S_TOKENS, _S_HIDDEN, _S_KV = 1, 2, 3, 4, 5
_S_LAYER0 = 16


def layer_weight_shapes(s: ModelShape) -> Dict[str, tuple]:
    return {
        "wq": (s.q_dim, s.hidden), "wk": (s.kv_dim, s.hidden), "wv": (s.kv_dim, s.hidden),
        "wo": (s.hidden, s.q_dim), "w_gate": (s.intermediate, s.hidden), "w_up": (s.intermediate, s.hidden),
        "w_down": (s.hidden, s.intermediate),
    }


def make_weights(s: ModelShape, seed: int, device="cpu", sigma: float = 0.02) -> dict:
    """Random-init weight set: bf16 matrices `[out][in]` ~ N(0, sigma^2); every norm gain exactly 1.0."""
    ones = lambda n: torch.ones(n, dtype=torch.bfloat16, device=device)
    w = {"embed": normal(seed, _S_EMBED, (s.vocab, s.hidden), sigma, torch.bfloat16, device),
         "lm_head": None if s.tie_embeddings else
         normal(seed, _S_LMHEAD, (s.vocab, s.hidden), sigma, torch.bfloat16, device),
         "g_final": ones(s.hidden), "layers": []}
    shapes = layer_weight_shapes(s)
    for l in range(s.n_layers):
        lw = {}
        for i, name in enumerate(_PER_LAYER):
            lw[name] = normal(seed, _S_LAYER0 + l * 8 + i, shapes[name], sigma, torch.bfloat16, device)
        lw["g_in"], lw["g_post"] = ones(s.hidden), ones(s.hidden)
        lw["g_q"], lw["g_k"] = ones(s.head_dim), ones(s.head_dim)
        w["layers"].append(lw)
    return w


def random_gains(w: dict, seed: int) -> None:
    """Replace the unit norm gains by bf16 values ~ 1 + N(0, 0.1^2) (tests only: makes gain bugs visible)."""
    k = 0
    def g(t):
        nonlocal k
        k += 1
        return (1.0 + normal(seed, 1000 + k, t.shape, 0.1, torch.float32, t.device)).to(torch.bfloat16)
    w["g_final"] = g(w["g_final"])
    for lw in w["layers"]:
        for name in ("g_in", "g_post", "g_q", "g_k"):
            lw[name] = g(lw[name])


def prompt_tokens(s: ModelShape, seed: int, n: int, device="cpu", batch_index: int = 0) -> torch.Tensor:
    return tokens(seed, 100000 + _S_TOKENS + batch_index, n, s.vocab, device)


def hidden_state(s: ModelShape, seed: int, device="cpu") -> torch.Tensor:
    """fp32 `[hidden]` ~ N(0,1): the input of the single-layer decode workload."""
    return normal(seed, _S_HIDDEN, (s.hidden,), 1.0, torch.float32, device)


def kv_fill(s: ModelShape, seed: int, layer: int, n_pos: int, device="cpu", batch_index: int = 0):
    """Raw cache contents for one layer of one sequence: (K, V), each bf16 `[n_kv_heads][n_pos][head_dim]`
    ~ N(0,1).  K is what the cache holds (already normalised and rotated), not a pre-norm projection."""
    base = _S_KV + 4096 * (batch_index + 1) + 2 * layer
    shape = (s.n_kv_heads, n_pos, s.head_dim)
    return (normal(seed, base, shape, 1.0, torch.bfloat16, device),
            normal(seed, base + 1, shape, 1.0, torch.bfloat16, device))
