"""Helpers for the GPU parity tests: build the CUDA model and the oracle from the same seeded weights."""
import torch

from paper_2512_21571_b200 import synth


def to_cpu(w: dict) -> dict:
    c = lambda t: None if t is None else t.cpu().contiguous()
    return {"embed": c(w["embed"]), "lm_head": c(w.get("lm_head")), "g_final": c(w["g_final"]),
            "layers": [{k: c(v) for k, v in lw.items()} for lw in w["layers"]]}


def make_pair(oracle_mod, shape, seed, max_seq, max_batch=1, max_tokens=None, gains=False, sigma=0.02):
    """(cuda model, oracle, gpu weights).  Weights are generated once on the GPU and copied to the host."""
    from paper_2512_21571_b200 import binding
    w = synth.make_weights(shape, seed, device="cuda", sigma=sigma)
    if gains:
        synth.random_gains(w, seed + 1)
    m = binding.Model(shape, w, max_seq=max_seq, max_batch=max_batch, max_tokens=max_tokens)
    o = oracle_mod.Oracle(shape, to_cpu(w), max_seq=max_seq)
    return m, o, w


def rel_l2(a: torch.Tensor, b: torch.Tensor) -> float:
    """max over rows of ||a - b|| / ||b|| (b = oracle)."""
    a, b = a.double().cpu(), b.double().cpu()
    a, b = a.reshape(-1, a.shape[-1]), b.reshape(-1, b.shape[-1])
    return ((a - b).norm(dim=-1) / b.norm(dim=-1)).max().item()


def split_bf16(x: torch.Tensor):
    """fp32 -> (hi, lo) bf16 pair with hi + lo ~ x to 16 mantissa bits: test input for the two-term GEMM operand."""
    hi = x.to(torch.bfloat16)
    return hi, (x - hi.float()).to(torch.bfloat16)


def fp8_dequantised(oracle_mod, wc: dict, tied: bool) -> dict:
    """The weight set of the FP8 weight format as the oracle sees it: every multiplied matrix replaced by
    dequantise(quantise(W)) under the oracle's own row rule (CPU tensors in, CPU tensors out).  A tied embedding is the
    lm_head, so it is replaced too; an untied embedding table is only gathered from and stays as it is."""
    dq = lambda W: oracle_mod.dequantise_rows_e4m3(*oracle_mod.quantise_rows_e4m3(W.contiguous()))
    out = {"embed": dq(wc["embed"]) if tied else wc["embed"],
           "lm_head": None if wc.get("lm_head") is None else dq(wc["lm_head"]), "g_final": wc["g_final"], "layers": []}
    for lw in wc["layers"]:
        out["layers"].append({k: (dq(v) if k.startswith("w") else v) for k, v in lw.items()})
    return out
