#!/usr/bin/env python
"""Throughput benchmark of the Qwen3 forward pass behind the nnc C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the hot path over one batch: a batch-1 decode step (the default workload, the
Qwen3-8B shape with the cache pre-filled to 4096 positions and 128-step decode passes), a batched decode
step, or one prompt-phase call.  Prints ONE JSON line (rank 0).  Inputs are seeded and synthetic.

  value      device-timed throughput, inputs resident in HBM (CUDA events on the launching stream)
  e2e        the same metric through the *_host entry points: host->device copy of the tokens and
             device->host copy of the logits inside the timed region, one synchronisation per step
  roofline   the dominant kernel timed alone over operands larger than L2, against the measured peak: launched
             back to back the way the step launches it (`frac`), and one launch at a time (`isolated_frac`)
  step_roofline  algorithmic bytes (or FLOPs) of a whole step over the step time
  prefill    (default workload only) the prompt-phase half of the metric: one call of 4 x 2048 tokens on the same
             model shape, tokens/s and model FLOPs over the measured bf16 tensor-core peak
  cpu_baseline   the CPU oracle, as it stands, on the host cores, on a bounded sample of the workload

With --gpus N > 1 (launched by torch.distributed.run) every rank runs an independent replica: the forward
pass of one sequence does not shard without collectives, so there is no data-path communication; time is the
max over ranks and value the sum of the replicas' work over it.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2512_21571_b200 import synth  # noqa: E402

L2_BYTES = 126 * 1024 * 1024

WORKLOADS = {
    # name: (shape, kind, context before the pass, steps per pass, batch)
    "qwen3-8b-decode-b1-ctx4096": dict(shape="qwen3-8b", kind="decode", ctx=4096, pass_steps=128, batch=1, seed=3),
    "qwen3-1.7b-decode-b1-ctx512": dict(shape="qwen3-1.7b", kind="decode", ctx=512, pass_steps=256, batch=1, seed=2),
    "qwen3-0.6b-decode-b1-ctx64": dict(shape="qwen3-0.6b", kind="decode", ctx=64, pass_steps=64, batch=1, seed=1),
    "qwen3-8b-decode-b1-ctx4096-fp8": dict(shape="qwen3-8b", kind="decode", ctx=4096, pass_steps=128, batch=1, seed=3,
                                           weight_format=1),
    "qwen3-8b-decode-b32-ctx8192": dict(shape="qwen3-8b", kind="decode", ctx=8192, pass_steps=16, batch=32, seed=4),
    "qwen3-8b-prefill-4x2048": dict(shape="qwen3-8b", kind="prefill", ctx=0, tokens=2048, batch=4, seed=4),
    "qwen3-1.7b-prefill-1x512": dict(shape="qwen3-1.7b", kind="prefill", ctx=0, tokens=512, batch=1, seed=2),
}
DEFAULT_WORKLOAD = "qwen3-8b-decode-b1-ctx4096"


def load_peaks():
    """Measured denominators (written by the harness that owns the machine); else the stated fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def measured_traffic(key: str):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of a kernel from the profiler capture
    recorded in profiles/dram_traffic.json -- or None when there is no capture for `key` or the kernel's source file
    has changed since the capture was taken (the record holds the file's SHA-1 at that time)."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            rec = json.load(f).get(key)
        if not rec:
            return None
        with open(os.path.join(ROOT, rec["source"]), "rb") as f:
            if hashlib.sha1(f.read()).hexdigest() != rec["source_sha1"]:
                return None
        return float(rec["bytes_per_launch"])
    except (OSError, ValueError, KeyError):
        return None


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, device_index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = torch.cuda.get_device_properties(device_index).uuid
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(f"GPU-{uuid}")
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(f"GPU-{uuid}".encode())
            self._reasons_fn = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                pynvml.nvmlDeviceGetCurrentClocksThrottleReasons
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # no NVML: report that rather than invent numbers
            self.nv, self.err = None, repr(e)

    _NAMES = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
              0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x100: "display_clocks_setting",
              0x10: "sync_boost"}

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = self._reasons_fn(self.h)
                for bit, name in self._NAMES.items():
                    if r & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.nv:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "error": self.err}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s), "power_w_max": max(self.power) if self.power else None}


def dist_setup(n_gpus: int):
    """(rank, world).  One process per GPU; rendezvous from the torchrun environment."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    if world != n_gpus and rank == 0:
        print(f"bench.py: --gpus {n_gpus} but WORLD_SIZE={world}; using WORLD_SIZE", file=sys.stderr)
    return rank, world


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


def max_over_ranks(ms: float, world: int) -> float:
    """Device time of the slowest rank (every rank returns the same number)."""
    if world == 1:
        return ms
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(ms_local: float, steps: int, units_per_step: int, world: int):
    """(ms of the slowest rank, units/s of all replicas together): every rank did `steps * units_per_step` units."""
    ms = max_over_ranks(ms_local, world)
    return ms, world * steps * units_per_step / (ms * 1e-3)


def build_model(wl, max_tokens=None, w=None):
    from paper_2512_21571_b200 import binding
    shape = synth.SHAPES[wl["shape"]]
    seed = wl["seed"]
    if w is None:
        w = synth.make_weights(shape, seed, device="cuda")
    if wl["kind"] == "decode":
        max_seq = wl["ctx"] + wl["pass_steps"]
        mt = max(wl["batch"], 1)
    else:
        max_seq = wl["tokens"]
        mt = wl["batch"] * wl["tokens"]
    m = binding.Model(shape, w, max_seq=max_seq, max_batch=wl["batch"], max_tokens=max_tokens or mt,
                      weight_format=wl.get("weight_format", 0))
    if wl["ctx"]:
        for b in range(wl["batch"]):
            for l in range(shape.n_layers):
                k, v = synth.kv_fill(shape, seed + 1000, l, wl["ctx"], device="cuda", batch_index=b)
                m.kv_import(l, b, k, v)
        m.set_length(wl["ctx"])
    torch.cuda.synchronize()
    return m, shape, w


def decode_bytes_per_step(shape, batch, ctx_mid, weight_format=0):
    wbytes = shape.weight_bytes_per_decode_step()
    if weight_format == 1:   # FP8 codes: one byte per weight plus one fp32 scale per output row
        rows = shape.n_layers * (shape.q_dim + 2 * shape.kv_dim + shape.hidden + 2 * shape.intermediate + shape.hidden) + shape.vocab
        wbytes = wbytes // 2 + 4 * rows
    return wbytes + batch * ctx_mid * shape.kv_bytes_per_position()


def prefill_flops(shape, batch, T):
    per_layer = (shape.q_dim + 2 * shape.kv_dim) * shape.hidden + shape.hidden * shape.q_dim \
        + 3 * shape.intermediate * shape.hidden
    proj = 2.0 * batch * T * shape.n_layers * per_layer
    attn = 2.0 * 2.0 * batch * shape.n_layers * shape.n_q_heads * shape.head_dim * (T * (T + 1) / 2)
    head = 2.0 * batch * shape.vocab * shape.hidden  # last position only
    return proj, attn, head


def prefill_roofline(shape, wl, ms_per_call, peaks):
    """Model FLOPs of one prompt-phase call over its time, against the measured bf16 tensor-core peaks; `issued` adds
    the second bf16 term of the operands that are fed as value + residual (QKV input, Q and P inside attention)."""
    proj, attn, head = prefill_flops(shape, wl["batch"], wl["tokens"])
    total = proj + attn + head
    qkv = 2.0 * wl["batch"] * wl["tokens"] * shape.n_layers * (shape.q_dim + 2 * shape.kv_dim) * shape.hidden
    issued = total + qkv + attn
    ach = total / (ms_per_call * 1e-3) / 1e12
    return {"bound": "tensor", "flops_per_step": total, "projection_flops": proj, "attention_flops": attn,
            "achieved": round(ach, 1), "unit": "TFLOP/s (model FLOPs)",
            "peak": peaks["bf16_tflops"], "frac": round(ach / peaks["bf16_tflops"], 4), "peak_source": peaks["source"] + " (burst)",
            "frac_of_sustained": round(ach / peaks["bf16_tflops_sustained"], 4), "frac_of_nominal_2250": round(ach / 2250.0, 4),
            "issued_tflops": round(issued / (ms_per_call * 1e-3) / 1e12, 1)}


def time_decode(m, shape, wl, steps, warmup, world):
    B = wl["batch"]
    toks = torch.stack([synth.tokens(wl["seed"] + 2000, b, steps + warmup, shape.vocab) for b in range(B)], 1).cuda()
    logits = torch.empty(B, shape.vocab, device="cuda")
    am = torch.zeros(1, dtype=torch.int32, device="cuda") if B == 1 else None
    tok = torch.zeros(B, dtype=torch.int32, device="cuda")

    def run(n, first):
        for i in range(n):
            if (i % wl["pass_steps"]) == 0:
                m.set_length(wl["ctx"])
            tok.copy_(toks[first + i])
            m.decode_step(tok, logits, am)

    run(warmup, 0)
    barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = m.launch_count
    sampler = ClockSampler(torch.cuda.current_device())
    with sampler:
        e0.record()
        run(steps, warmup)
        e1.record()
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    launches = m.launch_count - n0 + steps  # + the token copy of each step
    barrier(world)
    return ms, launches, sampler.summary()


def time_decode_e2e(m, shape, wl, steps, warmup, world):
    B = wl["batch"]
    toks = torch.stack([synth.tokens(wl["seed"] + 2000, b, steps + warmup, shape.vocab) for b in range(B)], 1)
    tok_h = torch.zeros(B, dtype=torch.int32).pin_memory()
    logits_h = torch.empty(B, shape.vocab, dtype=torch.float32).pin_memory()
    am_h = torch.zeros(1, dtype=torch.int32).pin_memory() if B == 1 else None

    def run(n, first):
        for i in range(n):
            if (i % wl["pass_steps"]) == 0:
                m.set_length(wl["ctx"])
            tok_h.copy_(toks[first + i])
            m.decode_step_host(tok_h, logits_h, am_h)

    run(min(warmup, 3), 0)
    barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    run(steps, warmup)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    barrier(world)
    h2d = tok_h.numel() * 4
    d2h = logits_h.numel() * 4 + (4 if am_h is not None else 0)
    return ms, h2d, d2h


def time_prefill(m, shape, wl, steps, warmup, world, host=False):
    B, T = wl["batch"], wl["tokens"]
    toks = torch.stack([synth.prompt_tokens(shape, wl["seed"] + 1000, T, batch_index=b) for b in range(B)])
    logits = torch.empty(B, shape.vocab, device="cuda")
    if host:
        toks_h = toks.contiguous().pin_memory()
        logits_h = torch.empty(B, shape.vocab).pin_memory()
        call = lambda: m.prefill_host(toks_h, logits_h)
    else:
        toks_d = toks.cuda().contiguous()
        call = lambda: m.prefill(toks_d, logits)
    for _ in range(warmup):
        m.set_length(0)
        call()
    barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = m.launch_count
    sampler = ClockSampler(torch.cuda.current_device())
    with sampler:
        e0.record()
        for _ in range(steps):
            m.set_length(0)
            call()
        e1.record()
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    barrier(world)
    return ms, m.launch_count - n0, sampler.summary(), B * T * 4, B * shape.vocab * 4


def kernel_roofline_gemv(shape, peaks, w, fp8=False):
    """The dominant decode kernel -- the fused RMSNorm + gate/up GEMV + SwiGLU -- timed alone with CUDA events
    over every layer's own matrix in turn (each larger than L2, so nothing is re-read from cache)."""
    from paper_2512_21571_b200 import binding
    H, I = shape.hidden, shape.intermediate
    n_mats = min(shape.n_layers, 12)
    mats = []
    for l in range(n_mats):
        if w is None:   # --kernel-only: no model was built; any seeded matrix of the shape will do
            mats.append(synth.normal(9, 100 + l, (2 * I, H), 0.02, torch.bfloat16, "cuda"))
            continue
        lw = w["layers"][l]
        wgu = torch.empty(2 * I, H, dtype=torch.bfloat16, device="cuda")
        wgu[0::2] = lw["w_gate"]
        wgu[1::2] = lw["w_up"]
        mats.append(wgu)
    if fp8:   # the same matrices as E4M3 codes + row scales
        q = [binding.op_quantise_rows_e4m3(W, want_dequant=False)[:2] for W in mats]
        mats = None
        run = lambda i, chained: binding.op_gemv_fp8(q[i][0], q[i][1], x, mode=2, gain=gain, y=y, chained=chained)
        n_mats = len(q)
    else:
        run = lambda i, chained: binding.op_gemv(mats[i], x, mode=2, gain=gain, y=y, chained=chained)
    x = synth.normal(9, 1, (H,), 1.0, torch.float32, "cuda")
    gain = torch.ones(H, dtype=torch.bfloat16, device="cuda")
    y = torch.empty(I, dtype=torch.float32, device="cuda")
    wb = 1 if fp8 else 2
    reps = 3 if 2 * I * H * wb * n_mats > 4 * L2_BYTES else 1
    for i in range(min(3, n_mats)):
        run(i, True)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = 0
    e0.record()
    for _ in range(reps):
        for i in range(n_mats):
            run(i, True)   # launched as inside the decode graph
            n += 1
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / n
    # one launch at a time: plain stream order, an event pair around every launch, so no launch hides its start-up
    # under its predecessor's tail
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_mats)]
    for i, (a, b) in enumerate(pairs):
        a.record()
        run(i, False)
        b.record()
    torch.cuda.synchronize()
    iso = sorted(a.elapsed_time(b) * 1e3 for a, b in pairs)
    us_iso = iso[len(iso) // 2]
    nbytes = 2 * I * H * wb + (4 * 2 * I if fp8 else 0)
    ach = nbytes / (us * 1e-6) / 1e9
    ach_iso = nbytes / (us_iso * 1e-6) / 1e9
    return {"bound": "hbm", "kernel": "gemv_stream_kernel<SwiGLU, norm prologue%s>" % (", FP8 codes" if fp8 else ""), "shape": [2 * I, H],
            "achieved": round(ach, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(ach / peaks["hbm_gbs"], 4),
            "peak_source": peaks["source"], "bytes_per_launch": nbytes, "us_per_launch": round(us, 2),
            "launches_timed": n, "how": "back-to-back launches with programmatic stream serialization, as in the decode graph",
            "isolated_us_per_launch": round(us_iso, 2), "isolated_achieved": round(ach_iso, 1),
            "isolated_frac": round(ach_iso / peaks["hbm_gbs"], 4),
            "traffic": measured_traffic("gemv_stream_kernel<SwiGLU%s>:%dx%d" % (",fp8" if fp8 else "", 2 * I, H))}


def kernel_roofline_gemm(shape, peaks, T):
    """The dominant prompt-phase kernel -- the tcgen05 GEMM on the gate/up shape with the SwiGLU epilogue -- timed
    alone in the form the prompt phase uses (one fp16 term, scaled fp16 weight copy).  `achieved` counts MODEL FLOPs,
    2 * T * 2I * H per launch; the two-bf16-term form of the same product is reported beside it."""
    from paper_2512_21571_b200 import binding
    H, I = shape.hidden, shape.intermediate
    X = synth.normal(9, 1, (T, H), 1.0, torch.bfloat16, "cuda")
    X_lo = synth.normal(9, 2, (T, H), 0.004, torch.bfloat16, "cuda")
    W = synth.normal(9, 3, (2 * I, H), 0.02, torch.bfloat16, "cuda")
    X16 = X.to(torch.float16)
    W16, scales = binding.op_to_f16_scaled(W)
    model_flops = 2.0 * T * 2 * I * H
    runs = {"f16": lambda: binding.op_gemm_swiglu_f16(X16, W16, out_scale=scales[1:]),
            "bf16_two_terms": lambda: binding.op_gemm_swiglu(X, W, X_lo=X_lo)}
    if T <= 128:
        runs.pop("f16")
    out = {}
    for name, fn in runs.items():
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 10
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        out[name] = e0.elapsed_time(e1) * 1e3 / n
    assert binding.op_status() == 0
    head = "f16" if "f16" in out else "bf16_two_terms"
    us = out[head]
    ach = model_flops / (us * 1e-6) / 1e12
    res = {"bound": "tensor", "kernel": "gemm_tc_kernel<SwiGLU, %s>" % ("one fp16 term" if head == "f16" else "two bf16 terms"),
           "shape": [T, 2 * I, H], "achieved": round(ach, 1), "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
           "frac": round(ach / peaks["bf16_tflops"], 4), "peak_source": peaks["source"] + " (burst; fp16 and bf16 share the rate)",
           "frac_of_sustained": round(ach / peaks["bf16_tflops_sustained"], 4),
           "flops_per_launch": model_flops, "us_per_launch": round(us, 1), "launches_timed": 10,
           "traffic": measured_traffic("gemm_tc_kernel<SwiGLU,f16>:%dx%dx%d" % (T, 2 * I, H)) if head == "f16" else None}
    if "bf16_two_terms" in out and head == "f16":
        us2 = out["bf16_two_terms"]
        res["bf16_two_terms"] = {"us_per_launch": round(us2, 1), "model_tflops": round(model_flops / (us2 * 1e-6) / 1e12, 1),
                                 "issued_tflops": round(2 * model_flops / (us2 * 1e-6) / 1e12, 1)}
    return res


def kernel_roofline_attn(shape, peaks, batch, ctx):
    """The dominant kernel of batched decode at long context -- the split-range flash-decode -- timed alone on a
    cache of the workload's size (larger than L2); algorithmic bytes = the K and V rows it has to read once."""
    from paper_2512_21571_b200 import binding
    nq, nkv = shape.n_q_heads, shape.n_kv_heads
    max_seq = ctx + 64
    kc = synth.normal(9, 11, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    vc = synth.normal(9, 12, (batch, nkv, max_seq, 128), 1.0, torch.bfloat16, "cuda")
    q = synth.normal(9, 13, (batch, nq, 128), 1.0, torch.float32, "cuda")
    scratch = torch.empty(binding.lib.nnc_attn_scratch_bytes(batch, nq, ctx), dtype=torch.uint8, device="cuda")
    scratch.zero_()
    for _ in range(3):
        binding.op_attn_decode(q, kc, vc, ctx, scratch)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = 10
    e0.record()
    for _ in range(n):
        binding.op_attn_decode(q, kc, vc, ctx, scratch)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / n
    nbytes = 2.0 * batch * nkv * ctx * 128 * 2
    ach = nbytes / (us * 1e-6) / 1e9
    return {"bound": "hbm", "kernel": "attn_decode_kernel<G=%d>" % (nq // nkv), "shape": [batch, nkv, ctx, 128],
            "achieved": round(ach, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(ach / peaks["hbm_gbs"], 4),
            "peak_source": peaks["source"], "bytes_per_launch": int(nbytes), "us_per_launch": round(us, 2),
            "launches_timed": n, "traffic": measured_traffic("attn_decode_kernel<G=%d>:b%d_ctx%d" % (nq // nkv, batch, ctx))}


def kernel_roofline_attn_prefill(shape, peaks, batch, T):
    """The prompt-phase attention kernel timed alone: causal attention of `batch` sequences of T new tokens (no past),
    in the one-fp16-term form the prompt phase uses and, beside it, the two-bf16-term form.  Model FLOPs =
    4 * 128 * T (T + 1) / 2 per head."""
    from paper_2512_21571_b200 import binding
    nq, nkv = shape.n_q_heads, shape.n_kv_heads
    qkv = synth.normal(9, 21, (batch * T, (nq + 2 * nkv) * 128), 1.0, torch.float32, "cuda")
    kc = synth.normal(9, 22, (batch, nkv, T, 128), 1.0, torch.bfloat16, "cuda")
    vc = synth.normal(9, 23, (batch, nkv, T, 128), 1.0, torch.bfloat16, "cuda")
    k16, v16 = kc.to(torch.float16), vc.to(torch.float16)
    runs = {"f16": lambda: binding.op_attn_prefill_f16(qkv, k16, v16, T, nq, 0),
            "bf16_two_terms": lambda: binding.op_attn_prefill(qkv, kc, vc, T, nq, 0)}
    us = {}
    n = 10
    for name, fn in runs.items():
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        us[name] = e0.elapsed_time(e1) * 1e3 / n
    assert binding.op_status() == 0
    flops = 4.0 * 128 * batch * nq * (T * (T + 1) / 2)
    ach = flops / (us["f16"] * 1e-6) / 1e12
    return {"bound": "tensor", "kernel": "attn_prefill_f16_kernel (one fp16 term; beside it attn_prefill_tc_kernel, two bf16 terms)", "shape": [batch, nq, T, 128],
            "achieved": round(ach, 1), "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": round(ach / peaks["bf16_tflops"], 4),
            "peak_source": peaks["source"] + " (burst)", "flops_per_launch": flops,
            "us_per_launch": round(us["f16"], 1), "launches_timed": n,
            "bf16_two_terms": {"us_per_launch": round(us["bf16_two_terms"], 1),
                               "model_tflops": round(flops / (us["bf16_two_terms"] * 1e-6) / 1e12, 1)},
            "traffic": measured_traffic("attn_prefill_f16_kernel:b%d_T%d" % (batch, T))}


# ---- the CPU oracle leg (reported baseline; the only place the product's bench touches oracle/) ------------

def oracle_leg(wl, shape, w_gpu, steps, warmup, budget_s=25.0):
    """Times the CPU oracle on a bounded sample of the workload.  Returns (unit value, description dict)."""
    import oracle
    oracle.build()
    import psutil
    cores = len(os.sched_getaffinity(0))
    torch.set_num_threads(cores)
    need = shape.weight_bytes_per_decode_step() * (1 if shape.tie_embeddings else 1) + (2 << 30)
    avail = psutil.virtual_memory().available
    n_layers = shape.n_layers
    if need * 1.3 > avail:  # not enough host memory for the whole model: sample layers
        n_layers = max(1, int(shape.n_layers * avail / (need * 1.5)))
    import dataclasses
    sub = dataclasses.replace(shape, n_layers=n_layers)
    c = lambda t: None if t is None else t.cpu().contiguous()
    wc = {"embed": c(w_gpu["embed"]), "lm_head": c(w_gpu.get("lm_head")), "g_final": c(w_gpu["g_final"]),
          "layers": [{k: c(v) for k, v in lw.items()} for lw in w_gpu["layers"][:n_layers]]}
    if wl["kind"] == "decode":
        o = oracle.Oracle(sub, wc, max_seq=wl["ctx"] + steps + warmup + 2)
        for l in range(n_layers):
            k, v = synth.kv_fill(shape, wl["seed"] + 1000, l, wl["ctx"], device=w_gpu["embed"].device)
            o.kv_import(l, k.cpu(), v.cpu())
        toks = synth.tokens(wl["seed"] + 2000, 0, steps + warmup, shape.vocab)
        for i in range(warmup):
            o.forward(toks[i:i + 1])
        t0 = time.perf_counter()
        done = 0
        for i in range(steps):
            o.forward(toks[warmup + i:warmup + i + 1])
            done += 1
            if time.perf_counter() - t0 > budget_s:
                break
        dt = time.perf_counter() - t0
        frac = sub.weight_bytes_per_decode_step() / shape.weight_bytes_per_decode_step()
        per_step = dt / done / frac if n_layers < shape.n_layers else dt / done
        sample = f"{done} batch-1 decode steps of one sequence at context {wl['ctx']}"
        if n_layers < shape.n_layers:
            sample += f", first {n_layers} of {shape.n_layers} layers + lm_head, time scaled by weight bytes"
        if wl["batch"] > 1:
            sample += f"; one of the {wl['batch']} sequences (tokens/s of a single sequence)"
        o.close()
        return 1.0 / per_step, {"cores": cores, "kind": "oracle", "sample": sample}
    # prompt phase: a short prefix of one sequence; FLOPs scale the time to the full call
    Ts = 64
    o = oracle.Oracle(sub, wc, max_seq=Ts + 1)
    toks = synth.prompt_tokens(shape, wl["seed"] + 1000, Ts)
    t0 = time.perf_counter()
    o.forward(toks)
    dt = time.perf_counter() - t0
    o.close()
    frac = sub.n_layers / shape.n_layers
    sample = f"one {Ts}-token prompt prefix of one sequence"
    if n_layers < shape.n_layers:
        sample += f", first {n_layers} of {shape.n_layers} layers (time scaled by layer count)"
    return Ts / (dt / frac), {"cores": cores, "kind": "oracle", "sample": sample}


def run_reference(args, wl, rank, world):
    """--impl reference: the CPU oracle as it stands, on the host cores, same metric / unit / config."""
    if rank != 0:
        return
    shape = synth.SHAPES[wl["shape"]]
    if torch.cuda.is_available():
        torch.cuda.set_device(0)
        w = synth.make_weights(shape, wl["seed"], device="cuda")
    else:
        w = synth.make_weights(shape, wl["seed"], device="cpu")
    t0 = time.perf_counter()
    steps = args.steps
    value, desc = oracle_leg(wl, shape, w, steps, min(args.warmup, 1), budget_s=150.0)
    unit = "tokens/s"
    line = {"impl": "reference", "metric": metric_name(wl), "value": round(value, 4), "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(1e3 / value * (wl["batch"] * wl.get("tokens", 1) if wl["kind"] == "prefill" else 1), 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_of(wl), "cpu_baseline": dict(desc, value=round(value, 4), unit=unit),
            "e2e": {"value": round(value, 4), "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": round(time.perf_counter() - t0, 1)}
    print(json.dumps(line), flush=True)


def metric_name(wl):
    if wl["kind"] == "decode":
        return f"Qwen3 decode tok/s @bs{wl['batch']}"
    return "Qwen3 prefill tok/s"


def config_of(wl):
    c = {"workload": None, "model_shape": wl["shape"], "batch": wl["batch"], "l2": "inputs larger than L2 (weights streamed once per step)",
         "weights": "random init N(0, 0.02^2) bf16" + (", quantised at create time to FP8 E4M3 codes with a power-of-two "
                    "scale per output row" if wl.get("weight_format", 0) == 1 else ""), "tokens": "uniform random ids"}
    for k, v in WORKLOADS.items():
        if v is wl:
            c["workload"] = k
    if wl["kind"] == "decode":
        c["context"] = f"{wl['ctx']} growing to {wl['ctx'] + wl['pass_steps']}, then reset (passes of {wl['pass_steps']} steps)"
    else:
        c["tokens_per_sequence"] = wl["tokens"]
    return c


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the isolated-kernel and prompt-phase extras")
    ap.add_argument("--kernel-only", action="store_true",
                    help="time only the dominant kernel of the workload on ~2.4 GB of operands (small enough for a "
                         "multi-pass profiler capture) and print its roofline object")
    ap.add_argument("--kernel", default="dominant", choices=["dominant", "attention"],
                    help="with --kernel-only on a prompt-phase workload: the GEMM (dominant) or the attention kernel")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]
    if args.steps is None:
        args.steps = 128 if wl["kind"] == "decode" and wl["batch"] == 1 else (16 if wl["kind"] == "decode" else 3)
    if args.warmup is None:
        args.warmup = 8 if wl["kind"] == "decode" else 3
    args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        run_reference(args, wl, rank, int(os.environ.get("WORLD_SIZE", "1")))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    rank, world = dist_setup(args.gpus)
    peaks = load_peaks()
    if args.kernel_only:
        shape = synth.SHAPES[wl["shape"]]
        if wl["kind"] == "decode" and wl["batch"] == 1:
            roof = kernel_roofline_gemv(shape, peaks, None, fp8=wl.get("weight_format", 0) == 1)
        elif wl["kind"] == "decode":
            roof = kernel_roofline_attn(shape, peaks, wl["batch"], wl["ctx"])
        elif args.kernel == "attention":
            roof = kernel_roofline_attn_prefill(shape, peaks, 1, wl["tokens"])
        else:
            roof = kernel_roofline_gemm(shape, peaks, max(wl["batch"] * wl.get("tokens", 1), 32))
        print(json.dumps({"kernel_only": True, "config": config_of(wl), "roofline": roof}), flush=True)
        return
    m, shape, w = build_model(wl)
    steps, warmup = args.steps, args.warmup

    if wl["kind"] == "decode":
        ms, launches, clocks = time_decode(m, shape, wl, steps, warmup, world)
        units_per_step = wl["batch"]
        ms, value = whole_job_throughput(ms, steps, units_per_step, world)
        ms_e, h2d, d2h = time_decode_e2e(m, shape, wl, steps, warmup, world)
        ms_e, e2e_value = whole_job_throughput(ms_e, steps, units_per_step, world)
        ctx_mid = wl["ctx"] + min(steps, wl["pass_steps"]) / 2.0
        nbytes = decode_bytes_per_step(shape, wl["batch"], ctx_mid, wl.get("weight_format", 0))
        ach = nbytes / (ms / steps * 1e-3) / 1e9
        step_roof = {"bound": "hbm", "bytes_per_step": int(nbytes), "achieved": round(ach, 1), "unit": "GB/s",
                     "peak": peaks["hbm_gbs"], "frac": round(ach / peaks["hbm_gbs"], 4), "peak_source": peaks["source"],
                     "frac_of_nominal_8000": round(ach / 8000.0, 4)}
    else:
        ms, launches, clocks, h2d, d2h = time_prefill(m, shape, wl, steps, warmup, world)
        units_per_step = wl["batch"] * wl["tokens"]
        ms, value = whole_job_throughput(ms, steps, units_per_step, world)
        ms_e, _, _, h2d, d2h = time_prefill(m, shape, wl, steps, 1, world, host=True)
        ms_e, e2e_value = whole_job_throughput(ms_e, steps, units_per_step, world)
        step_roof = prefill_roofline(shape, wl, ms / steps, peaks)

    line = {"metric": metric_name(wl), "value": round(value, 2), "unit": "tokens/s", "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": round(ms / steps, 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16",
            "dtype_detail": "bf16 weights and KV cache, fp32 residual stream and accumulation; tensor-core operands: two bf16 "
                            "terms, or one fp16 term with exact fp16 weight copies (prompt phase: O, gate/up, down)",
            "data": "synthetic",
            "config": config_of(wl), "clocks": clocks,
            "e2e": {"value": round(e2e_value, 2), "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": round(ms_e / steps, 4)},
            "gpu_launches": int(launches), "step_roofline": step_roof,
            "replicas": "independent replicas, no data-path collective" if world > 1 else None}

    if rank == 0 and not args.no_extras:
        if wl["kind"] == "decode" and wl["batch"] == 1:
            line["roofline"] = kernel_roofline_gemv(shape, peaks, w, fp8=wl.get("weight_format", 0) == 1)
        elif wl["kind"] == "decode":
            line["roofline"] = kernel_roofline_attn(shape, peaks, wl["batch"], wl["ctx"])
        else:
            T = wl["batch"] * wl.get("tokens", 1)
            line["roofline"] = kernel_roofline_gemm(shape, peaks, max(T, 32))
    m.close()
    del m
    if wl is WORKLOADS[DEFAULT_WORKLOAD] and not args.no_extras:
        # the prompt-phase half of the metric, same model shape and weights: one call of 4 x 2048 tokens
        pwl = WORKLOADS["qwen3-8b-prefill-4x2048"]
        torch.cuda.empty_cache()
        pm, _, _ = build_model(pwl, w=w)
        p_steps = 3
        pms, p_launches, p_clocks, _, _ = time_prefill(pm, shape, pwl, p_steps, 3, world)
        pms, p_value = whole_job_throughput(pms, p_steps, pwl["batch"] * pwl["tokens"], world)
        pms_e, _, _, ph2d, pd2h = time_prefill(pm, shape, pwl, p_steps, 1, world, host=True)
        pms_e, p_e2e = whole_job_throughput(pms_e, p_steps, pwl["batch"] * pwl["tokens"], world)
        pm.close()
        del pm
        line["prefill"] = {"metric": metric_name(pwl), "value": round(p_value, 1), "unit": "tokens/s", "steps": p_steps, "warmup": 3,
                           "ms_per_step": round(pms / p_steps, 3), "config": config_of(pwl), "clocks": p_clocks,
                           "e2e": {"value": round(p_e2e, 1), "unit": "tokens/s", "h2d_bytes_per_step": ph2d,
                                   "d2h_bytes_per_step": pd2h},
                           "gpu_launches": int(p_launches), "step_roofline": prefill_roofline(shape, pwl, pms / p_steps, peaks)}
        if rank == 0:
            line["prefill"]["roofline"] = kernel_roofline_gemm(shape, peaks, pwl["batch"] * pwl["tokens"])
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, desc = oracle_leg(wl, shape, w, 12, 1)
        line["cpu_baseline"] = dict(desc, value=round(v, 4), unit="tokens/s")
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
