"""The bounds-checked debugging build (libnnc_checked.so: the same sources compiled with -DNNC_BOUNDS_CHECK).

compute-sanitizer is not available where this library is developed, so the kernels carry their own checks in that
build: indices that rest on the host's capacity checks are compared with their extents at the point of use, a miss
is counted and the access skipped.  Here: the build compiles and exports the full ABI (CPU), and on a GPU a child
process drives tiny models, ragged GEMV / GEMM shapes, both attention kernels and the FP8 path through it -- zero
misses, results bit-identical to the normal library -- and then sees the counter report a planted, memory-free miss."""
import ctypes as C
import os
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def checked_lib():
    from paper_2512_21571_b200 import build
    build.build()
    return build.build(checked=True)


def test_checked_build_exports_the_same_abi(checked_lib):
    import re
    lib = C.CDLL(checked_lib)
    text = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "nnc.h")).read(), flags=re.S)
    for name in sorted(set(re.findall(r"\b(nnc_[a-z0-9_]+)\s*\(", text))):
        assert hasattr(lib, name), name


def test_normal_build_says_it_is_not_checked():
    from paper_2512_21571_b200 import binding
    assert binding.bounds_check_report() == (-1, 0)


_CHILD = textwrap.dedent("""
    import sys, torch
    sys.path.insert(0, {root!r}); sys.path.insert(0, {root!r} + "/tests")
    from paper_2512_21571_b200 import binding as nnc, synth
    out = {{}}
    for name, seed, fmt in (("tiny", 1, 0), ("tiny-untied", 2, 0), ("tiny", 3, 1)):
        shape = synth.SHAPES[name]
        w = synth.make_weights(shape, seed, device="cuda", sigma=0.05)
        m = nnc.Model(shape, w, max_seq=200, max_tokens=150, weight_format=fmt)
        toks = synth.prompt_tokens(shape, seed, 150).cuda()
        lg = m.prefill(toks.view(1, 150), all_positions=True)            # prompt-phase form (fp16 one-term GEMMs)
        m.set_length(0)
        l2 = m.prefill(toks[:19].contiguous().view(1, 19))                # few-token form
        logits = torch.empty(shape.vocab, device="cuda")
        am = torch.zeros(1, dtype=torch.int32, device="cuda")
        steps = []
        for i in range(5):
            m.decode_step(toks[20 + i:21 + i].contiguous(), logits, am)  # batch-1 GEMV path, captured graph
            steps.append(logits.clone())
        assert m.device_status() == 0
        out[name + str(fmt)] = [lg.cpu(), l2.cpu()] + [t.cpu() for t in steps]
    # ragged single operations
    for n_out, n_in in ((1000, 384), (2050, 640), (8, 64)):
        W = synth.normal(5, 1, (n_out, n_in), 0.02, torch.bfloat16, "cuda")
        x = synth.normal(5, 2, (n_in,), 1.0, torch.float32, "cuda")
        out["gemv%d" % n_out] = [nnc.op_gemv(W, x, mode=0).cpu()]
    for T, N, K in ((5, 40, 64), (33, 1000, 384), (130, 264, 192)):
        X = synth.normal(6, 1, (T, K), 1.0, torch.float32, "cuda").to(torch.bfloat16)
        W = synth.normal(6, 2, (N, K), 0.02, torch.bfloat16, "cuda")
        out["gemm%d" % T] = [nnc.op_gemm(X, W).cpu()]
    scratch = torch.zeros(16384 + 2 * 65536 * 148, dtype=torch.uint8, device="cuda")
    X = synth.normal(7, 1, (32, 4096), 1.0, torch.float32, "cuda").to(torch.bfloat16)
    W = synth.normal(7, 2, (1024, 4096), 0.02, torch.bfloat16, "cuda")
    out["splitk"] = [nnc.op_gemm_splitk(X, W, scratch).cpu()]
    q = synth.normal(8, 1, (2, 8, 128), 1.0, torch.float32, "cuda")
    kc = synth.normal(8, 2, (2, 2, 700, 128), 1.0, torch.bfloat16, "cuda")
    vc = synth.normal(8, 3, (2, 2, 700, 128), 1.0, torch.bfloat16, "cuda")
    out["attn"] = [nnc.op_attn_decode(q, kc, vc, 651).cpu()]
    assert nnc.op_status() == 0
    torch.cuda.synchronize()
    report = nnc.bounds_check_report()
    nnc.lib.nnc_bounds_check_selftest(777, None)
    planted = nnc.bounds_check_report()
    torch.save({{"out": out, "report": report, "planted": planted}}, sys.argv[1])
""")


@pytest.mark.gpu
def test_checked_build_runs_clean_and_matches_the_normal_build(checked_lib, tmp_path):
    import torch
    prog = tmp_path / "child.py"
    prog.write_text(_CHILD.format(root=ROOT))
    results = {}
    for tag, lib in (("normal", None), ("checked", checked_lib)):
        env = dict(os.environ)
        env.pop("NNC_LIBRARY", None)
        if lib:
            env["NNC_LIBRARY"] = lib
        res = tmp_path / (tag + ".pt")
        r = subprocess.run([sys.executable, str(prog), str(res)], capture_output=True, text=True, timeout=900, env=env)
        assert r.returncode == 0, r.stdout + r.stderr
        results[tag] = torch.load(res)
    assert results["normal"]["report"] == (-1, 0)
    assert results["checked"]["report"] == (0, 0), "the checked build counted out-of-range indices"
    assert results["checked"]["planted"] == (1, 777)
    for key, tensors in results["normal"]["out"].items():
        for a, b in zip(tensors, results["checked"]["out"][key]):
            assert torch.equal(a, b), key


def test_tracing_build_compiles(tmp_path):
    """-DNNC_TRACE adds per-CTA timeline records (nnc_trace_enable / nnc_trace_dump) used when tuning; it is not part of
    the product library, so all that is checked here is that the instrumented sources still compile."""
    from paper_2512_21571_b200 import build
    csrc = os.path.join(ROOT, "paper_2512_21571_b200", "csrc")
    for name in ("decode_misc.cu", "nnc_api.cu", "attn_prefill_f16.cu"):
        cmd = ["nvcc", *build.NVCC_FLAGS, "-DNNC_TRACE", "-DNNC_TUNING", "-c", os.path.join(csrc, name), "-o",
               str(tmp_path / (name + ".o"))]
        r = subprocess.run(cmd, capture_output=True, text=True)
        assert r.returncode == 0, r.stderr
