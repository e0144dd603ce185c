"""Pins of the oracle's second weight precision (FP8 E4M3 codes, one power-of-two scale per output row).

The E4M3 grid is a published format, so the pins are its table values written out by hand, exhaustive
decode/encode identity over all 254 finite codes, round-to-nearest-even at hand-picked ties, saturation, torch's own
float8_e4m3fn cast on in-range values (a library routine that never touches the oracle's code), and, for the row
rule, the exponent definition, error bounds that follow from the grid, and exactness of the dequantised values."""
import math

import numpy as np
import pytest
import torch


def test_e4m3_table_values(oracle_mod):
    d = oracle_mod.e4m3_to_f32
    assert d(0x00) == 0.0 and math.copysign(1.0, d(0x80)) == -1.0 and d(0x80) == 0.0
    assert d(0x01) == 2.0 ** -9 and d(0x07) == 7 * 2.0 ** -9          # subnormals: m * 2^-9
    assert d(0x08) == 2.0 ** -6                                       # smallest normal
    assert d(0x38) == 1.0 and d(0x39) == 1.125 and d(0x3C) == 1.5 and d(0xBC) == -1.5
    assert d(0x40) == 2.0 and d(0x77) == 240.0 and d(0x78) == 256.0
    assert d(0x7E) == 448.0 and d(0xFE) == -448.0                     # largest finite value
    assert math.isnan(d(0x7F)) and math.isnan(d(0xFF))                # no infinities in this format


def test_e4m3_decode_then_encode_is_the_identity_and_the_grid_is_monotone(oracle_mod):
    prev = None
    for c in range(0x7F):
        v = oracle_mod.e4m3_to_f32(c)
        assert oracle_mod.f32_to_e4m3(v) == c
        assert oracle_mod.f32_to_e4m3(-v) == (c | 0x80)
        if prev is not None:
            assert v > prev
        prev = v


def test_e4m3_rounding_is_nearest_even_and_saturates(oracle_mod):
    e = oracle_mod.f32_to_e4m3
    assert e(1.0625) == 0x38            # tie between 1.0 (even mantissa) and 1.125
    assert e(1.1875) == 0x3A            # tie between 1.125 (odd) and 1.25 (even)
    assert e(1.0626) == 0x39 and e(1.0624) == 0x38
    assert e(2.0 ** -10) == 0x00        # tie between 0 and the smallest subnormal
    assert e(1.5 * 2.0 ** -10) == 0x01 and e(3 * 2.0 ** -10) == 0x02   # 1.5 steps: tie between 1 and 2 -> 2
    assert e(7.5 * 2.0 ** -9) == 0x08   # tie between the largest subnormal (7, odd) and the smallest normal (8)
    assert e(1.9999) == 0x40            # rounding up carries into the next binade
    assert e(464.0) == 0x7E and e(449.0) == 0x7E and e(1e9) == 0x7E and e(float("inf")) == 0x7E
    assert e(-1e9) == 0xFE
    assert e(float("nan")) & 0x7F == 0x7F


def test_e4m3_encode_matches_torch_float8_cast_in_range(oracle_mod):
    g = torch.Generator().manual_seed(5)
    x = torch.cat([(torch.rand(20000, generator=g) * 2 - 1) * 448,
                   (torch.rand(20000, generator=g) * 2 - 1) * 0.05,
                   torch.randn(20000, generator=g)])
    want = x.to(torch.float8_e4m3fn).view(torch.uint8)
    got = torch.tensor([oracle_mod.f32_to_e4m3(float(v)) for v in x], dtype=torch.uint8)
    nz = x.to(torch.float8_e4m3fn).float() != 0        # the sign of a zero result is not compared
    assert torch.equal(got[nz], want[nz])
    assert torch.equal(got[~nz] & 0x7F, want[~nz] & 0x7F)


def test_row_exponent_is_the_smallest_that_fits(oracle_mod):
    rows = torch.tensor([[448.0, 1.0, 0.0, -3.0],       # fits exactly: e = 0
                         [450.0, 1.0, 0.0, -3.0],       # just above: e = 1
                         [-0.0859375, 0.02, 0.0, 0.0],  # 448 * 2^-13 < 0.0859375 <= 448 * 2^-12
                         [0.0, 0.0, 0.0, 0.0],          # all-zero row
                         [224.0, 0.5, 0.0, 0.0],        # 224 = 448 / 2 exactly: e = -1
                         [1.0, 0.0, 0.0, 0.0]], dtype=torch.bfloat16)
    codes, exps = oracle_mod.quantise_rows_e4m3(rows)
    assert exps.tolist() == [0, 1, -12, 0, -1, -8]
    assert codes[0, 0] == 0x7E and codes[1, 0] == 0x76 and codes[4, 0] == 0x7E     # 450 / 2 = 225 -> 224 = 0x76
    assert codes[3].tolist() == [0, 0, 0, 0]
    for o in range(rows.shape[0]):
        amax = rows[o].float().abs().max().item()
        e = int(exps[o])
        if amax > 0:
            assert amax <= 448 * 2.0 ** e and amax > 448 * 2.0 ** (e - 1)


def test_round_trip_error_bound_and_exact_bf16_values(oracle_mod):
    from paper_2512_21571_b200 import synth
    W = synth.normal(17, 3, (64, 512), 0.02, torch.bfloat16)
    W[5] = 0
    W[7, 3] = 1.5            # an outlier stretches that row's scale
    codes, exps = oracle_mod.quantise_rows_e4m3(W)
    D = oracle_mod.dequantise_rows_e4m3(codes, exps)
    # dequantised value = grid value * 2^e exactly (recomputed in float64 from the format's definition)
    c = codes.numpy().astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    ex, man = (c >> 3) & 15, c & 7
    grid = np.where(ex == 0, man * 2.0 ** -9, (1 + man / 8.0) * 2.0 ** (ex - 7.0)) * sign
    want = grid * (2.0 ** exps.numpy().astype(np.float64))[:, None]
    assert np.array_equal(D.double().numpy(), want)
    # nearest grid point: at most half a step away -- 2^-4 relative in the normal range, 2^-10 * 2^e below it
    w, d = W.double().numpy(), D.double().numpy()
    step = 2.0 ** exps.numpy().astype(np.float64)[:, None]
    bound = np.maximum(np.abs(w) * 2.0 ** -4, step * 2.0 ** -10)
    assert (np.abs(w - d) <= bound).all()
    assert (np.sign(d) * np.sign(w) >= 0).all()
    # the dequantised matrix is a fixed point of the rule (values, not codes: the exponent may drop by one)
    c2, e2 = oracle_mod.quantise_rows_e4m3(D)
    assert torch.equal(oracle_mod.dequantise_rows_e4m3(c2, e2), D)
    # brute force on one row: no other grid point is closer than the chosen one
    o = 7
    cand = np.array([oracle_mod.e4m3_to_f32(k) for k in range(0x7F)] + [-oracle_mod.e4m3_to_f32(k) for k in range(0x7F)])
    for k in range(0, 512, 37):
        x = w[o, k] / step[o, 0]
        assert abs(grid[o, k] - x) <= np.abs(cand - x).min() + 1e-12


def test_matmul_with_dequantised_rows_equals_scaled_code_products(oracle_mod):
    """y_o = 2^e_o * sum_k grid(code_ok) x_k: the row scale commutes with the sum (brute force in float64)."""
    from paper_2512_21571_b200 import synth
    W = synth.normal(19, 1, (24, 128), 0.02, torch.bfloat16)
    x = synth.normal(19, 2, (1, 128), 1.0, torch.float32)
    codes, exps = oracle_mod.quantise_rows_e4m3(W)
    D = oracle_mod.dequantise_rows_e4m3(codes, exps)
    got = oracle_mod.matmul(D, x)[0].double().numpy()
    grid = np.array([[oracle_mod.e4m3_to_f32(int(c)) for c in row] for row in codes.numpy()], dtype=np.float64)
    want = (grid @ x[0].double().numpy()) * 2.0 ** exps.numpy().astype(np.float64)
    assert np.allclose(got, want, rtol=1e-5, atol=1e-6)
