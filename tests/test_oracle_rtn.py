"""Pins for the oracle's storage conversions, RTN quantizer and dequantizer.

None of these re-types the oracle's formula: they check the oracle against
numpy/torch conversions, mathematical bounds, closed-form grids and brute force.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
import moqe_workloads as wl


# ---------------------------------------------------------------- conversions
def test_f16_conversion_matches_numpy():
    g = np.random.default_rng(1)
    vals = np.concatenate([
        g.standard_normal(4000).astype(np.float32) * np.float32(10.0) ** g.integers(-9, 6, 4000).astype(np.float32),
        np.array([0.0, -0.0, 1.0, 65504.0, 65519.9, 65520.0, 70000.0, np.inf, -np.inf,
                  2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0000001, 2.0 ** -14, 2.0 ** -14 * 0.99999,
                  6.1e-5, 5.96e-8, 2.98e-8, 1e-10, 1.00048828125, 1.0009765625 + 2.0 ** -12], dtype=np.float32),
    ])
    ours = oracle.f32_to_f16_bits(vals)
    with np.errstate(over="ignore"):
        ref = vals.astype(np.float16).view(np.uint16)
    assert np.array_equal(ours, ref)
    # and back: every finite half value
    allh = np.arange(0, 0x7C00, dtype=np.uint16)
    back = oracle.f16_bits_to_f32(allh)
    assert np.array_equal(back, allh.view(np.float16).astype(np.float32))


def test_bf16_conversion_matches_torch():
    g = np.random.default_rng(2)
    vals = (g.standard_normal(5000) * 10.0 ** g.integers(-20, 20, 5000)).astype(np.float32)
    vals = np.concatenate([vals, np.array([1.00390625, 1.01171875, 1.0 + 2.0 ** -8, 3.0e38, 0.0], dtype=np.float32)])
    ours = oracle.f32_to_bf16_bits(vals)
    ref = torch.from_numpy(vals).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    # the workload generator's own rounding must agree with both
    assert np.array_equal(wl.f32_to_bf16_bits(vals), ref)


# ---------------------------------------------------------------- helpers
CASES = [(8, 0, True), (8, 128, False), (4, 128, False), (4, 128, True), (4, 0, False),
         (4, 32, False), (3, 128, False), (3, 64, False), (3, 32, True), (2, 64, False)]


def _grid(scales, zeros, group, K):
    s = oracle.f16_bits_to_f32(scales).astype(np.float64)
    z = oracle.f16_bits_to_f32(zeros).astype(np.float64)
    g = K if group == 0 else group
    return np.repeat(s, g, axis=1), np.repeat(z, g, axis=1)


@pytest.mark.parametrize("bits,group,sym", CASES)
def test_code_range_and_roundtrip_bound(bits, group, sym):
    N, K = 48, 512
    W = wl.weights_f32(f"rtn/{bits}/{group}/{sym}", N, K)
    codes, scales, zeros = oracle.quantize_rtn(W, bits, group, sym)
    L = 2 ** bits - 1
    assert codes.dtype == np.uint8 and codes.max() <= L
    if sym:
        assert codes.min() >= 1                      # restricted symmetric range: code 0 unused
    s, z = _grid(scales, zeros, group, K)
    assert np.all(z == np.round(z)) and z.min() >= 0 and z.max() <= L
    if sym:
        assert np.all(z == 2 ** (bits - 1))
    What = oracle.dequantize(codes, scales, zeros, group).astype(np.float64)
    # dequantization is exact: s * (c - z) with an 11-bit and a <=9-bit significand
    assert np.array_equal(What, s * (codes.astype(np.float64) - z))
    err = np.abs(W.astype(np.float64) - What)
    unclamped = np.rint(W.astype(np.float64) / s) + z
    inside = (unclamped >= (1 if sym else 0)) & (unclamped <= L)
    slack = np.abs(W.astype(np.float64)) * 2.0 ** -23 + 1e-30      # one fp32 ulp of the quotient
    assert np.all(err[inside] <= s[inside] / 2 + slack[inside])
    # clamping: never for the symmetric grid, at most one step at the top for the asymmetric one
    if sym:
        assert inside.all()
    else:
        assert np.all(unclamped[~inside] == L + 1)
        assert np.all(err[~inside] <= s[~inside] * (0.5 + L * 2.0 ** -11) + slack[~inside])
        assert (~inside).mean() < 0.02


@pytest.mark.parametrize("bits,group,sym", CASES)
def test_extreme_elements(bits, group, sym):
    N, K = 16, 256
    W = wl.weights_f32(f"rtn-ext/{bits}/{group}/{sym}", N, K)
    g = K if group == 0 else group
    W[3, :g] = np.abs(W[3, :g]) + 0.001            # an all-positive group
    W[5, :g] = -np.abs(W[5, :g]) - 0.001           # an all-negative group
    codes, scales, zeros = oracle.quantize_rtn(W, bits, group, sym)
    L = 2 ** bits - 1
    qmax = 2 ** (bits - 1) - 1
    zf = oracle.f16_bits_to_f32(zeros)
    Wg = W.reshape(N, K // g, g)
    cg = codes.reshape(N, K // g, g).astype(np.int64)
    for n in range(N):
        for gi in range(K // g):
            w, c = Wg[n, gi], cg[n, gi]
            if sym:
                assert abs(int(c[np.argmax(np.abs(w))]) - 2 ** (bits - 1)) == qmax
            else:
                if w.min() < 0:
                    assert c[np.argmin(w)] == 0
                if w.max() > 0:
                    assert c[np.argmax(w)] >= L - 1
                if w.min() > 0:
                    assert zf[n, gi] == 0
                if w.max() < 0:
                    assert zf[n, gi] == L


@pytest.mark.parametrize("bits,group,sym", CASES)
def test_closed_form_grid_is_recovered_exactly(bits, group, sym):
    """W built ON a power-of-two grid must come back as exactly that grid."""
    N, K = 24, 384 if group in (0, 32, 64, 128) else 256
    g = K if group == 0 else group
    G = K // g
    rs = np.random.default_rng(bits * 1000 + g + int(sym))
    L = 2 ** bits - 1
    half = 2 ** (bits - 1)
    s0 = 2.0 ** rs.integers(-12, -3, size=(N, G))
    if sym:
        q0 = rs.integers(-(half - 1), half, size=(N, G, g))
        q0[:, :, 0] = half - 1
        q0[:, :, 1] = -(half - 1)
        z0 = np.full((N, G), half)
        c0 = q0 + half
    else:
        z0 = rs.integers(0, L + 1, size=(N, G))
        c0 = rs.integers(0, L + 1, size=(N, G, g))
        c0[:, :, 0] = 0
        c0[:, :, 1] = L
    W = (s0[:, :, None] * (c0 - z0[:, :, None])).reshape(N, K).astype(np.float32)
    codes, scales, zeros = oracle.quantize_rtn(W, bits, group, sym)
    assert np.array_equal(codes, c0.reshape(N, K).astype(np.uint8))
    assert np.array_equal(oracle.f16_bits_to_f32(scales), s0.astype(np.float32))
    assert np.array_equal(oracle.f16_bits_to_f32(zeros), z0.astype(np.float32))
    assert np.array_equal(oracle.dequantize(codes, scales, zeros, group), W)


def test_special_cases():
    N, K = 8, 256
    W = wl.weights_f32("rtn-special", N, K)
    # per-channel == one group of K
    a = oracle.quantize_rtn(W, 4, 0, False)
    b = oracle.quantize_rtn(W, 4, K, False)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))
    # deterministic
    c = oracle.quantize_rtn(W.copy(), 4, 0, False)
    assert all(np.array_equal(x, y) for x, y in zip(a, c))
    # all-zero matrix: degenerate groups -> scale 1, codes = z, dequant 0
    for sym in (True, False):
        codes, scales, zeros = oracle.quantize_rtn(np.zeros((N, K), np.float32), 4, 128, sym)
        assert np.all(oracle.f16_bits_to_f32(scales) == 1.0)
        assert np.all(codes == (8 if sym else 0))
        assert np.all(oracle.dequantize(codes, scales, zeros, 128) == 0.0)
    # scale that underflows fp16 to zero is degenerate too
    codes, scales, zeros = oracle.quantize_rtn(np.full((2, 64), 1e-9, np.float32), 4, 0, False)
    assert np.all(oracle.f16_bits_to_f32(scales) == 1.0) and np.all(codes == 0)
    # b=8 symmetric on a matrix of +-a only: codes are the two ends of the grid
    sgn = np.where(np.random.default_rng(0).random((N, K)) < 0.5, -1.0, 1.0).astype(np.float32)
    sgn[:, 0], sgn[:, 1] = 1.0, -1.0
    codes, scales, zeros = oracle.quantize_rtn(sgn * np.float32(0.0127), 8, 0, True)
    assert set(np.unique(codes)) == {1, 255}
    assert np.array_equal(codes == 255, sgn > 0)
    # a single group
    codes, scales, zeros = oracle.quantize_rtn(W[:1, :32], 3, 32, False)
    assert scales.shape == (1, 1) and codes.shape == (1, 32)
    # bad arguments
    with pytest.raises(ValueError):
        oracle.quantize_rtn(W, 4, 100, False)


@pytest.mark.parametrize("bits,sym", [(2, False), (2, True), (3, False), (4, False), (4, True), (8, True), (8, False)])
def test_brute_force_nearest_code(bits, sym):
    """4x8 tiles: the returned code is the grid point nearest to w (exact arithmetic)."""
    rs = np.random.default_rng(100 + bits + int(sym))
    L = 2 ** bits - 1
    for trial in range(6):
        W = (rs.standard_normal((4, 8)) * 0.02).astype(np.float32)
        codes, scales, zeros = oracle.quantize_rtn(W, bits, 8, sym)
        s = oracle.f16_bits_to_f32(scales)
        z = oracle.f16_bits_to_f32(zeros)
        for n in range(4):
            sF, zF = Fraction(float(s[n, 0])), int(z[n, 0])
            lo_code = 1 if sym else 0
            for k in range(8):
                wF = Fraction(float(W[n, k]))
                errs = [abs(wF - sF * (c - zF)) for c in range(lo_code, L + 1)]
                best = min(errs)
                got = errs[int(codes[n, k]) - lo_code]
                # equal to the minimum, up to one fp32 rounding of the quotient w/s
                assert got - best <= sF * Fraction(1, 2 ** 22)
