"""Pins for the oracle's routed GEMM (each row times ITS expert's dequantized weight)."""
import numpy as np
import pytest

import oracle
import moqe_workloads as wl


def _experts(W, specs):
    out = []
    for bits, group, sym in specs:
        c, s, z = oracle.quantize_rtn(W, bits, group, sym)
        out.append(oracle.dequantize(c, s, z, group))
    return out


SPECS = [(8, 0, True), (4, 128, False), (3, 128, False)]


def test_brute_force_small():
    """Pure-Python fp64 loops on 4x8, 8x16 and M=3 problems (N != K so a transposed operand fails)."""
    for (M, N, K, seed) in [(4, 8, 16, 0), (8, 16, 32, 1), (3, 5, 64, 2)]:
        rs = np.random.default_rng(seed)
        Xb = wl.f32_to_bf16_bits(rs.standard_normal((M, K)).astype(np.float32))
        Xf = wl.bf16_bits_to_f32(Xb)
        What = [(rs.standard_normal((N, K)) * 0.02).astype(np.float32) for _ in range(3)]
        ids = rs.integers(0, 3, size=M).astype(np.int32)
        Y, Yf = oracle.routed_gemm(Xb, ids, What, want_f32=True)
        Y64 = oracle.routed_gemm_f64(Xb, ids, What)
        for m in range(M):
            for n in range(N):
                acc = 0.0
                for k in range(K):
                    acc += float(Xf[m, k]) * float(What[ids[m]][n, k])
                assert abs(Y64[m, n] - acc) <= 1e-15 * max(1.0, abs(acc))
                assert abs(float(Yf[m, n]) - acc) <= 1e-6 * (abs(acc) + 0.05)
        assert np.array_equal(Y, wl.f32_to_bf16_bits(Yf))


def test_exact_integer_case():
    """On-grid W (power-of-two scale) and small-integer X: every partial sum is an integer below
    2^24 times the scale, so the fp32 result must equal the int64 product exactly."""
    rs = np.random.default_rng(5)
    M, N, K = 9, 24, 512
    q = rs.integers(-127, 128, size=(N, K))
    q[:, 0], q[:, 1] = 127, -127
    s0 = 2.0 ** -9
    W = (q * s0).astype(np.float32)
    c, s, z = oracle.quantize_rtn(W, 8, 0, True)
    What = oracle.dequantize(c, s, z, 0)
    assert np.array_equal(What, W)
    Xi = rs.integers(-8, 9, size=(M, K))
    Xb = wl.f32_to_bf16_bits(Xi.astype(np.float32))
    ids = np.zeros(M, np.int32)
    _, Yf = oracle.routed_gemm(Xb, ids, [What], want_f32=True)
    exact = (Xi.astype(np.int64) @ q.astype(np.int64).T).astype(np.float64) * s0
    assert np.array_equal(Yf.astype(np.float64), exact)


def test_single_expert_equivalence_and_locality():
    w = wl.get("tiny")
    layer = w.layers[0]
    Wfull, X = wl.layer_inputs(w, layer)
    Wfull, X = Wfull[:96, :], X[:40, :]                  # N=96 != K=1024
    What = _experts(Wfull, SPECS)
    M = X.shape[0]
    rs = np.random.default_rng(6)
    ids = rs.integers(0, 3, size=M).astype(np.int32)
    Y = oracle.routed_gemm(X, ids, What)
    # all ids equal  ==  that expert alone (one expert per sample: the others never matter)
    for e in range(3):
        Ye = oracle.routed_gemm(X, np.full(M, e, np.int32), What)
        Y1 = oracle.routed_gemm(X, np.zeros(M, np.int32), [What[e]])
        assert np.array_equal(Ye, Y1)
        assert np.array_equal(Y[ids == e], Ye[ids == e])          # row-locality
        ref = wl.bf16_bits_to_f32(X).astype(np.float64) @ What[e].astype(np.float64).T
        got = wl.bf16_bits_to_f32(Ye).astype(np.float64)
        assert np.max(np.abs(got - ref)) <= 2.0 ** -8 * np.max(np.abs(ref)) + 1e-6
    # batch shuffle: outputs shuffle identically, bit for bit
    p = rs.permutation(M)
    assert np.array_equal(oracle.routed_gemm(X[p], ids[p], What), Y[p])
    # row sampling returns the same rows
    rows = np.array([39, 0, 7, 7, 21], np.int32)
    assert np.array_equal(oracle.routed_gemm(X, ids, What, rows=rows), Y[rows])
    # sorting by expert, multiplying, and scattering back is the same thing
    _, offsets, perm, _ = oracle.permutation(ids, 3)
    Yp = oracle.routed_gemm(oracle.permute_rows(X, perm), ids[perm], What)
    assert np.array_equal(oracle.unpermute_rows(Yp, perm), Y)


def test_identity_input_returns_weight_rows():
    rs = np.random.default_rng(7)
    N, K = 40, 64
    W = (rs.standard_normal((N, K)) * 0.02).astype(np.float32)
    What = _experts(W, [(4, 32, False), (8, 0, True)])
    Xb = wl.f32_to_bf16_bits(np.eye(K, dtype=np.float32))
    ids = (np.arange(K) % 2).astype(np.int32)
    Y = oracle.routed_gemm(Xb, ids, What)                        # [K][N]
    for m in range(K):
        assert np.array_equal(Y[m], wl.f32_to_bf16_bits(What[ids[m]][:, m].copy()))


def test_fp32_accumulation_error_is_far_below_tolerance():
    rs = np.random.default_rng(8)
    M, N, K = 4, 64, 11008
    W = (rs.standard_normal((N, K)) * 0.02).astype(np.float32)
    What = _experts(W, [(4, 128, False)])
    Xb = wl.activations_bf16("gemm-acc", M, K)
    ids = np.zeros(M, np.int32)
    _, Yf = oracle.routed_gemm(Xb, ids, What, want_f32=True)
    Y64 = oracle.routed_gemm_f64(Xb, ids, What)
    assert np.mean(np.abs(Yf - Y64)) < 5e-5
    assert np.max(np.abs(Yf - Y64)) < 5e-4


def test_errors():
    Xb = np.zeros((2, 8), np.uint16)
    What = [np.zeros((4, 8), np.float32)]
    with pytest.raises(ValueError):
        oracle.routed_gemm(Xb, np.array([0, 1], np.int32), What)
    with pytest.raises(ValueError):
        oracle.routed_gemm(Xb, np.array([0, 0], np.int32), [np.zeros((4, 16), np.float32)])
