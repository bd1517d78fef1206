"""Pins of the oracle's two fused steps around the routed product (Section 4.4: whole expert forwards are what the
paper times): the gated pair silu(X.Wg^T) * (X.Wu^T) and the residual add.  Closed forms (X = I), special values of
silu, and reductions to the already pinned plain product.  No GPU."""
import numpy as np

import oracle
import moqe_workloads as wl


def _bf16(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _f32(bits):
    return wl.bf16_bits_to_f32(bits)


def test_gated_pair_closed_form_with_identity_inputs():
    g = np.random.default_rng(2)
    K = N = 24
    X = _bf16(np.eye(K))
    Wg = [(_f32(_bf16(g.standard_normal((N, K)) * 3))) for _ in range(2)]      # bf16-representable values
    Wu = [(_f32(_bf16(g.standard_normal((N, K))))) for _ in range(2)]
    ids = (np.arange(K) % 2).astype(np.int32)
    Y = _f32(oracle.routed_gated_pair(X, ids, Wg, Wu))
    for m in range(K):
        a = Wg[ids[m]][:, m].astype(np.float64)
        b = Wu[ids[m]][:, m].astype(np.float64)
        ref = a / (1.0 + np.exp(-a)) * b
        # one bf16 rounding of a value computed in fp32: within one bf16 ulp of the fp64 value, mostly equal
        assert np.all(np.abs(Y[m] - ref) <= np.maximum(np.abs(ref), 1e-30) * 2.0 ** -7)
        assert np.mean(Y[m] == _f32(_bf16(ref))) > 0.95


def test_gated_pair_special_values():
    K, N = 8, 4
    X = _bf16(np.eye(K)[:4])
    Wu = [np.full((N, K), 2.0, np.float32)]
    # silu(0) = 0 exactly
    Y = oracle.routed_gated_pair(X, np.zeros(4, np.int32), [np.zeros((N, K), np.float32)], Wu)
    assert np.all(_f32(Y) == 0.0)
    # far right: silu(a) = a; far left: silu(a) = -0
    Y = _f32(oracle.routed_gated_pair(X, np.zeros(4, np.int32), [np.full((N, K), 64.0, np.float32)], Wu))
    assert np.all(Y == 128.0)
    Y = _f32(oracle.routed_gated_pair(X, np.zeros(4, np.int32), [np.full((N, K), -120.0, np.float32)], Wu))
    assert np.all(np.abs(Y) < 1e-30)
    # silu(a) - silu(-a) = a, checked through two calls with opposite gate weights and up = 1
    a = np.array([[0.5, 1.0, 2.0, 3.0, 0.25, 4.0, 1.5, 0.125]] * N, np.float32)
    one = [np.ones((N, K), np.float32)]
    Xe = _bf16(np.eye(K))
    yp = _f32(oracle.routed_gated_pair(Xe, np.zeros(K, np.int32), [a], one)).astype(np.float64)
    yn = _f32(oracle.routed_gated_pair(Xe, np.zeros(K, np.int32), [-a], one)).astype(np.float64)
    assert np.all(np.abs((yp - yn) - a.T) <= np.abs(a.T) * 2.0 ** -7)
    # the gate decides the sign pattern, the up projection scales: swapping them changes the result
    b = np.linspace(-2, 2, N * K, dtype=np.float32).reshape(N, K)
    y1 = oracle.routed_gated_pair(Xe, np.zeros(K, np.int32), [a], [b])
    y2 = oracle.routed_gated_pair(Xe, np.zeros(K, np.int32), [b], [a])
    assert not np.array_equal(y1, y2)


def test_gated_pair_uses_each_rows_expert_and_the_plain_products():
    g = np.random.default_rng(3)
    M, K, N, E = 7, 64, 10, 3
    X = wl.activations_bf16("ep/X", M, K)
    Wg = [g.standard_normal((N, K)).astype(np.float32) * 0.2 for _ in range(E)]
    Wu = [g.standard_normal((N, K)).astype(np.float32) * 0.2 for _ in range(E)]
    ids = g.integers(0, E, size=M).astype(np.int32)
    Y = _f32(oracle.routed_gated_pair(X, ids, Wg, Wu)).astype(np.float64)
    _, a = oracle.routed_gemm(X, ids, Wg, want_f32=True)       # the pinned plain product, fp32 accumulators
    _, b = oracle.routed_gemm(X, ids, Wu, want_f32=True)
    ref = a.astype(np.float64) / (1.0 + np.exp(-a.astype(np.float64))) * b.astype(np.float64)
    assert np.all(np.abs(Y - ref) <= np.maximum(np.abs(ref), 1e-30) * 2.0 ** -7)
    # row locality: a row's output does not depend on the others
    Y1 = _f32(oracle.routed_gated_pair(X[3:4], ids[3:4], Wg, Wu))
    assert np.array_equal(Y1[0], _f32(oracle.routed_gated_pair(X, ids, Wg, Wu))[3])


def test_residual_add_reduces_to_the_plain_product_and_to_the_residual():
    g = np.random.default_rng(4)
    M, K, N, E = 6, 48, 9, 2
    X = wl.activations_bf16("ep/Xr", M, K)
    W = [g.standard_normal((N, K)).astype(np.float32) * 0.1 for _ in range(E)]
    ids = g.integers(0, E, size=M).astype(np.int32)
    R = _bf16(g.standard_normal((M, N)))
    zero = np.zeros((M, N), np.uint16)
    assert np.array_equal(oracle.routed_gemm_residual(X, ids, W, zero), oracle.routed_gemm(X, ids, W))
    assert np.array_equal(oracle.routed_gemm_residual(np.zeros_like(X), ids, W, R), R)
    # exact small integers: Y = X.W^T + R exactly
    Xi = g.integers(-4, 5, size=(M, K)).astype(np.float32)
    Wi = [g.integers(-3, 4, size=(N, K)).astype(np.float32) for _ in range(E)]
    Ri = g.integers(-50, 51, size=(M, N)).astype(np.float32)
    Y = _f32(oracle.routed_gemm_residual(_bf16(Xi), ids, Wi, _bf16(Ri)))
    ref = np.stack([Xi[m] @ Wi[ids[m]].T for m in range(M)]) + Ri
    assert np.array_equal(Y, _f32(_bf16(ref)))
    # the residual is added BEFORE the single rounding: a + r rounded once differs from round(a) + r rounded
    A = _f32(oracle.routed_gemm(X, ids, W))
    Y2 = _f32(_bf16(A + _f32(R)))
    Y3 = _f32(oracle.routed_gemm_residual(X, ids, W, R))
    assert np.all(np.abs(Y2 - Y3) <= (np.abs(A) + np.abs(_f32(R))) * 2.0 ** -7 + 1e-30)
    _, acc = oracle.routed_gemm(X, ids, W, want_f32=True)
    assert np.array_equal(Y3, _f32(_bf16(acc + _f32(R))))       # the unrounded accumulator plus the residual, rounded once
