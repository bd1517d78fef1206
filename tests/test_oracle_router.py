"""Pins of the oracle's router front end (Section 3.2: feature vector -> MLP -> one score per expert) and of the load
report (Section 3.3: P_i, F_i, L_bal = N * sum P_i F_i): brute force in pure Python, closed forms with exact small
integers, hand-worked numbers, and the invariants the definitions imply.  No GPU."""
import math

import numpy as np

import oracle
import moqe_workloads as wl


def _bf16(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_router_mlp_brute_force_on_a_tiny_ragged_batch():
    g = np.random.default_rng(1)
    H, D, E = 5, 4, 3
    off = np.array([0, 3, 4, 4, 9], np.int32)                  # 3 rows, 1 row, NO rows, 5 rows
    Xf = wl.bf16_bits_to_f32(_bf16(g.standard_normal((9, H))))
    W1 = g.standard_normal((D, H)).astype(np.float32)
    W2 = g.standard_normal((E, D)).astype(np.float32)
    logits, pooled = oracle.router_mlp(_bf16(Xf), off, W1, W2)
    for s in range(4):
        r0, r1 = int(off[s]), int(off[s + 1])
        pool = [sum(float(Xf[r][h]) for r in range(r0, r1)) / (r1 - r0) if r1 > r0 else 0.0 for h in range(H)]
        hid = [max(0.0, sum(pool[h] * float(W1[d][h]) for h in range(H))) for d in range(D)]
        for h in range(H):
            assert abs(pooled[s][h] - pool[h]) <= 1e-15
        for e in range(E):
            ref = sum(hid[d] * float(W2[e][d]) for d in range(D))
            assert abs(logits[s][e] - ref) <= 1e-13
    assert np.all(logits[2] == 0.0)                            # the empty sample: pooled 0 -> logits 0


def test_router_mlp_closed_forms_with_exact_integers():
    H = 6
    X = np.array([[1, 2, 3, 4, 5, 6], [3, 2, 1, 0, -1, -2], [2, 2, 2, 2, 2, 2], [-4, 0, 4, 8, -8, 2]], np.float32)
    off = np.array([0, 2, 3, 4], np.int32)
    eye = np.eye(H, dtype=np.float32)
    # W1 = I, W2 = I: logits = relu(mean of the sample's rows)
    logits, pooled = oracle.router_mlp(_bf16(X), off, eye, eye)
    assert np.array_equal(pooled[0], [2, 2, 2, 2, 2, 2]) and np.array_equal(pooled[1], X[2]) and np.array_equal(pooled[2], X[3])
    assert np.array_equal(logits[2], [0, 0, 4, 8, 0, 2])       # the ReLU removes the negative means
    # W1 = -I: only the negative means survive, with their sign flipped
    logits, _ = oracle.router_mlp(_bf16(X), off, -eye, eye)
    assert np.array_equal(logits[2], [4, 0, 0, 0, 8, 0])
    # W2 sums the hidden units with weights (1, 2, ..): a hand-computed number
    W2 = np.arange(1, H + 1, dtype=np.float32)[None, :]
    logits, _ = oracle.router_mlp(_bf16(X), off, eye, W2)
    assert logits[2, 0] == 3 * 4 + 4 * 8 + 6 * 2 and logits[0, 0] == 2 * 21
    # scaling W2 scales the scores; the order of a sample's rows does not matter (exact with small integers)
    lg2, _ = oracle.router_mlp(_bf16(X), off, eye, 4 * W2)
    assert np.array_equal(lg2, 4 * logits)
    lg3, _ = oracle.router_mlp(_bf16(X[[1, 0, 2, 3]]), off, eye, W2)
    assert np.array_equal(lg3, logits)


def test_load_report_hand_example_and_invariants():
    # two samples, two experts: p = [[1/4, 3/4], [1/2, 1/2]]; dispatched to expert 1 and expert 0
    logits = np.array([[0.0, math.log(3.0)], [0.0, 0.0]])
    P, F, L = oracle.load_report(logits, np.array([1, 0], np.int32))
    assert np.allclose(P, [0.375, 0.625], atol=1e-15) and np.array_equal(F, [0.5, 0.5])
    assert abs(L - 1.0) < 1e-15                                # 2 * (0.375 * 0.5 + 0.625 * 0.5)
    # perfect balance: uniform scores, every expert gets the same number of samples -> L_bal = 1
    E, S = 4, 12
    P, F, L = oracle.load_report(np.zeros((S, E)), np.arange(S, dtype=np.int32) % E)
    assert np.allclose(P, 0.25) and np.allclose(F, 0.25) and abs(L - 1.0) < 1e-15
    # collapse: every sample surely to expert 0 -> L_bal = N
    lg = np.full((S, E), -1000.0)
    lg[:, 0] = 0.0
    P, F, L = oracle.load_report(lg, np.zeros(S, np.int32))
    assert abs(L - E) < 1e-12
    # random case: sums are one, softmax is shift-invariant, brute force
    g = np.random.default_rng(5)
    lg = g.standard_normal((S, E)) * 3
    ids = g.integers(0, E, size=S).astype(np.int32)
    P, F, L = oracle.load_report(lg, ids)
    assert abs(P.sum() - 1) < 1e-14 and abs(F.sum() - 1) < 1e-15
    P2, F2, L2 = oracle.load_report(lg + g.standard_normal((S, 1)) * 10, ids)
    assert np.allclose(P, P2, atol=1e-13) and abs(L - L2) < 1e-12
    Pb = [0.0] * E
    for s in range(S):
        ex = [math.exp(lg[s][e]) for e in range(E)]
        for e in range(E):
            Pb[e] += ex[e] / sum(ex) / S
    Fb = [float(np.sum(ids == e)) / S for e in range(E)]
    assert np.allclose(P, Pb, atol=1e-14) and np.allclose(F, Fb)
    assert abs(L - E * sum(a * b for a, b in zip(Pb, Fb))) < 1e-13
    # a planted mistake would show: F follows the ids, not the scores
    _, F3, _ = oracle.load_report(lg, np.zeros(S, np.int32))
    assert np.array_equal(F3, [1, 0, 0, 0])


def test_workload_router_matches_the_input_generator_within_fp32():
    """The workload module manufactures fp32 logits for the routed workload with numpy; the oracle's fp64 front end on
    the same weights must agree with it to fp32 accuracy (two independent implementations of the same definition)."""
    w = wl.get("qwen7b_mixed")
    layer = w.layers[0]
    off = np.array([0, 1, 2, 40, 41], np.int32)
    X = wl.activations_bf16("router/pin", int(off[-1]), layer.K)
    H, E = layer.K, w.n_experts
    w1 = wl.normal_f32(f"{w.name}/router/w1", (256, H), 1.0 / np.sqrt(H))
    w2 = wl.normal_f32(f"{w.name}/router/w2", (E, 256), 1.0 / np.sqrt(256.0))
    logits, pooled = oracle.router_mlp(X, off, w1, w2)
    gen = wl.router_logits(w, pooled=wl.mean_pool(X, off))
    assert np.allclose(pooled, wl.mean_pool(X, off), atol=1e-5)
    assert np.allclose(logits, gen, atol=2e-4)
