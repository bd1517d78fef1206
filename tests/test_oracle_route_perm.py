"""Pins for the oracle's hard routing and stable counting-sort permutation."""
import numpy as np
import pytest

import oracle
import moqe_workloads as wl


def test_route_is_first_max():
    g = np.random.default_rng(3)
    for E in (1, 2, 3, 4, 5):
        logits = g.standard_normal((257, E)).astype(np.float32)
        assert np.array_equal(oracle.route(logits), np.argmax(logits, axis=1).astype(np.int32))
    # ties -> smallest index
    t = np.array([[1, 1, 0], [0, 2, 2], [5, 5, 5], [-1, -3, -1]], dtype=np.float32)
    assert oracle.route(t).tolist() == [0, 1, 0, 0]
    # integer-valued logits with many ties
    li = g.integers(0, 3, size=(500, 5)).astype(np.float32)
    assert np.array_equal(oracle.route(li), np.argmax(li, axis=1))


def test_route_invariances():
    g = np.random.default_rng(4)
    logits = g.permutation(64 * 5).reshape(64, 5).astype(np.float32)     # distinct integers: no ties
    ids = oracle.route(logits)
    col = g.permutation(5)
    ids_p = oracle.route(logits[:, col])
    assert np.array_equal(col[ids_p], ids)
    shift = g.integers(-1000, 1000, size=(64, 1)).astype(np.float32)
    assert np.array_equal(oracle.route(logits + shift), ids)              # exact integer shifts
    # softmax is monotone: routing on probabilities equals routing on logits
    z = logits.astype(np.float64) / 50.0
    p = np.exp(z - z.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    assert np.array_equal(oracle.route(p.astype(np.float32)), ids)


def test_route_nan_rules():
    nan = np.float32("nan")
    t = np.array([[nan, 1, 2], [3, nan, 1], [nan, nan, nan], [nan, -np.inf, nan], [np.inf, nan, np.inf]], np.float32)
    assert oracle.route(t).tolist() == [2, 0, 0, 1, 0]


def test_route_workload_logits_are_one_hot_recoverable():
    for name in ("tiny", "llama7b_decode", "llama7b_prefill", "resnet50_1x1"):
        w = wl.get(name)
        logits = wl.router_logits(w)
        ids = oracle.route(logits)
        assert ids.shape == (w.n_samples,) and ids.min() >= 0 and ids.max() < w.n_experts
        assert np.all(logits[np.arange(w.n_samples), ids] == 1.0)
    # skewed routing follows its probabilities roughly (8 samples only -> use a larger draw)
    w = wl.get("llama7b_prefill")
    big = wl.Workload("skew-check", w.layers, w.experts, (1,) * 4000, "skewed", w.routing_probs)
    f = np.bincount(oracle.route(wl.router_logits(big)), minlength=3) / 4000.0
    assert np.allclose(f, [0.7, 0.2, 0.1], atol=0.03)


@pytest.mark.parametrize("M,E", [(0, 3), (1, 1), (17, 2), (1000, 3), (4160, 4), (5000, 5)])
def test_permutation_properties(M, E):
    g = np.random.default_rng(M * 7 + E)
    ids = g.integers(0, E, size=M).astype(np.int32)
    if E >= 3 and M > 0:
        ids[ids == 1] = 0                                      # an expert that receives no rows
    counts, offsets, perm, inv = oracle.permutation(ids, E)
    assert counts.sum() == M and offsets[0] == 0 and offsets[E] == M          # sum_i F_i = 1
    assert np.array_equal(counts, np.bincount(ids, minlength=E))
    assert np.array_equal(np.diff(offsets), counts)
    assert np.array_equal(np.sort(perm), np.arange(M))                       # bijection
    srt = ids[perm]
    assert np.all(np.diff(srt) >= 0)                                        # grouped by expert
    same = np.diff(srt) == 0
    assert np.all(np.diff(perm)[same] > 0)                                  # stable
    assert np.array_equal(perm, np.argsort(ids, kind="stable").astype(np.int32))
    assert np.array_equal(inv[perm], np.arange(M))
    for e in range(E):
        assert np.all(ids[perm[offsets[e]:offsets[e + 1]]] == e)


def test_permute_unpermute_roundtrip_and_errors():
    g = np.random.default_rng(9)
    M, Cc, E = 333, 40, 4
    X = g.integers(0, 65536, size=(M, Cc)).astype(np.uint16)
    ids = g.integers(0, E, size=M).astype(np.int32)
    _, _, perm, inv = oracle.permutation(ids, E)
    Xp = oracle.permute_rows(X, perm)
    assert np.array_equal(Xp, X[perm])
    assert np.array_equal(oracle.unpermute_rows(Xp, perm), X)
    bad = ids.copy()
    bad[5] = E
    with pytest.raises(ValueError):
        oracle.permutation(bad, E)
    bad[5] = -1
    with pytest.raises(ValueError):
        oracle.permutation(bad, E)


def test_expand_ids():
    ids = np.array([2, 0, 1], np.int32)
    off = np.array([0, 3, 3, 7], np.int32)
    assert oracle.expand_ids(ids, off).tolist() == [2, 2, 2, 1, 1, 1, 1]
    for name in ("tiny", "qwen7b_mixed"):
        w = wl.get(name)
        off = w.row_offsets(w.layers[0])
        sid = np.arange(w.n_samples, dtype=np.int32) % w.n_experts
        assert np.array_equal(oracle.expand_ids(sid, off), np.repeat(sid, np.diff(off)))
