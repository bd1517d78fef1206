"""GPU parity: routing arg-max, id expansion, stable counting sort, gather / scatter -- all bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import moqe_workloads as wl

pytestmark = pytest.mark.gpu


def test_route_matches_oracle():
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev
    g = np.random.default_rng(21)
    for S, E in [(1, 1), (16, 3), (68, 4), (1000, 5), (70000, 2)]:
        logits = g.standard_normal((S, E)).astype(np.float32)
        logits[g.random((S, E)) < 0.05] = np.float32("nan")
        logits[::7] = np.round(logits[::7])                      # ties
        if S > 3:
            logits[3] = np.float32("nan")
        ids = moqe.moqe_route(torch.from_numpy(logits).to(dev())).cpu().numpy()
        assert np.array_equal(ids, oracle.route(logits))
    for name in wl.WORKLOAD_ORDER:
        w = wl.get(name)
        if w.routing == "router_mlp":
            X = wl.activations_bf16(f"{name}/pool", w.M_of(w.layers[0]), w.layers[0].K)
            logits = wl.router_logits(w, pooled=wl.mean_pool(X, w.row_offsets(w.layers[0])))
        else:
            logits = wl.router_logits(w)
        ids = moqe.moqe_route(torch.from_numpy(logits).to(dev())).cpu().numpy()
        assert np.array_equal(ids, oracle.route(logits))


def test_expand_ids_matches_oracle():
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev
    for name in ("tiny", "qwen7b_mixed", "resnet50_1x1"):
        w = wl.get(name)
        off = w.row_offsets(w.layers[0])
        sid = (np.arange(w.n_samples) * 7 % w.n_experts).astype(np.int32)
        got = moqe.moqe_expand_ids(torch.from_numpy(sid).to(dev()), torch.from_numpy(off).to(dev()), int(off[-1]))
        assert np.array_equal(got.cpu().numpy(), oracle.expand_ids(sid, off))


@pytest.mark.parametrize("M,E", [(0, 3), (1, 1), (17, 2), (1000, 3), (1024, 4), (1025, 4), (5000, 5), (70001, 3),
                                 (802816, 3), (4160, 32)])
def test_sort_matches_oracle(M, E):
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev
    g = np.random.default_rng(M + E)
    ids = g.integers(0, E, size=M).astype(np.int32)
    if E >= 3:
        ids[ids == 1] = 0                                        # an expert with no rows
    _, perm, offsets = moqe.moqe_permute(None, torch.from_numpy(ids).to(dev()), E)
    counts, off_ref, perm_ref, _ = oracle.permutation(ids, E)
    assert np.array_equal(offsets.cpu().numpy(), off_ref)
    assert np.array_equal(perm.cpu().numpy(), perm_ref)
    assert moqe.moqe_async_status() == moqe.OK


@pytest.mark.parametrize("S,E,rows", [(1, 1, None), (16, 3, None), (16, 3, "ragged"), (1024, 5, None), (100, 32, "ragged"),
                                      (7, 4, "empty-samples")])
def test_route_permute_in_one_launch_matches_the_three_oracle_steps(S, E, rows):
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev
    g = np.random.default_rng(S * 31 + E)
    logits = g.standard_normal((S, E)).astype(np.float32)
    logits[g.random((S, E)) < 0.05] = np.float32("nan")
    logits[::5] = np.round(logits[::5])                          # ties
    if E >= 3:
        logits[:, 1] = -100.0                                    # an expert with no rows
    if rows is None:
        off, M = None, S
    else:
        n = g.integers(0 if rows == "empty-samples" else 1, 1024 // S + 1, size=S)
        off = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
        M = int(off[-1])
    ids, row_ids, perm, offsets = moqe.moqe_route_permute(torch.from_numpy(logits).to(dev()),
                                                          None if off is None else torch.from_numpy(off).to(dev()), M)
    ids_ref = oracle.route(logits)
    rid_ref = ids_ref if off is None else oracle.expand_ids(ids_ref, off)
    _, off_ref, perm_ref, _ = oracle.permutation(rid_ref, E)
    assert np.array_equal(ids.cpu().numpy(), ids_ref)
    assert np.array_equal(row_ids.cpu().numpy(), rid_ref)
    assert np.array_equal(offsets.cpu().numpy(), off_ref)
    assert np.array_equal(perm.cpu().numpy(), perm_ref)
    # beyond the single-block limit nothing is launched
    big = torch.zeros((1025, 2), dtype=torch.float32, device=dev())
    with pytest.raises(moqe.MoqeError):
        moqe.moqe_route_permute(big, None, 1025)


@pytest.mark.parametrize("M,C,E", [(64, 1024, 2), (333, 40, 4), (4160, 3584, 4), (5000, 8, 3)])
def test_permute_unpermute_rows(M, C, E):
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev, bf16_to_torch, torch_to_bits
    g = np.random.default_rng(M * 3 + C)
    X = g.integers(0, 65536, size=(M, C)).astype(np.uint16)
    ids = g.integers(0, E, size=M).astype(np.int32)
    Xp, perm, offsets = moqe.moqe_permute(bf16_to_torch(X), torch.from_numpy(ids).to(dev()), E)
    _, _, perm_ref, _ = oracle.permutation(ids, E)
    assert np.array_equal(perm.cpu().numpy(), perm_ref)
    assert np.array_equal(torch_to_bits(Xp), oracle.permute_rows(X, perm_ref))
    back = moqe.moqe_unpermute(Xp, perm)
    assert np.array_equal(torch_to_bits(back), X)


def test_invalid_ids_are_reported_not_trapped():
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev, bf16_to_torch, torch_to_bits
    g = np.random.default_rng(5)
    for M in (100, 3000):
        E = 3
        ids = g.integers(0, E, size=M).astype(np.int32)
        bad = np.array([4, M // 2, M - 1])
        ids[bad] = [E, -1, 99]
        X = g.integers(1, 65536, size=(M, 16)).astype(np.uint16)
        Xp, perm, offsets = moqe.moqe_permute(bf16_to_torch(X), torch.from_numpy(ids).to(dev()), E)
        assert moqe.moqe_async_status() == moqe.ERR_EXPERT_ID
        assert moqe.moqe_async_status() == moqe.OK                # cleared by the read
        good = np.setdiff1d(np.arange(M), bad)
        _, off_ref, perm_ref, _ = oracle.permutation(ids[good], E)
        off = offsets.cpu().numpy()
        assert np.array_equal(off, off_ref)                       # offsets[E] counts the valid rows only
        p = perm.cpu().numpy()
        assert np.array_equal(p[: off[E]], good[perm_ref])
        assert np.array_equal(p[off[E]:], bad)                    # invalid rows last, in order
        Xp_bits = torch_to_bits(Xp)
        assert np.all(Xp_bits[off[E]:] == 0)
        assert np.array_equal(Xp_bits[: off[E]], X[p[: off[E]]])
