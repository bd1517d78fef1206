"""GPU parity: the routed dequant-GEMM against the oracle, element by element, on seeded inputs.

Tolerance (stated by the target: bf16 output, fp32 accumulation): max relative error 1e-2
(|d| / max(|ref|, rms(ref))) and mean absolute error <= 2e-3, both sides rounded to bf16.
"""
import numpy as np
import pytest
import torch

import oracle
import moqe_workloads as wl

pytestmark = pytest.mark.gpu

ALL_FORMATS = [(8, 0, True), (4, 128, False), (3, 128, False), (4, 128, True), (3, 64, False), (4, 0, False),
               (4, 32, False), (8, 128, False), (3, 32, True), (4, 256, False), (2, 128, False), (2, 64, True)]


def _run(X, ids, gpu, path=0):
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev, bf16_to_torch, torch_to_bits
    # the output starts as NaN everywhere: an element that no kernel wrote fails the comparison
    N = gpu[0].N
    Y = torch.full((X.shape[0], N), float("nan"), dtype=torch.bfloat16, device=dev())
    moqe.moqe_routed_qgemm(bf16_to_torch(X), torch.from_numpy(ids).to(dev()), gpu, Y=Y, path=path)
    st = moqe.moqe_async_status()
    return torch_to_bits(Y), st


def _paths():
    import paper_2508_09204_b200 as moqe
    return [moqe.PATH_STREAM, moqe.PATH_TCGEN05]


@pytest.mark.parametrize("path", [1, 3, 4])
def test_tiny_workload_full_compare(path):
    """Config 'tiny': 1024x1024, W8 per-channel + W4 g128, 4 sequences x 16 tokens, every element compared."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close, assert_expert_matches
    w = wl.get("tiny")
    layer = w.layers[0]
    W, X = wl.layer_inputs(w, layer)
    gpu, What, canon = build_experts(W, w.experts)
    for e, c in zip(gpu, canon):
        assert_expert_matches(e, c)
    ids = oracle.expand_ids(oracle.route(wl.router_logits(w)), w.row_offsets(layer))
    Y, st = _run(X, ids, gpu, path)
    assert st == moqe.OK
    ref = oracle.routed_gemm(X, ids, What)
    mx, mean = assert_close(Y, ref, "tiny")
    assert mean < 2e-4            # in practice the two sides differ by a few bf16 roundings only


@pytest.mark.parametrize("path", [1, 3, 4])
@pytest.mark.parametrize("M,N,K", [(1, 128, 128), (5, 200, 320), (16, 384, 1280), (37, 136, 2304), (64, 1000, 640),
                                   (150, 264, 1408)])
def test_all_formats_small_shapes(path, M, N, K):
    """Every supported format as its own expert; ragged N (not a multiple of 16/128), K not a multiple of 128,
    several K blobs and splits, an expert that gets no rows."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close
    specs = [f for f in ALL_FORMATS if f[1] == 0 or K % f[1] == 0]
    W = wl.weights_f32(f"qg/{N}/{K}", N, K)
    X = wl.activations_bf16(f"qg/{M}/{K}", M, K)
    gpu, What, _ = build_experts(W, specs)
    E = len(specs)
    rs = np.random.default_rng(M + N + K)
    ids = rs.integers(0, E, size=M).astype(np.int32)
    if M > 4:
        ids[ids == 2] = 0                                        # expert 2 idle
    Y, st = _run(X, ids, gpu, path)
    assert st == moqe.OK
    assert_close(Y, oracle.routed_gemm(X, ids, What), f"M{M} N{N} K{K}")


DECODE_FORMATS = [(8, 0, True), (4, 128, False), (3, 128, False), (4, 128, True), (4, 0, False), (8, 128, False), (2, 128, False), (2, 0, True), (2, 256, False),
                  (4, 256, False), (3, 0, True), (8, 0, False), (3, 256, True)]


@pytest.mark.parametrize("M,N,K", [(1, 128, 128), (5, 200, 320), (16, 384, 1280), (13, 136, 2304), (16, 1000, 640),
                                   (7, 4096, 1024), (16, 512, 11008), (9, 128, 32768), (17, 200, 320), (32, 384, 1280),
                                   (29, 1000, 640), (32, 512, 11008), (24, 128, 32768)])
def test_decode_kernel_all_formats(M, N, K):
    """The decode kernel (path 5: at most 32 rows; above 16 its instantiation with four token blocks per expert, per-channel experts or groups of >= 128 k): every such
    format as its own expert, ragged N, K not a multiple of 128, split K with several contributors per segment
    (dozens in the last, one-tile-wide case, where most CTAs hold nothing but the middle of a segment), an expert
    that gets no rows."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close
    specs = [f for f in DECODE_FORMATS if f[1] == 0 or K % f[1] == 0]
    W = wl.weights_f32(f"dq/{N}/{K}", N, K)
    X = wl.activations_bf16(f"dq/{M}/{K}", M, K)
    gpu, What, _ = build_experts(W, specs)
    rs = np.random.default_rng(7 * M + N + K)
    ids = rs.integers(0, len(specs), size=M).astype(np.int32)
    if M > 4:
        ids[ids == 2] = 0                                        # expert 2 idle
    for _ in range(2):                                           # twice: the arrival counters must come back to zero
        Y, st = _run(X, ids, gpu, moqe.PATH_DECODE)
        assert st == moqe.OK
        assert_close(Y, oracle.routed_gemm(X, ids, What), f"decode M{M} N{N} K{K}")
    # batch shuffle: rows move with their inputs, bit for bit
    pm = rs.permutation(M)
    Yp, _ = _run(X[pm], ids[pm], gpu, moqe.PATH_DECODE)
    assert np.array_equal(Yp, Y[pm])


def test_decode_kernel_several_layers_in_one_launch():
    """q/k/v-like and gate/up-like groups: layers of different N (and formats) that share the routing, one launch;
    every layer must equal its own single-layer call bit for bit, and the oracle within tolerance."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close, dev, bf16_to_torch, torch_to_bits
    M, K = 11, 1536
    shapes = [(512, [(8, 0, True), (4, 128, False), (3, 128, False)]),
              (136, [(4, 128, True), (8, 128, False), (4, 256, False)]),
              (1000, [(3, 0, True), (4, 0, False), (8, 0, False)])]
    ids = np.random.default_rng(5).integers(0, 3, size=M).astype(np.int32)
    ids[ids == 1] = 2                                            # expert 1 idle in every layer
    idd = torch.from_numpy(ids).to(dev())
    _, perm, offsets = moqe.moqe_permute(None, idd, 3)
    Xs, Ys, gpus, refs, singles = [], [], [], [], []
    for li, (N, specs) in enumerate(shapes):
        W = wl.weights_f32(f"multi/{li}", N, K)
        X = wl.activations_bf16(f"multi/X{li}", M, K)
        gpu, What, _ = build_experts(W, specs)
        Xd = bf16_to_torch(X)
        Xs.append(Xd)
        gpus.append(gpu)
        Ys.append(torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev()))
        refs.append(oracle.routed_gemm(X, ids, What))
        singles.append(torch_to_bits(moqe.moqe_routed_qgemm(Xd, idd, gpu, path=moqe.PATH_DECODE)))
    ws = moqe.alloc_workspace(moqe.moqe_routed_qgemm_workspace(M, shapes[0][0], K, 3))
    moqe.moqe_routed_qgemm_workspace_clear(ws, M, shapes[0][0], K, 3)
    for _ in range(2):
        for Y in Ys:
            Y.fill_(float("nan"))
        moqe.moqe_routed_qgemm_sorted_multi(Xs, perm, offsets, gpus, Ys, ws)
        assert moqe.moqe_async_status() == moqe.OK
        for li in range(len(shapes)):
            got = torch_to_bits(Ys[li])
            assert_close(got, refs[li], f"multi layer {li}")
            assert_close(got, singles[li], f"multi vs single, layer {li}")   # (split points differ: not the same bits)
    # the same call twice gives the same bits (deterministic reduction)
    again = [torch_to_bits(Y).copy() for Y in Ys]
    moqe.moqe_routed_qgemm_sorted_multi(Xs, perm, offsets, gpus, Ys, ws)
    assert moqe.moqe_async_status() == moqe.OK
    for li in range(len(shapes)):
        assert np.array_equal(torch_to_bits(Ys[li]), again[li])


def test_decode_kernel_refuses_what_it_cannot_take():
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, dev, bf16_to_torch
    W = wl.weights_f32("dq/refuse", 128, 256)
    gpu, _, _ = build_experts(W, [(4, 32, False)])
    X = wl.activations_bf16("dq/refuse/X", 4, 256)
    with pytest.raises(Exception):
        moqe.moqe_routed_qgemm(bf16_to_torch(X), torch.zeros(4, dtype=torch.int32, device=dev()), gpu, path=moqe.PATH_DECODE)


@pytest.mark.parametrize("path", [1, 3, 4, 5])
def test_exact_integer_case_on_gpu(path):
    """On-grid W8 weights with power-of-two scale and small-integer activations: the exact int64 product."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts
    rs = np.random.default_rng(55)
    M, N, K = (16 if path == 5 else 24), 256, 512
    q = rs.integers(-127, 128, size=(N, K))
    q[:, 0], q[:, 1] = 127, -127
    s0 = 2.0 ** -9
    W = (q * s0).astype(np.float32)
    Xi = rs.integers(-8, 9, size=(M, K))
    X = wl.f32_to_bf16_bits(Xi.astype(np.float32))
    gpu, _, _ = build_experts(W, [(8, 0, True)])
    Y, st = _run(X, np.zeros(M, np.int32), gpu, path)
    exact = (Xi.astype(np.int64) @ q.astype(np.int64).T).astype(np.float64) * s0
    assert np.array_equal(Y, wl.f32_to_bf16_bits(exact.astype(np.float32)))


@pytest.mark.parametrize("path", [1, 3, 4, 5])
def test_degenerate_batches(path):
    """All rows to one expert, a shuffled batch, M = 0, ids outside [0, E) -- on every kernel; the decode kernel
    (path 5) takes batches of at most 32 rows."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close, dev, bf16_to_torch
    N, K = 256, 512
    Mb = 32 if path == 5 else 40
    W = wl.weights_f32("deg", N, K)
    specs = [(8, 0, True), (4, 128, False), (3, 128, False)]
    gpu, What, _ = build_experts(W, specs)
    # all rows to one expert == that expert alone (one expert per sample)
    X = wl.activations_bf16("deg/X", Mb, K)
    for e in range(3):
        ids = np.full(Mb, e, np.int32)
        Y, st = _run(X, ids, gpu, path)
        Y1, _ = _run(X, np.zeros(Mb, np.int32), [gpu[e]], path)
        assert st == moqe.OK
        if path == 1:
            # the streaming kernel splits K at points that depend on the set of experts in the call, so the
            # fp32 summation order (not the value within tolerance) may differ between the two calls
            assert_close(Y, Y1, f"expert {e} alone")
        else:
            assert np.array_equal(Y, Y1)
        assert_close(Y, oracle.routed_gemm(X, ids, What), f"single expert {e}")
    # batch shuffle: rows move with their inputs, bit for bit
    rs = np.random.default_rng(3)
    ids = rs.integers(0, 3, size=Mb).astype(np.int32)
    Y, _ = _run(X, ids, gpu, path)
    p = rs.permutation(Mb)
    Yp, _ = _run(X[p], ids[p], gpu, path)
    assert np.array_equal(Yp, Y[p])
    # M = 0
    Y0 = moqe.moqe_routed_qgemm(torch.empty((0, K), dtype=torch.bfloat16, device=dev()),
                                torch.empty(0, dtype=torch.int32, device=dev()), gpu, path=path)
    assert Y0.shape == (0, N)
    # invalid ids: zero rows + latched status, other rows unaffected
    bad = ids.copy()
    bad[[3, Mb - 3]] = [7, -2]
    Yb, st = _run(X, bad, gpu, path)
    assert st == moqe.ERR_EXPERT_ID
    assert np.all(Yb[[3, Mb - 3]] == 0)
    keep = np.setdiff1d(np.arange(Mb), [3, Mb - 3])
    if path in (1, 5):
        # the split-K kernels place their split points by the rows each expert received, so taking two rows
        # out may change the fp32 summation order (not the value within tolerance) of the others
        assert_close(Yb[keep], Y[keep], "rows beside the invalid ones")
    else:
        assert np.array_equal(Yb[keep], Y[keep])
    # a single row, and a whole batch, on one expert of several: the untouched experts must cost nothing and
    # the result must be that expert's
    for Ms in (1, Mb):
        ids1 = np.full(Ms, 2, np.int32)
        Ys, st = _run(X[:Ms], ids1, gpu, path)
        assert st == moqe.OK
        assert_close(Ys, oracle.routed_gemm(X[:Ms], ids1, What), f"{Ms} rows on expert 2")


def test_tcgen05_kernel_full_token_tiles_every_element():
    """The tcgen05 kernel with 256-token tiles (path 4): 1536 rows over three experts -- several full token tiles and a
    ragged one per expert, three channel tiles, eight k-blocks -- every element against the oracle."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close
    M, N, K = 1536, 384, 1024
    W = wl.weights_f32("tc/full", N, K)
    X = wl.activations_bf16("tc/full/X", M, K)
    gpu, What, _ = build_experts(W, [(8, 0, True), (4, 128, False), (3, 128, False)])
    ids = np.repeat(np.array([0, 1, 2, 1, 0, 2], np.int32), [600, 300, 200, 212, 24, 200])
    assert ids.size == M
    for path in (3, 4):
        Y, st = _run(X, ids, gpu, path)
        assert st == moqe.OK
        assert_close(Y, oracle.routed_gemm(X, ids, What), f"path {path}, M{M} N{N} K{K}")


@pytest.mark.parametrize("M,N,K", [(200, 64, 256), (777, 256, 64), (1500, 1000, 1024), (392, 264, 200)])
def test_dense_weights_kernel(M, N, K):
    """The dense-weights GEMM (path 6: large batches on small layers): per-channel, grouped and 32-k-group experts,
    per-image-like runs of rows and scattered rows, ragged tiles, ragged N and K, an idle expert; every element."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close
    specs = [f for f in [(8, 0, True), (4, 0, False), (4, 32, False), (3, 64, False), (8, 128, False), (2, 0, False), (2, 64, False)] if f[1] == 0 or K % f[1] == 0]
    W = wl.weights_f32(f"dn/{N}/{K}", N, K)
    X = wl.activations_bf16(f"dn/{M}/{K}", M, K, relu=True)
    gpu, What, _ = build_experts(W, specs)
    E = len(specs)
    rs = np.random.default_rng(M + N)
    for routing in ("runs", "images", "scattered"):
        if routing == "runs":                                    # whole runs of 64 rows share an expert (read in place)
            ids = np.repeat(rs.integers(0, E, size=(M + 63) // 64), 64)[:M].astype(np.int32)
        elif routing == "images":                                # runs of 196 rows: boxes read in place next to gathered ones
            ids = np.repeat(rs.integers(0, E, size=(M + 195) // 196), 196)[:M].astype(np.int32)
        else:
            ids = rs.integers(0, E, size=M).astype(np.int32)
        ids[ids == 1] = 0                                        # expert 1 idle
        Y, st = _run(X, ids, gpu, moqe.PATH_DENSE)
        assert st == moqe.OK
        assert_close(Y, oracle.routed_gemm(X, ids, What), f"dense {routing} M{M} N{N} K{K}")


def test_argument_errors():
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, dev
    W1 = wl.weights_f32("err1", 128, 256)
    W2 = wl.weights_f32("err2", 256, 256)
    g1, _, _ = build_experts(W1, [(4, 128, False)])
    g2, _, _ = build_experts(W2, [(4, 128, False)])
    X = torch.zeros((8, 256), dtype=torch.bfloat16, device=dev())
    ids = torch.zeros(8, dtype=torch.int32, device=dev())
    with pytest.raises(moqe.MoqeError) as ei:
        moqe.moqe_routed_qgemm(X, ids, [g1[0], g2[0]])
    assert ei.value.code == moqe.ERR_MISMATCH
    with pytest.raises(moqe.MoqeError) as ei:
        moqe.moqe_routed_qgemm(X, ids, g1, workspace=torch.empty(256, dtype=torch.uint8, device=dev()))
    assert ei.value.code == moqe.ERR_WORKSPACE


@pytest.mark.parametrize("path,M", [(1, 16), (1, 48), (3, 300), (5, 16), (5, 9)])
def test_presorted_entry_point_matches(path, M):
    """moqe_permute once + moqe_routed_qgemm_sorted per layer == moqe_routed_qgemm, bit for bit, call after call
    (the split-K arrival counters must come back to zero by themselves)."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, dev, bf16_to_torch, torch_to_bits
    N, K = 384, 2048
    W = wl.weights_f32("sorted", N, K)
    X = wl.activations_bf16(f"sorted/{M}", M, K)
    gpu, What, _ = build_experts(W, [(8, 0, True), (4, 128, False), (3, 128, False)])
    ids = np.random.default_rng(M).integers(0, 3, size=M).astype(np.int32)
    Xd, idd = bf16_to_torch(X), torch.from_numpy(ids).to(dev())
    ref = torch_to_bits(moqe.moqe_routed_qgemm(Xd, idd, gpu, path=path))
    _, perm, offsets = moqe.moqe_permute(None, idd, 3)
    ws = moqe.alloc_workspace(moqe.moqe_routed_qgemm_workspace(M, N, K, 3))
    ws.fill_(0xFF)
    moqe.moqe_routed_qgemm_workspace_clear(ws, M, N, K, 3)
    for _ in range(3):
        Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
        moqe.moqe_routed_qgemm_sorted(Xd, perm, offsets, gpu, Y, ws, path=path)
        assert moqe.moqe_async_status() == moqe.OK
        assert np.array_equal(torch_to_bits(Y), ref)
    from gpu_helpers import assert_close
    assert_close(ref, oracle.routed_gemm(X, ids, What), "sorted")
