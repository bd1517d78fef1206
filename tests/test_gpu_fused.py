"""GPU parity of the two fused steps around the routed product of a decode batch (Section 4.4: whole expert forwards
are what the paper times): the gated pair silu(X.Wg^T) * (X.Wu^T) and the residual add, against the oracle's fp32
versions (rounded once), at the tolerance of the routed product."""
import numpy as np
import pytest
import torch

import oracle
import moqe_workloads as wl

pytestmark = pytest.mark.gpu

FORMATS = [(8, 0, True), (4, 128, False), (3, 128, False), (4, 0, False), (8, 128, False), (3, 256, True)]


def _setup(moqe, M, E, seed):
    from gpu_helpers import dev
    ids = np.random.default_rng(seed).integers(0, E, size=M).astype(np.int32)
    if M > 4:
        ids[ids == 1] = 0                                       # expert 1 idle
    idd = torch.from_numpy(ids).to(dev())
    _, perm, offsets = moqe.moqe_permute(None, idd, E)
    return ids, perm, offsets


@pytest.mark.parametrize("M,N,K", [(1, 128, 128), (7, 200, 640), (16, 384, 2304), (13, 1000, 1280), (9, 128, 16384)])
def test_gated_pair(M, N, K):
    """Whole segments and segments split over many CTAs (the last case: one channel tile, 128 k-blocks), ragged N,
    K not a multiple of 128, every decode format, an idle expert; twice on the same workspace, same bits."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close, dev, bf16_to_torch, torch_to_bits
    specs = [f for f in FORMATS if f[1] == 0 or K % f[1] == 0]
    E = len(specs)
    Wg = wl.weights_f32(f"fused/g/{N}/{K}", N, K, 0.05)
    Wu = wl.weights_f32(f"fused/u/{N}/{K}", N, K, 0.05)
    X = wl.activations_bf16(f"fused/X/{M}/{K}", M, K)
    gg, Whg, _ = build_experts(Wg, specs)
    gu, Whu, _ = build_experts(Wu, specs)
    ids, perm, offsets = _setup(moqe, M, E, M + N)
    ws = moqe.alloc_workspace(moqe.moqe_routed_qgemm_workspace(M, N, K, E))
    moqe.moqe_routed_qgemm_workspace_clear(ws, M, N, K, E)
    ref = oracle.routed_gated_pair(X, ids, Whg, Whu)
    prev = None
    for _ in range(2):
        Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
        moqe.moqe_routed_qgemm_sorted_gated(bf16_to_torch(X), perm, offsets, gg, gu, Y, ws)
        assert moqe.moqe_async_status() == moqe.OK
        got = torch_to_bits(Y)
        assert_close(got, ref, f"gated M{M} N{N} K{K}")
        assert prev is None or np.array_equal(prev, got)
        prev = got
    # the plain product on the same workspace still works afterwards (counters were left at zero)
    Yp = torch.empty((M, N), dtype=torch.bfloat16, device=dev())
    moqe.moqe_routed_qgemm_sorted(bf16_to_torch(X), perm, offsets, gg, Yp, ws, path=moqe.PATH_DECODE)
    assert_close(torch_to_bits(Yp), oracle.routed_gemm(X, ids, Whg), "plain after gated")


@pytest.mark.parametrize("M,N,K", [(5, 200, 640), (16, 512, 4096), (3, 128, 16384)])
def test_residual_add(M, N, K):
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close, dev, bf16_to_torch, torch_to_bits
    specs = [(8, 0, True), (4, 128, False), (3, 128, False)]
    W = wl.weights_f32(f"fused/r/{N}/{K}", N, K)
    X = wl.activations_bf16(f"fused/rX/{M}/{K}", M, K)
    R = wl.activations_bf16(f"fused/R/{M}/{N}", M, N)
    gpu, What, _ = build_experts(W, specs)
    ids, perm, offsets = _setup(moqe, M, 3, 3 * M)
    ws = moqe.alloc_workspace(moqe.moqe_routed_qgemm_workspace(M, N, K, 3))
    moqe.moqe_routed_qgemm_workspace_clear(ws, M, N, K, 3)
    ref = oracle.routed_gemm_residual(X, ids, What, R)
    Y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
    moqe.moqe_routed_qgemm_sorted_residual(bf16_to_torch(X), perm, offsets, gpu, bf16_to_torch(R), Y, ws)
    assert moqe.moqe_async_status() == moqe.OK
    assert_close(torch_to_bits(Y), ref, f"residual M{M} N{N} K{K}")
    # in place: the residual stream is the output
    Yi = bf16_to_torch(R).clone()
    moqe.moqe_routed_qgemm_sorted_residual(bf16_to_torch(X), perm, offsets, gpu, Yi, Yi, ws)
    assert np.array_equal(torch_to_bits(Yi), torch_to_bits(Y))


def test_fused_entry_points_refuse_what_the_decode_kernel_cannot_take():
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, dev, bf16_to_torch
    W = wl.weights_f32("fused/refuse", 128, 256)
    g4, _, _ = build_experts(W, [(4, 128, False)])
    g8, _, _ = build_experts(W, [(8, 0, True)])
    g32, _, _ = build_experts(W, [(4, 32, False)])
    X = bf16_to_torch(wl.activations_bf16("fused/refuse/X", 4, 256))
    idd = torch.zeros(4, dtype=torch.int32, device=dev())
    _, perm, offsets = moqe.moqe_permute(None, idd, 1)
    ws = moqe.alloc_workspace(moqe.moqe_routed_qgemm_workspace(4, 128, 256, 1))
    moqe.moqe_routed_qgemm_workspace_clear(ws, 4, 128, 256, 1)
    Y = torch.empty((4, 128), dtype=torch.bfloat16, device=dev())
    with pytest.raises(moqe.MoqeError) as ei:
        moqe.moqe_routed_qgemm_sorted_gated(X, perm, offsets, g4, g8, Y, ws)       # formats differ
    assert ei.value.code == moqe.ERR_MISMATCH
    with pytest.raises(moqe.MoqeError) as ei:
        moqe.moqe_routed_qgemm_sorted_gated(X, perm, offsets, g32, g32, Y, ws)     # groups of 32 k
    assert ei.value.code == moqe.ERR_UNSUPPORTED
