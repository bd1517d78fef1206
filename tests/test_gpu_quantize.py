"""GPU parity: RTN expert construction, packing, export / import -- bit-exact against the oracle."""
import os

import numpy as np
import pytest
import torch

import oracle
import moqe_workloads as wl

pytestmark = pytest.mark.gpu

CASES = [(8, 0, True), (8, 128, False), (8, 0, False), (4, 128, False), (4, 128, True), (4, 0, False),
         (4, 32, False), (4, 64, True), (3, 128, False), (3, 64, False), (3, 32, True), (3, 0, False), (4, 256, False),
         (2, 128, False), (2, 0, True), (2, 32, False), (2, 64, True)]


@pytest.mark.parametrize("bits,group,sym", CASES)
@pytest.mark.parametrize("N,K", [(1024, 1024), (200, 768), (64, 256), (8, 64)])
def test_quantize_matches_oracle(bits, group, sym, N, K):
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_expert_matches
    if group and K % group:
        pytest.skip("group does not divide K")
    W = wl.weights_f32(f"gq/{N}/{K}", N, K)
    W[1, : min(K, 64)] = 0.0                       # degenerate pieces
    if N > 5:
        W[5] = np.abs(W[5]) + 1e-3                 # all-positive row
    gpu, _, canon = build_experts(W, [(bits, group, sym)])
    assert_expert_matches(gpu[0], canon[0])
    e = gpu[0]
    assert (e.N, e.K, e.bits, e.group, e.sym) == (N, K, bits, group, bool(sym))
    assert e.code_bytes == N * K * bits // 8
    G = 1 if group == 0 else K // group
    assert e.meta_bytes == N * G * 2 * (1 if sym else 2)
    # export -> import -> export is the identity (packing round trip through another expert)
    c, s, z = moqe.moqe_expert_export(e)
    e2 = moqe.moqe_expert_import(bits, group, sym, c, s, z)
    assert_expert_matches(e2, canon[0])
    assert moqe.moqe_async_status() == moqe.OK


def test_closed_form_grid_on_gpu():
    """The same closed-form pin as for the oracle: an on-grid W must come back as its own grid."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev, torch_to_bits
    rs = np.random.default_rng(11)
    N, K, g, bits = 256, 512, 128, 4
    L = 15
    s0 = 2.0 ** rs.integers(-12, -3, size=(N, K // g))
    z0 = rs.integers(0, L + 1, size=(N, K // g))
    c0 = rs.integers(0, L + 1, size=(N, K // g, g))
    c0[:, :, 0], c0[:, :, 1] = 0, L
    W = (s0[:, :, None] * (c0 - z0[:, :, None])).reshape(N, K).astype(np.float32)
    e = moqe.moqe_quantize_rtn(torch.from_numpy(W).to(dev()), bits, g, False)
    c, s, z = moqe.moqe_expert_export(e)
    assert np.array_equal(c.cpu().numpy(), c0.reshape(N, K).astype(np.uint8))
    assert np.array_equal(s.float().cpu().numpy(), s0.astype(np.float32))
    assert np.array_equal(z.float().cpu().numpy(), z0.astype(np.float32))


def test_storage_ratios_match_the_papers_table():
    """Packed code bytes per weight are b/8: FP16 : Int8 : Int4 = 1 : 1/2 : 1/4 (paper, appendix table)."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev
    path = os.path.join(os.path.dirname(__file__), "golden", "storage_ratios.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    W = torch.from_numpy(wl.weights_f32("ratios", 256, 512)).to(dev())
    fp16_bytes = 256 * 512 * 2
    e8 = moqe.moqe_quantize_rtn(W, 8, 0, True)
    e4 = moqe.moqe_quantize_rtn(W, 4, 0, True)
    for name, fp16, int8, int4, unit in rows:
        assert abs(float(int8) / float(fp16) - e8.code_bytes / fp16_bytes) < 0.02
        assert abs(float(int4) / float(fp16) - e4.code_bytes / fp16_bytes) < 0.02
    # what is really allocated (and what a parked expert's image holds): codes + scales / zero-points, nothing else when
    # N and K are multiples of 128 -- for every format, true 3.0 bits per weight included
    for bits, group, sym in [(8, 0, True), (4, 0, True), (4, 128, False), (3, 128, False), (3, 0, False), (4, 32, False), (8, 128, True), (2, 128, False), (2, 0, True)]:
        e = moqe.moqe_quantize_rtn(W, bits, group, sym)
        assert e.code_bytes == 256 * 512 * bits // 8
        assert e.meta_bytes == 256 * (1 if group == 0 else 512 // group) * 2 * (1 if sym else 2)
        assert e.alloc_bytes == e.code_bytes + e.meta_bytes, (bits, group, sym)
        assert moqe.moqe_expert_offload(e).image_bytes == e.alloc_bytes
    # ragged shapes are padded to whole 128 x 128 tiles: the padding is accounted for exactly
    W2 = torch.from_numpy(wl.weights_f32("ratios2", 200, 320)).to(dev())
    e = moqe.moqe_quantize_rtn(W2, 4, 64, False)
    assert e.alloc_bytes == 256 * 384 * 4 // 8 + 256 * (384 // 64) * 2 * 2


def test_argument_errors():
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev
    W = torch.zeros((16, 64), dtype=torch.float32, device=dev())
    for bits, group, code in [(5, 0, moqe.ERR_UNSUPPORTED), (4, 48, moqe.ERR_SHAPE), (4, 96, moqe.ERR_SHAPE)]:
        with pytest.raises(moqe.MoqeError) as ei:
            moqe.moqe_quantize_rtn(W, bits, group, False)
        assert ei.value.code == code
    W2 = torch.zeros((16, 60), dtype=torch.float32, device=dev())
    with pytest.raises(moqe.MoqeError) as ei:
        moqe.moqe_quantize_rtn(W2, 4, 0, False)
    assert ei.value.code == moqe.ERR_UNSUPPORTED
