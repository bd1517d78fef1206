"""Expert residency (Section 4.4 / appendix "Router model and expert loading overhead": experts parked in CPU RAM or on
disk and loaded when the routing changes): a packed expert must survive device -> pinned host -> file -> pinned host ->
device bit for bit, whatever its format, and a prefetch on a side stream must be usable by the next routed call."""
import os

import numpy as np
import pytest
import torch

import oracle
import moqe_workloads as wl

pytestmark = pytest.mark.gpu

FORMATS = [(8, 0, True), (4, 128, False), (3, 128, False), (4, 0, False), (3, 64, False), (4, 32, False), (8, 128, False)]


def _same_expert(moqe, a, b):
    ca, sa, za = moqe.moqe_expert_export(a)
    cb, sb, zb = moqe.moqe_expert_export(b)
    return torch.equal(ca, cb) and torch.equal(sa.view(torch.int16), sb.view(torch.int16)) and \
        torch.equal(za.view(torch.int16), zb.view(torch.int16))


@pytest.mark.parametrize("bits,group,sym", FORMATS)
def test_round_trip_through_host_memory_and_a_file(tmp_path, bits, group, sym):
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev
    N, K = 200, 384                                            # ragged N: padded channels travel too
    W = torch.from_numpy(wl.weights_f32(f"res/{bits}/{group}", N, K)).to(dev())
    e = moqe.moqe_quantize_rtn(W, bits, group, sym)
    h = moqe.moqe_expert_offload(e)
    assert (h.N, h.K, h.bits, h.group, h.sym) == (N, K, bits, group, sym)
    assert h.image_bytes == e.alloc_bytes
    path = str(tmp_path / "expert.moqe")
    moqe.moqe_expert_host_save(h, path)
    assert os.path.getsize(path) == h.image_bytes + 48
    h2 = moqe.moqe_expert_host_load(path)
    e2 = moqe.moqe_expert_prefetch(h2)
    torch.cuda.synchronize()
    assert _same_expert(moqe, e, e2)


def test_prefetch_on_a_side_stream_while_a_layer_runs():
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close, dev, bf16_to_torch, torch_to_bits
    N, K, M = 512, 1024, 12
    W = wl.weights_f32("res/side", N, K)
    X = wl.activations_bf16("res/side/X", M, K)
    gpu, What, _ = build_experts(W, [(8, 0, True), (4, 128, False), (3, 128, False)])
    ids = np.array([0, 1, 2] * 4, np.int32)
    parked = moqe.moqe_expert_offload(gpu[2])                  # expert 2 leaves the GPU ...
    gpu[2].close()
    Xd, idd = bf16_to_torch(X), torch.from_numpy(ids).to(dev())
    side = torch.cuda.Stream()
    back = moqe.moqe_expert_prefetch(parked, stream=side)      # ... and comes back on a side stream
    ready = torch.cuda.Event()
    ready.record(side)
    Y01 = moqe.moqe_routed_qgemm(Xd[ids != 2].contiguous(), idd[idd != 2].contiguous(), gpu[:2])   # meanwhile: the other two
    torch.cuda.current_stream().wait_event(ready)
    Y = moqe.moqe_routed_qgemm(Xd, idd, [gpu[0], gpu[1], back])
    assert moqe.moqe_async_status() == moqe.OK
    ref = oracle.routed_gemm(X, ids, What)
    assert_close(torch_to_bits(Y), ref, "after the prefetch")
    assert_close(torch_to_bits(Y01), ref[ids != 2], "during the prefetch")


def test_bad_files_are_refused(tmp_path):
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev
    W = torch.from_numpy(wl.weights_f32("res/bad", 128, 256)).to(dev())
    h = moqe.moqe_expert_offload(moqe.moqe_quantize_rtn(W, 4, 128, False))
    path = str(tmp_path / "e.moqe")
    moqe.moqe_expert_host_save(h, path)
    data = open(path, "rb").read()
    cases = {"missing": None, "truncated": data[:-16], "too long": data + b"\0" * 8, "bad magic": b"X" + data[1:],
             "unknown layout": data[:8] + (99).to_bytes(4, "little") + data[12:],
             "bits 5": data[:20] + (5).to_bytes(4, "little") + data[24:], "header only": data[:20]}
    for name, blob in cases.items():
        p = str(tmp_path / (name.replace(" ", "_") + ".moqe"))
        if blob is not None:
            open(p, "wb").write(blob)
        with pytest.raises(moqe.MoqeError) as ei:
            moqe.moqe_expert_host_load(p)
        assert ei.value.code in (moqe.ERR_IO, moqe.ERR_UNSUPPORTED, moqe.ERR_SHAPE), name
    with pytest.raises(moqe.MoqeError):
        moqe.moqe_expert_host_save(h, str(tmp_path / "no_such_dir" / "e.moqe"))
