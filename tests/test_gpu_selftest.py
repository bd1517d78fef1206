"""The bounded waits of the kernels, made to run out on purpose: one small kernel waits on an mbarrier nobody arrives
on, with a one-millisecond limit.  It must return by itself, report MOQE_ERR_TIMEOUT through the device status word,
and leave the context usable -- nothing traps, nothing hangs."""
import numpy as np
import pytest
import torch

import oracle
import moqe_workloads as wl

pytestmark = pytest.mark.gpu


def test_a_wait_that_nobody_ends_gives_up_and_the_next_call_works():
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import build_experts, assert_close, dev, bf16_to_torch, torch_to_bits
    assert moqe.moqe_async_status() == moqe.OK
    out = moqe.moqe_selftest_timeout(1000)
    assert moqe.moqe_async_status() == moqe.ERR_TIMEOUT           # (synchronises; reads and clears the status word)
    assert int(out.item()) == 2                                   # the wait returned false by itself
    assert moqe.moqe_async_status() == moqe.OK                    # cleared
    # an ordinary call right after it
    W = wl.weights_f32("selftest/W", 256, 512)
    X = wl.activations_bf16("selftest/X", 12, 512)
    gpu, What, _ = build_experts(W, [(8, 0, True), (4, 128, False)])
    ids = np.array([0, 1] * 6, np.int32)
    Y = moqe.moqe_routed_qgemm(bf16_to_torch(X), torch.from_numpy(ids).to(dev()), gpu)
    assert moqe.moqe_async_status() == moqe.OK
    assert_close(torch_to_bits(Y), oracle.routed_gemm(X, ids, What), "after the self-test")
    # argument errors are found on the host
    L = moqe.lib()
    assert L.moqe_selftest_timeout(0, out.data_ptr(), None) == moqe.ERR_SHAPE
    assert L.moqe_selftest_timeout(1000, None, None) == moqe.ERR_NULL
