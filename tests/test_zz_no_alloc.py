"""moqe_permute_static -- the sort/gather entry point for callers that cannot allocate device memory
(plug-ins inside a process whose memory pool belongs to the host framework, real-time loops that may
not take the allocator's lock) -- must give exactly what moqe_permute gives.  Collected last on purpose.

It is called straight through the C ABI with caller-owned buffers, twice in a row with different
batches, because all calls share one built-in scratch array that still holds the previous call's data.
"""
import ctypes as C

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _call_static(moqe, X, ids, E, Xp, perm, offsets):
    L = moqe.lib()
    stream = torch.cuda.current_stream().cuda_stream
    p = lambda t: None if t is None else C.c_void_p(t.data_ptr())
    Cc = 0 if X is None else X.shape[1]
    return L.moqe_permute_static(p(X), p(ids), ids.numel(), Cc, E, p(Xp), p(perm), p(offsets), stream)


def test_static_permute_matches_permute_twice_in_a_row():
    import paper_2508_09204_b200 as moqe
    dev = torch.device("cuda", 0)
    g = np.random.default_rng(2024)
    # two different batches back to back: a large one that fills the scratch, then a smaller one with
    # another expert count that must not be disturbed by what the first call left behind
    first = True
    for M, Cc, E in [(70001, 64, 5), (5000, 16, 3), (600, 8, 2), (moqe.PERMUTE_STATIC_MAX_ROWS, 8, 4)]:
        ids_h = g.integers(0, E, size=M).astype(np.int32)
        if E >= 3:
            ids_h[ids_h == 1] = 0
        ids = torch.from_numpy(ids_h).to(dev)
        X = torch.from_numpy(g.integers(0, 65536, size=(M, Cc)).astype(np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
        Xp_ref, perm_ref, off_ref = moqe.moqe_permute(X, ids, E)
        # outputs are allocated here, by the caller, before the call; the call itself allocates nothing
        Xp = torch.empty_like(X)
        perm = torch.full((M,), -7, dtype=torch.int32, device=dev)
        offsets = torch.full((E + 1,), -7, dtype=torch.int32, device=dev)
        if first:
            # the first call on a device looks up the address of the built-in scratch array (no allocation, but
            # it may load the module's data); the measurement below starts after it
            assert _call_static(moqe, X, ids, E, Xp, perm, offsets) == moqe.OK
            first = False
        torch.cuda.synchronize()
        before, before_free = torch.cuda.memory_allocated(dev), torch.cuda.mem_get_info(dev)[0]
        assert _call_static(moqe, X, ids, E, Xp, perm, offsets) == moqe.OK
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated(dev) == before          # nothing from torch's allocator
        assert torch.cuda.mem_get_info(dev)[0] == before_free      # and nothing from the driver either
        assert torch.equal(perm, perm_ref)
        assert torch.equal(offsets, off_ref)
        assert torch.equal(Xp.view(torch.int16), Xp_ref.view(torch.int16))
    # ids outside [0, E): sorted behind the valid rows exactly as moqe_permute does, but no status is latched
    M, Cc, E = 3000, 8, 3
    ids_h = g.integers(0, E, size=M).astype(np.int32)
    ids_h[[5, 77, 2999]] = [E, -1, 1000]
    ids = torch.from_numpy(ids_h).to(dev)
    X = torch.from_numpy(g.integers(0, 65536, size=(M, Cc)).astype(np.uint16).view(np.int16)).to(dev).view(torch.bfloat16)
    Xp_ref, perm_ref, off_ref = moqe.moqe_permute(X, ids, E)
    assert moqe.moqe_async_status() == moqe.ERR_EXPERT_ID           # (the allocating entry point latches it; now cleared)
    Xp = torch.empty_like(X)
    perm = torch.full((M,), -7, dtype=torch.int32, device=dev)
    offsets = torch.full((E + 1,), -7, dtype=torch.int32, device=dev)
    assert _call_static(moqe, X, ids, E, Xp, perm, offsets) == moqe.OK
    assert moqe.moqe_async_status() == moqe.OK
    assert int(offsets[E]) == M - 3
    assert torch.equal(perm, perm_ref) and torch.equal(offsets, off_ref)
    assert torch.equal(Xp.view(torch.int16), Xp_ref.view(torch.int16))
    # indices only, and the size limit
    ids = torch.zeros(2000, dtype=torch.int32, device=dev)
    perm = torch.empty(2000, dtype=torch.int32, device=dev)
    offsets = torch.empty(2, dtype=torch.int32, device=dev)
    assert _call_static(moqe, None, ids, 1, None, perm, offsets) == moqe.OK
    assert torch.equal(perm, torch.arange(2000, dtype=torch.int32, device=dev))
    assert offsets.tolist() == [0, 2000]
    L = moqe.lib()
    too_many = moqe.PERMUTE_STATIC_MAX_ROWS + 1
    fake = C.c_void_p(0x1000)                                   # rejected on the host before any use
    assert L.moqe_permute_static(None, fake, too_many, 0, 2, None, fake, fake, None) == moqe.ERR_WORKSPACE
