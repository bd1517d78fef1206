"""GPU parity of the router front end (Section 3.2) and the load report (Section 3.3) against the fp64 oracle.

The device computes in fp32, the oracle in fp64: logits are compared at 1e-4 * (1 + |logit|) -- a dot product of a few
thousand fp32 terms of size ~1 carries ~1e-6 relative error, the bound leaves two orders of margin -- and the expert id
must equal the oracle's wherever the oracle's top-2 margin exceeds twice that bound (elsewhere either of the two is a
correct arg-max of a value known only to the tolerance).  Counts follow the ids exactly."""
import numpy as np
import pytest
import torch

import oracle
import moqe_workloads as wl

pytestmark = pytest.mark.gpu

TOL = 1e-4


def _check(logits_gpu, ids_gpu, logits_ref):
    bound = TOL * (1.0 + np.abs(logits_ref))
    assert np.all(np.abs(logits_gpu.astype(np.float64) - logits_ref) <= bound)
    ids_ref = oracle.route(logits_ref.astype(np.float32))
    srt = np.sort(logits_ref, axis=1)
    margin = srt[:, -1] - srt[:, -2] if logits_ref.shape[1] > 1 else np.full(len(srt), np.inf)
    clear = margin > 2 * bound.max(axis=1)
    assert np.array_equal(ids_gpu[clear], ids_ref[clear])
    for s in np.nonzero(~clear)[0]:                            # a near-tie: any expert whose score is within the bound of the best
        assert logits_ref[s, ids_gpu[s]] >= srt[s, -1] - 2 * bound[s].max()
    # the device's ids are the first-max arg-max of the device's own logits, bit for bit
    assert np.array_equal(ids_gpu, oracle.route(logits_gpu))
    return ids_ref


@pytest.mark.parametrize("S_rows,H,D,E", [((1, 3, 0, 17, 1), 64, 16, 3), ((5,) * 9, 520, 40, 5), ((300, 1, 1, 2), 1024, 256, 2)])
def test_router_front_end_small(S_rows, H, D, E):
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev, bf16_to_torch
    off = np.zeros(len(S_rows) + 1, np.int32)
    off[1:] = np.cumsum(S_rows)
    X = wl.activations_bf16(f"router/{H}/{D}", int(off[-1]), H)
    W1 = wl.normal_f32(f"router/w1/{H}/{D}", (D, H), 1.0 / np.sqrt(H))
    W2 = wl.normal_f32(f"router/w2/{D}/{E}", (E, D), 1.0 / np.sqrt(D))
    ref, _ = oracle.router_mlp(X, off, W1, W2)
    lg, ids = moqe.moqe_router_mlp(bf16_to_torch(X), torch.from_numpy(off).to(dev()), torch.from_numpy(W1).to(dev()),
                                   torch.from_numpy(W2).to(dev()))
    assert moqe.moqe_async_status() == moqe.OK
    ids_h = ids.cpu().numpy()
    _check(lg.cpu().numpy(), ids_h, ref)
    # load report on the device's own logits and ids
    P, F, L, counts = moqe.moqe_router_load_report(lg, ids)
    Pr, Fr, Lr = oracle.load_report(lg.cpu().numpy().astype(np.float64), ids_h)
    assert np.allclose(P.cpu().numpy(), Pr, atol=1e-5) and np.array_equal(F.cpu().numpy(), Fr.astype(np.float32))
    assert abs(float(L) - Lr) <= 1e-5 * max(1.0, Lr)
    assert np.array_equal(counts.cpu().numpy(), np.bincount(ids_h, minlength=E))
    # same call, same bits
    lg2, ids2 = moqe.moqe_router_mlp(bf16_to_torch(X), torch.from_numpy(off).to(dev()), torch.from_numpy(W1).to(dev()),
                                     torch.from_numpy(W2).to(dev()))
    assert torch.equal(lg, lg2) and torch.equal(ids, ids2)


def test_router_of_the_mixed_workload_at_full_size():
    """qwen7b_mixed: 64 one-token sequences + 4 sequences of 1024 tokens, hidden 3584 -> 256 -> 4 experts."""
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev, bf16_to_torch
    w = wl.get("qwen7b_mixed")
    layer = w.layers[0]
    off = w.row_offsets(layer)
    X = wl.activations_bf16(f"{w.name}/{layer.name}/X", w.M_of(layer), layer.K, w.relu_inputs)
    H, E = layer.K, w.n_experts
    W1, W2 = wl.router_weights(w)
    ref, _ = oracle.router_mlp(X, off, W1, W2)
    lg, ids = moqe.moqe_router_mlp(bf16_to_torch(X), torch.from_numpy(off).to(dev()), torch.from_numpy(W1).to(dev()),
                                   torch.from_numpy(W2).to(dev()))
    assert moqe.moqe_async_status() == moqe.OK
    _check(lg.cpu().numpy(), ids.cpu().numpy(), ref)


def test_router_argument_errors():
    import paper_2508_09204_b200 as moqe
    from gpu_helpers import dev
    L = moqe.lib()
    t = torch.zeros(4096, dtype=torch.float32, device=dev())
    p = t.data_ptr()
    assert L.moqe_router_mlp(p, p, 2, 12, p, 4, p, 2, p, p, p, 1 << 20, None) == moqe.ERR_UNSUPPORTED     # H % 8
    assert L.moqe_router_mlp(p, p, 2, 16, p, 4, p, 2, p, p, p, 16, None) == moqe.ERR_WORKSPACE
    assert L.moqe_router_mlp(None, p, 2, 16, p, 4, p, 2, p, p, p, 1 << 20, None) == moqe.ERR_NULL
    assert L.moqe_router_mlp(p, p, 2, 16, p, 4, p, 99, p, p, p, 1 << 20, None) == moqe.ERR_UNSUPPORTED    # too many experts
    assert L.moqe_router_load_report(p, p, 0, 2, p, None, None) == moqe.ERR_SHAPE
