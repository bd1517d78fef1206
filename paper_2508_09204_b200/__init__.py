"""Python binding of ``libmoqe.so`` (the routed quantized-linear library for B200).

Argument marshalling only: every function takes torch CUDA tensors, passes
their device pointers and the current CUDA stream to the C-ABI call of the
same name (``include/moqe.h``), and returns torch tensors.  No arithmetic of
the method happens in Python, and there is no CPU fallback: if the shared
library is missing, loading fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmoqe.so")

OK = 0
ERR_NULL, ERR_SHAPE, ERR_UNSUPPORTED, ERR_ALLOC, ERR_WORKSPACE, ERR_MISMATCH, ERR_CUDA, ERR_EXPERT_ID, ERR_TIMEOUT, ERR_IO = range(1, 11)
MAX_EXPERTS = 32
PATH_AUTO, PATH_STREAM, PATH_TCGEN05, PATH_DECODE, PATH_DENSE = 0, 1, 2, 5, 6

EXPORTED = (
    "moqe_quantize_rtn", "moqe_expert_export", "moqe_expert_import", "moqe_expert_info", "moqe_expert_destroy",
    "moqe_route", "moqe_expand_ids", "moqe_route_permute", "moqe_permute_workspace", "moqe_permute", "moqe_permute_static", "moqe_unpermute",
    "moqe_routed_qgemm_workspace", "moqe_routed_qgemm", "moqe_routed_qgemm_path", "moqe_routed_qgemm_sorted",
    "moqe_routed_qgemm_sorted_multi", "moqe_routed_qgemm_workspace_clear", "moqe_async_status",
    "moqe_status_str", "moqe_launch_count", "moqe_tune", "moqe_selftest_timeout",
    "moqe_router_mlp_workspace", "moqe_router_mlp", "moqe_router_load_report",
    "moqe_routed_qgemm_sorted_gated", "moqe_routed_qgemm_sorted_residual",
    "moqe_expert_offload", "moqe_expert_prefetch", "moqe_expert_host_info", "moqe_expert_host_save", "moqe_expert_host_load",
    "moqe_expert_host_destroy",
)


class MoqeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_str(code)} (moqe_status {code})")


_lib = None


def lib() -> C.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2508_09204_b200.build` "
                "(there is no fallback implementation)")
        L = C.CDLL(LIB_PATH)
        vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
        L.moqe_quantize_rtn.argtypes = [vp, i32, i32, i32, i32, i32, vp, C.POINTER(vp)]
        L.moqe_expert_export.argtypes = [vp, vp, vp, vp, vp]
        L.moqe_expert_import.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, vp, C.POINTER(vp)]
        L.moqe_expert_info.argtypes = [vp] + [C.POINTER(i32)] * 5 + [C.POINTER(sz)] * 3
        L.moqe_expert_destroy.argtypes = [vp]
        L.moqe_route.argtypes = [vp, i32, i32, vp, vp]
        L.moqe_expand_ids.argtypes = [vp, vp, i32, i32, vp, vp]
        L.moqe_route_permute.argtypes = [vp, i32, i32, vp, i32, vp, vp, vp, vp, vp]
        L.moqe_permute_workspace.argtypes = [i32, i32]
        L.moqe_permute_workspace.restype = sz
        L.moqe_permute.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp, sz, vp]
        L.moqe_permute_static.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp]
        L.moqe_unpermute.argtypes = [vp, vp, i32, i32, vp, vp]
        L.moqe_routed_qgemm_workspace.argtypes = [i32, i32, i32, i32]
        L.moqe_routed_qgemm_workspace.restype = sz
        L.moqe_routed_qgemm.argtypes = [vp, vp, i32, C.POINTER(vp), i32, vp, vp, sz, vp]
        L.moqe_routed_qgemm_path.argtypes = [vp, vp, i32, C.POINTER(vp), i32, vp, vp, sz, vp, i32]
        L.moqe_routed_qgemm_sorted.argtypes = [vp, vp, vp, i32, C.POINTER(vp), i32, vp, vp, sz, vp, i32]
        L.moqe_routed_qgemm_sorted_multi.argtypes = [C.POINTER(vp), vp, vp, i32, i32, C.POINTER(vp), i32, C.POINTER(vp), vp, sz, vp]
        L.moqe_routed_qgemm_sorted_gated.argtypes = [vp, vp, vp, i32, C.POINTER(vp), C.POINTER(vp), i32, vp, vp, sz, vp]
        L.moqe_routed_qgemm_sorted_residual.argtypes = [vp, vp, vp, i32, C.POINTER(vp), i32, vp, vp, vp, sz, vp]
        L.moqe_routed_qgemm_workspace_clear.argtypes = [vp, sz, i32, i32, i32, i32, vp]
        L.moqe_async_status.argtypes = [vp]
        L.moqe_status_str.argtypes = [i32]
        L.moqe_status_str.restype = C.c_char_p
        L.moqe_tune.argtypes = [C.c_char_p, i32]
        L.moqe_selftest_timeout.argtypes = [C.c_uint, vp, vp]
        L.moqe_expert_offload.argtypes = [vp, vp, C.POINTER(vp)]
        L.moqe_expert_prefetch.argtypes = [vp, vp, C.POINTER(vp)]
        L.moqe_expert_host_info.argtypes = [vp] + [C.POINTER(i32)] * 5 + [C.POINTER(sz)]
        L.moqe_expert_host_save.argtypes = [vp, C.c_char_p]
        L.moqe_expert_host_load.argtypes = [C.c_char_p, C.POINTER(vp)]
        L.moqe_expert_host_destroy.argtypes = [vp]
        L.moqe_router_mlp_workspace.argtypes = [i32, i32, i32]
        L.moqe_router_mlp_workspace.restype = sz
        L.moqe_router_mlp.argtypes = [vp, vp, i32, i32, vp, i32, vp, i32, vp, vp, vp, sz, vp]
        L.moqe_router_load_report.argtypes = [vp, vp, i32, i32, vp, vp, vp]
        L.moqe_launch_count.argtypes = []
        L.moqe_launch_count.restype = C.c_ulonglong
        _lib = L
    return _lib


def status_str(code: int) -> str:
    return lib().moqe_status_str(int(code)).decode()


def _check(code: int, where: str):
    if code != OK:
        raise MoqeError(code, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}")
    return t.contiguous()


class Expert:
    """Owner of one ``moqe_expert*`` (destroyed with the Python object)."""

    def __init__(self, handle: int):
        self.handle = C.c_void_p(handle)
        N, K, bits, group, sym = (C.c_int() for _ in range(5))
        cb, mb, ab = (C.c_size_t() for _ in range(3))
        _check(lib().moqe_expert_info(self.handle, N, K, bits, group, sym, cb, mb, ab), "moqe_expert_info")
        self.N, self.K, self.bits, self.group, self.sym = N.value, K.value, bits.value, group.value, bool(sym.value)
        self.code_bytes, self.meta_bytes, self.alloc_bytes = cb.value, mb.value, ab.value

    @property
    def groups_per_row(self) -> int:
        return 1 if self.group == 0 else self.K // self.group

    def close(self):
        if self.handle is not None and self.handle.value:
            lib().moqe_expert_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class HostExpert:
    """Owner of one ``moqe_expert_host*``: a packed expert parked in pinned host memory."""

    def __init__(self, handle: int):
        self.handle = C.c_void_p(handle)
        N, K, bits, group, sym = (C.c_int() for _ in range(5))
        nb = C.c_size_t()
        _check(lib().moqe_expert_host_info(self.handle, N, K, bits, group, sym, nb), "moqe_expert_host_info")
        self.N, self.K, self.bits, self.group, self.sym = N.value, K.value, bits.value, group.value, bool(sym.value)
        self.image_bytes = nb.value

    def close(self):
        if self.handle is not None and self.handle.value:
            lib().moqe_expert_host_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def moqe_expert_offload(e: Expert) -> HostExpert:
    out = C.c_void_p()
    _check(lib().moqe_expert_offload(e.handle, _stream(), C.byref(out)), "moqe_expert_offload")
    return HostExpert(out.value)


def moqe_expert_prefetch(h: HostExpert, stream: Optional[torch.cuda.Stream] = None) -> Expert:
    """Enqueues the host-to-device copies on ``stream`` (default: the current one) and returns the new expert."""
    out = C.c_void_p()
    st = C.c_void_p(stream.cuda_stream) if stream is not None else _stream()
    _check(lib().moqe_expert_prefetch(h.handle, st, C.byref(out)), "moqe_expert_prefetch")
    return Expert(out.value)


def moqe_expert_host_save(h: HostExpert, path: str) -> None:
    _check(lib().moqe_expert_host_save(h.handle, os.fsencode(path)), "moqe_expert_host_save")


def moqe_expert_host_load(path: str) -> HostExpert:
    out = C.c_void_p()
    _check(lib().moqe_expert_host_load(os.fsencode(path), C.byref(out)), "moqe_expert_host_load")
    return HostExpert(out.value)


def moqe_quantize_rtn(W: torch.Tensor, bits: int, group: int, sym: bool) -> Expert:
    """RTN-quantize the fp32 device matrix ``W[N][K]`` into a packed expert."""
    W = _dev(W, torch.float32, "W")
    N, K = W.shape
    out = C.c_void_p()
    _check(lib().moqe_quantize_rtn(_ptr(W), N, K, int(bits), int(group), int(bool(sym)), _stream(), C.byref(out)),
           "moqe_quantize_rtn")
    return Expert(out.value)


def moqe_expert_export(e: Expert) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """-> (codes uint8 [N][K], scales fp16 [N][K/g], zeros fp16 [N][K/g])."""
    dev = torch.device("cuda", torch.cuda.current_device())
    codes = torch.empty((e.N, e.K), dtype=torch.uint8, device=dev)
    scales = torch.empty((e.N, e.groups_per_row), dtype=torch.float16, device=dev)
    zeros = torch.empty((e.N, e.groups_per_row), dtype=torch.float16, device=dev)
    _check(lib().moqe_expert_export(e.handle, _ptr(codes), _ptr(scales), _ptr(zeros), _stream()), "moqe_expert_export")
    return codes, scales, zeros


def moqe_expert_import(bits: int, group: int, sym: bool, codes: torch.Tensor, scales: torch.Tensor,
                       zeros: Optional[torch.Tensor]) -> Expert:
    codes = _dev(codes, torch.uint8, "codes")
    scales = _dev(scales, torch.float16, "scales")
    zeros = None if zeros is None else _dev(zeros, torch.float16, "zeros")
    N, K = codes.shape
    out = C.c_void_p()
    _check(lib().moqe_expert_import(N, K, int(bits), int(group), int(bool(sym)), _ptr(codes), _ptr(scales), _ptr(zeros),
                                    _stream(), C.byref(out)), "moqe_expert_import")
    return Expert(out.value)


def moqe_route(logits: torch.Tensor) -> torch.Tensor:
    """First-max arg-max over each row of fp32 ``logits[S][E]`` -> int32 ids."""
    logits = _dev(logits, torch.float32, "logits")
    S, E = logits.shape
    ids = torch.empty(S, dtype=torch.int32, device=logits.device)
    _check(lib().moqe_route(_ptr(logits), S, E, _ptr(ids), _stream()), "moqe_route")
    return ids


def moqe_expand_ids(ids: torch.Tensor, row_offsets: torch.Tensor, M: int) -> torch.Tensor:
    ids = _dev(ids, torch.int32, "ids")
    row_offsets = _dev(row_offsets, torch.int32, "row_offsets")
    row_ids = torch.empty(M, dtype=torch.int32, device=ids.device)
    _check(lib().moqe_expand_ids(_ptr(ids), _ptr(row_offsets), ids.numel(), int(M), _ptr(row_ids), _stream()),
           "moqe_expand_ids")
    return row_ids


def moqe_route_permute(logits: torch.Tensor, row_offsets: Optional[torch.Tensor], M: int):
    """moqe_route + moqe_expand_ids + moqe_permute (indices only) in one launch, for at most 1024 samples and rows.
    -> (ids int32 [S], row_ids int32 [M], perm int32 [M], offsets int32 [E+1])."""
    logits = _dev(logits, torch.float32, "logits")
    S, E = logits.shape
    dev = logits.device
    if row_offsets is not None:
        row_offsets = _dev(row_offsets, torch.int32, "row_offsets")
    ids = torch.empty(S, dtype=torch.int32, device=dev)
    row_ids = torch.empty(int(M), dtype=torch.int32, device=dev)
    perm = torch.empty(int(M), dtype=torch.int32, device=dev)
    offsets = torch.empty(E + 1, dtype=torch.int32, device=dev)
    _check(lib().moqe_route_permute(_ptr(logits), S, E, _ptr(row_offsets) if row_offsets is not None else None, int(M),
                                    _ptr(ids), _ptr(row_ids), _ptr(perm), _ptr(offsets), _stream()), "moqe_route_permute")
    return ids, row_ids, perm, offsets


def moqe_permute(X: Optional[torch.Tensor], row_ids: torch.Tensor, E: int):
    """-> (Xp or None, perm int32 [M], offsets int32 [E+1])."""
    row_ids = _dev(row_ids, torch.int32, "row_ids")
    M = row_ids.numel()
    dev = row_ids.device
    Cc = 0
    Xp = None
    if X is not None:
        X = _dev(X, torch.bfloat16, "X")
        Cc = X.shape[1]
        Xp = torch.empty_like(X)
    perm = torch.empty(M, dtype=torch.int32, device=dev)
    offsets = torch.empty(E + 1, dtype=torch.int32, device=dev)
    wsb = lib().moqe_permute_workspace(M, E)
    ws = torch.empty(max(wsb, 1), dtype=torch.uint8, device=dev)
    _check(lib().moqe_permute(_ptr(X), _ptr(row_ids), M, Cc, int(E), _ptr(Xp), _ptr(perm), _ptr(offsets), _ptr(ws), wsb,
                              _stream()), "moqe_permute")
    return Xp, perm, offsets


PERMUTE_STATIC_MAX_ROWS = 1 << 20


def moqe_permute_static(X: Optional[torch.Tensor], row_ids: torch.Tensor, E: int, Xp: Optional[torch.Tensor],
                        perm: torch.Tensor, offsets: torch.Tensor) -> None:
    """``moqe_permute`` without a workspace, for callers that must not allocate device memory.

    Every buffer, outputs included, is passed in by the caller; the C call keeps its scratch in a
    fixed array inside the library and allocates nothing.  Calls on one device must not overlap.
    """
    M = row_ids.numel()
    Cc = 0 if X is None else X.shape[1]
    _check(lib().moqe_permute_static(_ptr(X), _ptr(row_ids), M, Cc, int(E), _ptr(Xp), _ptr(perm), _ptr(offsets),
                                     _stream()), "moqe_permute_static")


def moqe_unpermute(Yp: torch.Tensor, perm: torch.Tensor) -> torch.Tensor:
    Yp = _dev(Yp, torch.bfloat16, "Yp")
    perm = _dev(perm, torch.int32, "perm")
    M, Cc = Yp.shape
    Y = torch.empty_like(Yp)
    _check(lib().moqe_unpermute(_ptr(Yp), _ptr(perm), M, Cc, _ptr(Y), _stream()), "moqe_unpermute")
    return Y


def moqe_routed_qgemm_workspace(M: int, N: int, K: int, E: int) -> int:
    return int(lib().moqe_routed_qgemm_workspace(int(M), int(N), int(K), int(E)))


def alloc_workspace(nbytes: int, device=None) -> torch.Tensor:
    """Device scratch of at least ``nbytes`` (256-byte aligned: torch's allocator returns 512-byte aligned blocks)."""
    dev = device if device is not None else torch.device("cuda", torch.cuda.current_device())
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=dev)


def moqe_routed_qgemm(X: torch.Tensor, row_ids: torch.Tensor, experts: Sequence[Expert],
                      Y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                      path: int = PATH_AUTO) -> torch.Tensor:
    """``Y[m] = X[m] . dequant(W_{row_ids[m]})^T`` for bf16 ``X[M][K]`` -> bf16 ``Y[M][N]``."""
    X = _dev(X, torch.bfloat16, "X")
    row_ids = _dev(row_ids, torch.int32, "row_ids")
    M, K = X.shape
    E = len(experts)
    if E == 0:
        raise MoqeError(ERR_SHAPE, "moqe_routed_qgemm")
    N = experts[0].N
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = alloc_workspace(moqe_routed_qgemm_workspace(M, N, K, E), X.device)
    arr = (C.c_void_p * E)(*[e.handle for e in experts])
    _check(lib().moqe_routed_qgemm_path(_ptr(X), _ptr(row_ids), M, arr, E, _ptr(Y), _ptr(workspace), workspace.numel(),
                                        _stream(), int(path)), "moqe_routed_qgemm")
    return Y


def moqe_routed_qgemm_workspace_clear(workspace: torch.Tensor, M: int, N: int, K: int, E: int) -> None:
    _check(lib().moqe_routed_qgemm_workspace_clear(_ptr(workspace), workspace.numel(), int(M), int(N), int(K), int(E),
                                                   _stream()), "moqe_routed_qgemm_workspace_clear")


def moqe_routed_qgemm_sorted(X: torch.Tensor, perm: torch.Tensor, offsets: torch.Tensor, experts: Sequence[Expert],
                             Y: torch.Tensor, workspace: torch.Tensor, path: int = PATH_AUTO,
                             _arr=None) -> torch.Tensor:
    """Routed product for a batch already sorted by ``moqe_permute`` (``perm``, ``offsets``).

    ``workspace`` must have been cleared once with ``moqe_routed_qgemm_workspace_clear``.
    """
    M, K = X.shape
    E = len(experts)
    arr = _arr if _arr is not None else (C.c_void_p * E)(*[e.handle for e in experts])
    _check(lib().moqe_routed_qgemm_sorted(_ptr(X), _ptr(perm), _ptr(offsets), M, arr, E, _ptr(Y), _ptr(workspace),
                                          workspace.numel(), _stream(), int(path)), "moqe_routed_qgemm_sorted")
    return Y


def moqe_routed_qgemm_sorted_gated(X: torch.Tensor, perm: torch.Tensor, offsets: torch.Tensor, gate: Sequence[Expert],
                                   up: Sequence[Expert], Y: torch.Tensor, workspace: torch.Tensor, _arrs=None) -> torch.Tensor:
    """``Y = silu(X . Wgate_e^T) * (X . Wup_e^T)`` for a sorted decode batch, one launch."""
    M = X.shape[0]
    E = len(gate)
    ag, au = _arrs if _arrs is not None else ((C.c_void_p * E)(*[e.handle for e in gate]), (C.c_void_p * E)(*[e.handle for e in up]))
    _check(lib().moqe_routed_qgemm_sorted_gated(_ptr(X), _ptr(perm), _ptr(offsets), M, ag, au, E, _ptr(Y), _ptr(workspace),
                                                workspace.numel(), _stream()), "moqe_routed_qgemm_sorted_gated")
    return Y


def moqe_routed_qgemm_sorted_residual(X: torch.Tensor, perm: torch.Tensor, offsets: torch.Tensor, experts: Sequence[Expert],
                                      R: torch.Tensor, Y: torch.Tensor, workspace: torch.Tensor, _arr=None) -> torch.Tensor:
    """``Y = X . W_e^T + R`` for a sorted decode batch (``R`` bf16 ``[M][N]``, may be ``Y``)."""
    M = X.shape[0]
    E = len(experts)
    arr = _arr if _arr is not None else (C.c_void_p * E)(*[e.handle for e in experts])
    _check(lib().moqe_routed_qgemm_sorted_residual(_ptr(X), _ptr(perm), _ptr(offsets), M, arr, E, _ptr(R), _ptr(Y),
                                                   _ptr(workspace), workspace.numel(), _stream()), "moqe_routed_qgemm_sorted_residual")
    return Y


def moqe_routed_qgemm_sorted_multi(Xs: Sequence[torch.Tensor], perm: torch.Tensor, offsets: torch.Tensor,
                                   experts: Sequence[Sequence[Expert]], Ys: Sequence[torch.Tensor],
                                   workspace: torch.Tensor, _arrs=None):
    """Several independent layers of one decode batch (same ``perm`` / ``offsets``) in one launch:
    ``Ys[l] = routed product of Xs[l] with experts[l]``.  Raises ``MoqeError(ERR_UNSUPPORTED)`` for batches the
    decode kernel does not take (use ``moqe_routed_qgemm_sorted`` per layer then)."""
    nl = len(Xs)
    E = len(experts[0])
    M = Xs[0].shape[0]
    if _arrs is None:
        xa = (C.c_void_p * nl)(*[_ptr(x) for x in Xs])
        ya = (C.c_void_p * nl)(*[_ptr(y) for y in Ys])
        ea = (C.c_void_p * (nl * E))(*[e.handle for layer in experts for e in layer])
    else:
        xa, ya, ea = _arrs
    _check(lib().moqe_routed_qgemm_sorted_multi(xa, _ptr(perm), _ptr(offsets), M, nl, ea, E, ya, _ptr(workspace),
                                                workspace.numel(), _stream()), "moqe_routed_qgemm_sorted_multi")
    return Ys


def moqe_async_status() -> int:
    """Synchronises the current stream and returns (and clears) the latched device error."""
    return int(lib().moqe_async_status(_stream()))


def moqe_tune(key: str, value: int) -> None:
    _check(lib().moqe_tune(key.encode(), int(value)), "moqe_tune")


def moqe_router_mlp(X: torch.Tensor, row_offsets: torch.Tensor, W1: torch.Tensor, W2: torch.Tensor,
                    workspace: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """-> (logits fp32 [S][E], ids int32 [S]) of the router front end, all on the device."""
    S, H, D, E = row_offsets.numel() - 1, X.shape[1], W1.shape[0], W2.shape[0]
    logits = torch.empty((S, E), dtype=torch.float32, device=X.device)
    ids = torch.empty((S,), dtype=torch.int32, device=X.device)
    need = int(lib().moqe_router_mlp_workspace(S, H, D))
    ws = workspace if workspace is not None else alloc_workspace(need, X.device)
    _check(lib().moqe_router_mlp(X.data_ptr(), row_offsets.data_ptr(), S, H, W1.data_ptr(), D, W2.data_ptr(), E,
                                 logits.data_ptr(), ids.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "moqe_router_mlp")
    return logits, ids


def moqe_router_load_report(logits: torch.Tensor, ids: torch.Tensor):
    """-> (P fp32 [E], F fp32 [E], L_bal fp32 scalar tensor, counts int32 [E])."""
    S, E = logits.shape
    report = torch.empty((2 * E + 1,), dtype=torch.float32, device=logits.device)
    counts = torch.empty((E,), dtype=torch.int32, device=logits.device)
    _check(lib().moqe_router_load_report(logits.data_ptr(), ids.data_ptr(), S, E, report.data_ptr(), counts.data_ptr(),
                                         _stream()), "moqe_router_load_report")
    return report[:E], report[E:2 * E], report[2 * E], counts


def moqe_selftest_timeout(limit_us: int = 1000) -> int:
    """Runs the bounded-wait self-test; returns what the kernel wrote (2 = the wait gave up by itself)."""
    out = torch.zeros(1, dtype=torch.int32, device=torch.device("cuda", torch.cuda.current_device()))
    _check(lib().moqe_selftest_timeout(int(limit_us), out.data_ptr(), _stream()), "moqe_selftest_timeout")
    return out


def moqe_launch_count() -> int:
    return int(lib().moqe_launch_count())
