"""Python face of the CPU oracle (``moqe_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
bench's CPU-baseline / reference legs.  The CUDA library and its binding never
import this package, and this package never imports them.

Every function here only marshals numpy arrays into the C routines; the
arithmetic is in the C file, which states what each routine follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moqe_oracle.c")
_LIB = os.path.join(_HERE, "libmoqe_oracle.so")

CFLAGS = ["-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-Wall"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", *CFLAGS, _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_f16_to_f32.restype = C.c_float
        _lib.oracle_f16_to_f32.argtypes = [C.c_uint16]
        _lib.oracle_f32_to_f16.restype = C.c_uint16
        _lib.oracle_f32_to_f16.argtypes = [C.c_float]
        _lib.oracle_f32_to_bf16.restype = C.c_uint16
        _lib.oracle_f32_to_bf16.argtypes = [C.c_float]
        _lib.oracle_bf16_to_f32.restype = C.c_float
        _lib.oracle_bf16_to_f32.argtypes = [C.c_uint16]
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(rc: int, what: str):
    if rc == -2:
        raise ValueError(f"{what}: expert id out of range")
    if rc != 0:
        raise ValueError(f"{what}: bad argument")


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def quantize_rtn(W: np.ndarray, bits: int, group: int, sym: bool):
    """-> (codes uint8 [N][K], scales fp16-bits [N][K/g], zeros fp16-bits [N][K/g])."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    g = K if group == 0 else group
    if g <= 0 or K % g:
        raise ValueError("group must divide K")
    codes = np.empty((N, K), dtype=np.uint8)
    scales = np.empty((N, K // g), dtype=np.uint16)
    zeros = np.empty((N, K // g), dtype=np.uint16)
    _chk(lib().oracle_quantize_rtn(_p(W), N, K, int(bits), int(group), int(bool(sym)),
                                   _p(codes), _p(scales), _p(zeros)), "quantize_rtn")
    return codes, scales, zeros


def dequantize(codes: np.ndarray, scales: np.ndarray, zeros: np.ndarray, group: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint16)
    zeros = np.ascontiguousarray(zeros, dtype=np.uint16)
    N, K = codes.shape
    out = np.empty((N, K), dtype=np.float32)
    _chk(lib().oracle_dequantize(_p(codes), _p(scales), _p(zeros), N, K, int(group), _p(out)), "dequantize")
    return out


def route(logits: np.ndarray) -> np.ndarray:
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    S, E = logits.shape
    ids = np.empty(S, dtype=np.int32)
    _chk(lib().oracle_route(_p(logits), S, E, _p(ids)), "route")
    return ids


def expand_ids(ids: np.ndarray, row_offsets: np.ndarray) -> np.ndarray:
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    row_offsets = np.ascontiguousarray(row_offsets, dtype=np.int32)
    S = len(ids)
    out = np.empty(int(row_offsets[-1]) if S else 0, dtype=np.int32)
    _chk(lib().oracle_expand_ids(_p(ids), _p(row_offsets), S, _p(out)), "expand_ids")
    return out


def permutation(row_ids: np.ndarray, E: int):
    """-> (counts[E], offsets[E+1], perm[M], inv[M]) of the stable counting sort."""
    row_ids = np.ascontiguousarray(row_ids, dtype=np.int32)
    M = len(row_ids)
    counts = np.empty(E, dtype=np.int32)
    offsets = np.empty(E + 1, dtype=np.int32)
    perm = np.empty(M, dtype=np.int32)
    inv = np.empty(M, dtype=np.int32)
    _chk(lib().oracle_permutation(_p(row_ids), M, E, _p(counts), _p(offsets), _p(perm), _p(inv)), "permutation")
    return counts, offsets, perm, inv


def permute_rows(X: np.ndarray, perm: np.ndarray) -> np.ndarray:
    X = np.ascontiguousarray(X, dtype=np.uint16)
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    M, Cc = X.shape
    out = np.empty_like(X)
    _chk(lib().oracle_permute_rows(_p(X), _p(perm), M, Cc, _p(out)), "permute_rows")
    return out


def unpermute_rows(Yp: np.ndarray, perm: np.ndarray) -> np.ndarray:
    Yp = np.ascontiguousarray(Yp, dtype=np.uint16)
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    M, Cc = Yp.shape
    out = np.empty_like(Yp)
    _chk(lib().oracle_unpermute_rows(_p(Yp), _p(perm), M, Cc, _p(out)), "unpermute_rows")
    return out


def _what_array(What: Sequence[np.ndarray]):
    keep = [np.ascontiguousarray(w, dtype=np.float32) for w in What]
    arr = (C.c_void_p * len(keep))(*[w.ctypes.data for w in keep])
    return keep, arr


def routed_gemm(X: np.ndarray, row_ids: np.ndarray, What: Sequence[np.ndarray],
                rows: Optional[np.ndarray] = None, want_f32: bool = False):
    """Y (bf16 bits) for all rows, or for the listed ``rows`` only.

    ``What[e]`` is expert e's dequantized fp32 ``[N][K]`` weight.  With
    ``want_f32`` the unrounded fp32 accumulators are returned as well.
    """
    X = np.ascontiguousarray(X, dtype=np.uint16)
    row_ids = np.ascontiguousarray(row_ids, dtype=np.int32)
    M, K = X.shape
    keep, arr = _what_array(What)
    N = keep[0].shape[0]
    for w in keep:
        if w.shape != (N, K):
            raise ValueError("experts disagree on shape")
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int32)
    R = M if rows is None else len(rows)
    Y = np.empty((R, N), dtype=np.uint16)
    Yf = np.empty((R, N), dtype=np.float32) if want_f32 else None
    _chk(lib().oracle_routed_gemm(_p(X), _p(row_ids), M, K, N, len(keep), arr, _p(rows), R, _p(Y), _p(Yf)),
         "routed_gemm")
    return (Y, Yf) if want_f32 else Y


def routed_gemm_f64(X: np.ndarray, row_ids: np.ndarray, What: Sequence[np.ndarray],
                    rows: Optional[np.ndarray] = None) -> np.ndarray:
    X = np.ascontiguousarray(X, dtype=np.uint16)
    row_ids = np.ascontiguousarray(row_ids, dtype=np.int32)
    M, K = X.shape
    keep, arr = _what_array(What)
    N = keep[0].shape[0]
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int32)
    R = M if rows is None else len(rows)
    Y = np.empty((R, N), dtype=np.float64)
    _chk(lib().oracle_routed_gemm_f64(_p(X), _p(row_ids), M, K, N, len(keep), arr, _p(rows), R, _p(Y)),
         "routed_gemm_f64")
    return Y


def router_mlp(X: np.ndarray, row_offsets: np.ndarray, W1: np.ndarray, W2: np.ndarray):
    """Router front end -> (logits fp64 [S][E], pooled fp64 [S][H]): mean-pooled rows, two-layer ReLU MLP, fp64."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    off = np.ascontiguousarray(row_offsets, dtype=np.int32)
    W1 = np.ascontiguousarray(W1, dtype=np.float32)
    W2 = np.ascontiguousarray(W2, dtype=np.float32)
    S, H, D, E = len(off) - 1, X.shape[1], W1.shape[0], W2.shape[0]
    if W1.shape[1] != H or W2.shape[1] != D or (S and off[-1] > X.shape[0]):
        raise ValueError("router_mlp: shapes disagree")
    pooled = np.empty((S, H), dtype=np.float64)
    logits = np.empty((S, E), dtype=np.float64)
    _chk(lib().oracle_router_mlp(_p(X), _p(off), S, H, _p(W1), D, _p(W2), E, _p(pooled), _p(logits)), "router_mlp")
    return logits, pooled


def load_report(logits: np.ndarray, ids: np.ndarray):
    """-> (P fp64 [E], F fp64 [E], L_bal): mean routing probability, dispatched fraction, balance term."""
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    S, E = logits.shape
    P = np.empty(E, dtype=np.float64)
    F = np.empty(E, dtype=np.float64)
    lb = C.c_double(0.0)
    _chk(lib().oracle_load_report(_p(logits), _p(ids), S, E, _p(P), _p(F), C.byref(lb)), "load_report")
    return P, F, float(lb.value)


def routed_gated_pair(X: np.ndarray, row_ids: np.ndarray, Wgate: Sequence[np.ndarray], Wup: Sequence[np.ndarray]) -> np.ndarray:
    """bf16 bits of silu(X.Wgate_e^T) * (X.Wup_e^T), fp32 throughout, rounded once."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    row_ids = np.ascontiguousarray(row_ids, dtype=np.int32)
    M, K = X.shape
    N = Wgate[0].shape[0]
    gk, ga = _what_array(Wgate)
    uk, ua = _what_array(Wup)
    Y = np.empty((M, N), dtype=np.uint16)
    _chk(lib().oracle_routed_gated_pair(_p(X), _p(row_ids), M, K, N, len(Wgate), ga, ua, _p(Y)), "routed_gated_pair")
    return Y


def routed_gemm_residual(X: np.ndarray, row_ids: np.ndarray, What: Sequence[np.ndarray], R: np.ndarray) -> np.ndarray:
    """bf16 bits of X.W_e^T + R (R bf16 bits), fp32, rounded once."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    row_ids = np.ascontiguousarray(row_ids, dtype=np.int32)
    R = np.ascontiguousarray(R, dtype=np.uint16)
    M, K = X.shape
    N = What[0].shape[0]
    wk, wa = _what_array(What)
    Y = np.empty((M, N), dtype=np.uint16)
    _chk(lib().oracle_routed_gemm_residual(_p(X), _p(row_ids), M, K, N, len(What), wa, _p(R), _p(Y)), "routed_gemm_residual")
    return Y


def f16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    L = lib()
    flat = np.ascontiguousarray(h, dtype=np.uint16).ravel()
    return np.array([L.oracle_f16_to_f32(int(v)) for v in flat], dtype=np.float32).reshape(np.shape(h))


def f32_to_f16_bits(f: np.ndarray) -> np.ndarray:
    L = lib()
    flat = np.ascontiguousarray(f, dtype=np.float32).ravel()
    return np.array([L.oracle_f32_to_f16(float(v)) for v in flat], dtype=np.uint16).reshape(np.shape(f))


def f32_to_bf16_bits(f: np.ndarray) -> np.ndarray:
    L = lib()
    flat = np.ascontiguousarray(f, dtype=np.float32).ravel()
    return np.array([L.oracle_f32_to_bf16(float(v)) for v in flat], dtype=np.uint16).reshape(np.shape(f))
