"""Shared plumbing of the GPU parity tests: the same seeded arrays go to the CPU
oracle (numpy) and to the CUDA library (torch device tensors, through the C-ABI
binding); results are compared here."""
import numpy as np
import torch

import oracle
import moqe_workloads as wl
import paper_2508_09204_b200 as moqe

# Tolerance of the routed GEMM (bf16 output, fp32 accumulate): both sides' bf16 outputs are
# widened to fp32; relative error is |d| / max(|ref|, rms(ref)).
MAX_REL_ERR = 1e-2
MEAN_ABS_ERR = 2e-3


def dev():
    return torch.device("cuda", 0)


def bf16_to_torch(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev()).view(torch.bfloat16)


def torch_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def build_experts(W: np.ndarray, specs):
    """-> (gpu experts, oracle dequantized fp32 weights, oracle (codes, scales, zeros))."""
    Wd = torch.from_numpy(W).to(dev())
    gpu, What, canon = [], [], []
    for sp in specs:
        bits, group, sym = (sp.bits, sp.group, sp.sym) if hasattr(sp, "bits") else sp
        gpu.append(moqe.moqe_quantize_rtn(Wd, bits, group, sym))
        c, s, z = oracle.quantize_rtn(W, bits, group, sym)
        canon.append((c, s, z))
        What.append(oracle.dequantize(c, s, z, group))
    return gpu, What, canon


def assert_expert_matches(e, canon):
    c, s, z = canon
    gc, gs, gz = moqe.moqe_expert_export(e)
    assert np.array_equal(gc.cpu().numpy(), c), "codes differ"
    assert np.array_equal(torch_to_bits(gs), s), "scales differ"
    assert np.array_equal(torch_to_bits(gz), z), "zero-points differ"


def compare_outputs(got_bits: np.ndarray, ref_bits: np.ndarray):
    got = wl.bf16_bits_to_f32(got_bits).astype(np.float64)
    ref = wl.bf16_bits_to_f32(ref_bits).astype(np.float64)
    assert got.shape == ref.shape
    assert np.all(np.isfinite(got))
    rho = np.sqrt(np.mean(ref ** 2)) if ref.size else 1.0
    d = np.abs(got - ref)
    rel = d / np.maximum(np.abs(ref), max(rho, 1e-30))
    return float(rel.max()) if ref.size else 0.0, float(d.mean()) if ref.size else 0.0


def _where_off(got_bits, ref_bits) -> str:
    """Which elements are outside the relative bar (for the failure message)."""
    got = wl.bf16_bits_to_f32(got_bits).astype(np.float64)
    ref = wl.bf16_bits_to_f32(ref_bits).astype(np.float64)
    rho = np.sqrt(np.mean(ref ** 2)) if ref.size else 1.0
    bad = np.abs(got - ref) / np.maximum(np.abs(ref), max(rho, 1e-30)) > MAX_REL_ERR
    r, c = np.nonzero(bad.reshape(bad.shape[0], -1))
    if r.size == 0:
        return "no element off"
    return (f"{r.size} elements off, rows {r.min()}..{r.max()} ({np.unique(r).size} rows: {np.unique(r)[:16].tolist()}), "
            f"columns {c.min()}..{c.max()} ({np.unique(c).size} columns), first got {got.reshape(bad.shape[0], -1)[r[0], c[0]]:.6g} "
            f"ref {ref.reshape(bad.shape[0], -1)[r[0], c[0]]:.6g}, zeros among them {(got.reshape(bad.shape[0], -1)[r, c] == 0).sum()}")


def assert_close(got_bits, ref_bits, what=""):
    mx, mean = compare_outputs(got_bits, ref_bits)
    assert mx <= MAX_REL_ERR, f"{what}: max relative error {mx:.3e} > {MAX_REL_ERR}; {_where_off(got_bits, ref_bits)}"
    assert mean <= MEAN_ABS_ERR, f"{what}: mean abs error {mean:.3e} > {MEAN_ABS_ERR}"
    return mx, mean


def sample_rows(offsets: np.ndarray, per_expert: int, seed: int, perm: np.ndarray) -> np.ndarray:
    """Original row indices: first and last row of every expert segment plus a seeded random set."""
    rs = np.random.default_rng(seed)
    rows = []
    for e in range(len(offsets) - 1):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi <= lo:
            continue
        pick = {lo, hi - 1}
        pick.update(int(v) for v in rs.integers(lo, hi, size=min(per_expert, hi - lo)))
        rows.extend(int(perm[j]) for j in sorted(pick))
    return np.array(sorted(set(rows)), dtype=np.int32)
