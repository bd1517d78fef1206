"""Seeded synthetic inputs for the routed quantized-linear workloads.

This module only *draws numbers and describes shapes*.  It contains none of the
method's arithmetic (no quantizer, no dequantizer, no argmax, no sort, no GEMM):
both the CPU oracle's tests and the CUDA library's tests feed on the arrays it
returns, and neither implementation imports the other.

Generator: numpy's Philox counter-based bit generator, keyed by
``(base_seed, stream)`` where ``stream`` is a stable 63-bit hash of the tensor's
name, so every tensor can be re-drawn independently and in any order.

The five workloads mirror the layer shapes, sequence lengths and per-sample
routing structure of the models the MoQE paper evaluates (Section 4: decoder
LLMs with sequences of at most 2048 tokens, ImageNet CNNs); the weights and
activations themselves are Gaussian stand-ins, not the paper's data.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

BASE_SEED = 20250809


# --------------------------------------------------------------------------
# random streams
# --------------------------------------------------------------------------
def _stream_key(name: str) -> int:
    h = hashlib.sha256(name.encode("utf-8")).digest()
    return int.from_bytes(h[:8], "little") >> 1


def rng(name: str, seed: int = BASE_SEED) -> np.random.Generator:
    """Independent generator for the tensor called ``name``."""
    return np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), _stream_key(name)]))


def normal_f32(name: str, shape: Sequence[int], std: float = 1.0, seed: int = BASE_SEED) -> np.ndarray:
    g = rng(name, seed)
    out = g.standard_normal(size=tuple(shape), dtype=np.float32)
    if std != 1.0:
        out *= np.float32(std)
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns.

    (Storage conversion of *inputs*; inputs are defined to be bf16.)
    """
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def activations_bf16(name: str, M: int, K: int, relu: bool = False, seed: int = BASE_SEED) -> np.ndarray:
    """``[M][K]`` bf16 bit patterns, N(0,1) (optionally passed through ReLU)."""
    x = normal_f32(name, (M, K), 1.0, seed)
    if relu:
        np.maximum(x, 0.0, out=x)
    return f32_to_bf16_bits(x)


def weights_f32(name: str, N: int, K: int, std: float = 0.02, seed: int = BASE_SEED) -> np.ndarray:
    """``[N][K]`` fp32 full-precision weight, N(0, std)."""
    return normal_f32(name, (N, K), std, seed)


# --------------------------------------------------------------------------
# workload descriptions
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class ExpertSpec:
    """One quantization expert's format: b-bit codes, group size along K
    (0 = one group per output channel), symmetric or asymmetric grid."""
    bits: int
    group: int
    sym: bool

    @property
    def tag(self) -> str:
        g = "pc" if self.group == 0 else f"g{self.group}"
        return f"W{self.bits}{'s' if self.sym else 'a'}-{g}"


@dataclass(frozen=True)
class LayerSpec:
    """A linear layer ``Y[M][N] = X[M][K] · W[N][K]^T``.  ``rows_per_sample``
    overrides the workload's per-sample row counts (CNN layers at different
    spatial resolutions)."""
    name: str
    N: int
    K: int
    rows_per_sample: Optional[int] = None


@dataclass(frozen=True)
class Workload:
    name: str
    layers: Tuple[LayerSpec, ...]
    experts: Tuple[ExpertSpec, ...]
    sample_rows: Tuple[int, ...]          # rows (tokens / pixels) of each sample
    routing: str                          # "uniform" | "skewed" | "router_mlp"
    routing_probs: Tuple[float, ...] = ()
    relu_inputs: bool = False
    kind: str = "decode"                  # "decode" | "prefill" | "mixed" | "conv"

    @property
    def n_samples(self) -> int:
        return len(self.sample_rows)

    @property
    def n_experts(self) -> int:
        return len(self.experts)

    def rows_of(self, layer: LayerSpec) -> np.ndarray:
        if layer.rows_per_sample is not None:
            return np.full(self.n_samples, layer.rows_per_sample, dtype=np.int64)
        return np.asarray(self.sample_rows, dtype=np.int64)

    def M_of(self, layer: LayerSpec) -> int:
        return int(self.rows_of(layer).sum())

    def row_offsets(self, layer: LayerSpec) -> np.ndarray:
        r = self.rows_of(layer)
        off = np.zeros(len(r) + 1, dtype=np.int32)
        off[1:] = np.cumsum(r)
        return off


_W8PC = ExpertSpec(8, 0, True)
_W4G128A = ExpertSpec(4, 128, False)
_W3G128A = ExpertSpec(3, 128, False)

_LLAMA7B = (
    LayerSpec("q_proj", 4096, 4096), LayerSpec("k_proj", 4096, 4096),
    LayerSpec("v_proj", 4096, 4096), LayerSpec("o_proj", 4096, 4096),
    LayerSpec("gate_proj", 11008, 4096), LayerSpec("up_proj", 11008, 4096),
    LayerSpec("down_proj", 4096, 11008),
)
_QWEN7B = (
    LayerSpec("q_proj", 3584, 3584), LayerSpec("k_proj", 512, 3584),
    LayerSpec("v_proj", 512, 3584), LayerSpec("o_proj", 3584, 3584),
    LayerSpec("gate_proj", 18944, 3584), LayerSpec("up_proj", 18944, 3584),
    LayerSpec("down_proj", 3584, 18944),
)
_RESNET = (
    LayerSpec("conv2_reduce_256to64_56x56", 64, 256, 56 * 56),
    LayerSpec("conv2_expand_64to256_56x56", 256, 64, 56 * 56),
    LayerSpec("conv4_reduce_1024to256_14x14", 256, 1024, 14 * 14),
    LayerSpec("conv4_expand_256to1024_14x14", 1024, 256, 14 * 14),
)

WORKLOADS = {
    "tiny": Workload(
        "tiny", (LayerSpec("linear", 1024, 1024),), (_W8PC, _W4G128A),
        (16,) * 4, "uniform", kind="decode"),
    "llama7b_decode": Workload(
        "llama7b_decode", _LLAMA7B, (_W8PC, _W4G128A, _W3G128A),
        (1,) * 16, "uniform", kind="decode"),
    "llama7b_prefill": Workload(
        "llama7b_prefill", _LLAMA7B, (_W8PC, _W4G128A, _W3G128A),
        (2048,) * 8, "skewed", (0.7, 0.2, 0.1), kind="prefill"),
    "qwen7b_mixed": Workload(
        "qwen7b_mixed", _QWEN7B,
        (_W8PC, ExpertSpec(4, 128, True), _W4G128A, ExpertSpec(3, 64, False)),
        (1,) * 64 + (1024,) * 4, "router_mlp", kind="mixed"),
    "resnet50_1x1": Workload(
        "resnet50_1x1", _RESNET,
        (_W8PC, ExpertSpec(4, 0, False), ExpertSpec(4, 32, False)),
        (1,) * 256, "uniform", relu_inputs=True, kind="conv"),
}
WORKLOAD_ORDER = ("tiny", "llama7b_decode", "llama7b_prefill", "qwen7b_mixed", "resnet50_1x1")


def get(name_or_index) -> Workload:
    if isinstance(name_or_index, int):
        return WORKLOADS[WORKLOAD_ORDER[name_or_index]]
    return WORKLOADS[name_or_index]


# --------------------------------------------------------------------------
# routing inputs (logits); the argmax itself belongs to the implementations
# --------------------------------------------------------------------------
def router_logits(w: Workload, seed: int = BASE_SEED, pooled: Optional[np.ndarray] = None) -> np.ndarray:
    """fp32 ``[S][E]`` router outputs whose arg-max is the sample's expert.

    * ``uniform`` / ``skewed``: a one-hot-like score row per sample; the hot
      column is drawn from the stated probabilities, the other columns get
      distinct smaller scores, so any correct first-max argmax recovers it.
    * ``router_mlp``: scores of a 2-layer fp32 MLP (hidden -> 256 -> E, ReLU,
      zero biases, random init) applied to ``pooled`` (``[S][hidden]`` fp32
      mean-pooled activations).  This stands in for the paper's trained router
      (Section 3.2); it only manufactures logits.
    """
    S, E = w.n_samples, w.n_experts
    if w.routing in ("uniform", "skewed"):
        g = rng(f"{w.name}/routing", seed)
        p = np.asarray(w.routing_probs, dtype=np.float64) if w.routing == "skewed" else np.full(E, 1.0 / E)
        hot = g.choice(E, size=S, p=p / p.sum())
        logits = g.uniform(-1.0, 0.0, size=(S, E)).astype(np.float32)
        logits[np.arange(S), hot] = np.float32(1.0)
        return logits
    if w.routing == "router_mlp":
        if pooled is None:
            raise ValueError("router_mlp routing needs the pooled activations")
        H = pooled.shape[1]
        w1 = normal_f32(f"{w.name}/router/w1", (256, H), 1.0 / np.sqrt(H), seed)
        w2 = normal_f32(f"{w.name}/router/w2", (E, 256), 1.0 / np.sqrt(256.0), seed)
        h = np.maximum(pooled.astype(np.float32) @ w1.T, np.float32(0.0))
        return (h @ w2.T).astype(np.float32)
    raise ValueError(w.routing)


def router_weights(w: Workload, seed: int = BASE_SEED):
    """The random fp32 weights ``(W1 [256][hidden], W2 [E][256])`` of the ``router_mlp`` workloads' stand-in router."""
    H, E = w.layers[0].K, w.n_experts
    w1 = normal_f32(f"{w.name}/router/w1", (256, H), 1.0 / np.sqrt(H), seed)
    w2 = normal_f32(f"{w.name}/router/w2", (E, 256), 1.0 / np.sqrt(256.0), seed)
    return w1, w2


def mean_pool(x_bf16: np.ndarray, row_offsets: np.ndarray) -> np.ndarray:
    """fp32 mean of each sample's rows (input preparation for ``router_mlp``)."""
    x = bf16_bits_to_f32(x_bf16)
    S = len(row_offsets) - 1
    out = np.empty((S, x.shape[1]), dtype=np.float32)
    for s in range(S):
        out[s] = x[row_offsets[s]:row_offsets[s + 1]].mean(axis=0, dtype=np.float32)
    return out


def layer_inputs(w: Workload, layer: LayerSpec, seed: int = BASE_SEED):
    """``(W fp32 [N][K], X bf16-bits [M][K])`` for one layer of a workload."""
    W = weights_f32(f"{w.name}/{layer.name}/W", layer.N, layer.K, 0.02, seed)
    X = activations_bf16(f"{w.name}/{layer.name}/X", w.M_of(layer), layer.K, w.relu_inputs, seed)
    return W, X
