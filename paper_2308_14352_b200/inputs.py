"""Seeded synthetic inputs for the sparse-MoE layer: activations, router weights,
expert weight matrices, per-expert bitwidths and load-shaping router biases.

This module is the only code shared by the CUDA path's tests/benchmarks and the CPU
checker.  It holds no quantisation, routing or FFN arithmetic: it only draws random
tensors with the shapes and value distributions of the paper's workloads (Table 1:
Switch-Transformer-base/large expert shapes; Section 4.2: a Mixtral-class 8-expert
top-2 SwiGLU model) and hands them to whoever asks.

Every tensor is a pure function of (seed, tensor id): numbers come from numpy's
counter-based Philox generator keyed by the seed and a packed tensor id, drawn in
fixed-size chunks so that the values do not depend on the number of worker threads.
"""
from __future__ import annotations

import dataclasses
import math
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_CHUNK = 1 << 22  # values per Philox stream; part of the recipe (changing it changes the data)

# tensor kinds (top byte of the tensor id)
_KIND_X = 1
_KIND_ROUTER = 2
_KIND_EXPERT = 3
_KIND_BITS = 4
_KIND_PRIOR = 5
_KIND_MISC = 6


@dataclasses.dataclass(frozen=True)
class LayerShape:
    """Static description of one MoE layer (paper Section 2.1: N experts, each an
    independent FFN, a router picking the Top-K)."""

    d_model: int
    d_ff: int
    n_experts: int
    top_k: int
    act: str  # "relu" (W_in, W_out) | "swiglu" (w1, w3, w2)
    gate_mode: str  # "softmax" | "softmax_renorm"
    group: int  # 0 = one scale per output channel, else scales per `group` inputs
    scale_dtype: str  # "f32" | "f16"
    act_dtype: str  # "f32" | "bf16"

    @property
    def n_matrices(self) -> int:
        return 2 if self.act == "relu" else 3

    def matrix_shape(self, m: int) -> Tuple[int, int]:
        """(N output channels, K inputs) of matrix m of an expert."""
        if self.act == "relu":
            return (self.d_ff, self.d_model) if m == 0 else (self.d_model, self.d_ff)
        return (self.d_ff, self.d_model) if m < 2 else (self.d_model, self.d_ff)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    shape: LayerShape
    n_layers: int
    tokens: Tuple[int, ...]  # batch sizes the workload is run at
    bits_rule: str  # "fixed" | "iid_25_50_25" | "exact_1_2_1"
    fixed_bits: Tuple[int, ...] = ()
    zipf_s: Optional[float] = None  # router loads follow Zipf(s) when set
    seed: int = 0


WORKLOADS: Dict[str, Workload] = {
    # single Switch-style layer, fp32 activations, per-output-channel fp32 scales
    "switch_tiny_fp32": Workload(
        "switch_tiny_fp32",
        LayerShape(768, 3072, 8, 1, "relu", "softmax", 0, "f32", "f32"),
        1, (16,), "fixed", (8, 4, 2, 4, 8, 2, 4, 8), None, 0),
    # Switch-base-like 12-layer decode stack
    "switch_base_decode": Workload(
        "switch_base_decode",
        LayerShape(768, 3072, 32, 1, "relu", "softmax", 128, "f16", "bf16"),
        12, (1, 8, 64), "iid_25_50_25", (), None, 1),
    # Switch-large-like prefill layer with Zipf(1.1) expert loads
    "switch_large_prefill": Workload(
        "switch_large_prefill",
        LayerShape(1024, 4096, 128, 1, "relu", "softmax", 128, "f16", "bf16"),
        1, (2048,), "exact_1_2_1", (), 1.1, 2),
    # Mixtral-like decode layer
    "mixtral_decode": Workload(
        "mixtral_decode",
        LayerShape(4096, 14336, 8, 2, "swiglu", "softmax_renorm", 128, "f16", "bf16"),
        1, (1, 4, 16, 32), "fixed", (4, 4, 8, 2, 4, 8, 2, 4), None, 3),
    # Mixtral-like 32-layer stack with host-resident experts and an HBM expert cache
    "mixtral_stack_cached": Workload(
        "mixtral_stack_cached",
        LayerShape(4096, 14336, 8, 2, "swiglu", "softmax_renorm", 128, "f16", "bf16"),
        32, (2048, 1), "fixed", (4, 4, 8, 2, 4, 8, 2, 4), None, 4),
}


def _tensor_id(kind: int, layer: int = 0, expert: int = 0, matrix: int = 0) -> int:
    assert 0 <= layer < (1 << 12) and 0 <= expert < (1 << 16) and 0 <= matrix < 16
    return (kind << 56) | (layer << 44) | (expert << 28) | (matrix << 24)


def _draw_chunk(seed: int, tid: int, chunk: int, n: int, out: np.ndarray) -> None:
    gen = np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, tid | chunk]))
    gen.standard_normal(n, dtype=np.float32, out=out)


def normal_f32(seed: int, tid: int, n: int, std: float = 1.0, threads: int = 8) -> np.ndarray:
    """n iid N(0, std^2) fp32 values, a pure function of (seed, tid)."""
    out = np.empty(n, dtype=np.float32)
    n_chunks = (n + _CHUNK - 1) // _CHUNK
    assert n_chunks < (1 << 24)
    jobs = [(c, c * _CHUNK, min(n, (c + 1) * _CHUNK)) for c in range(n_chunks)]
    if n_chunks <= 1 or threads <= 1:
        for c, lo, hi in jobs:
            _draw_chunk(seed, tid, c, hi - lo, out[lo:hi])
    else:
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(lambda j: _draw_chunk(seed, tid, j[0], j[2] - j[1], out[j[1]:j[2]]), jobs))
    if std != 1.0:
        out *= np.float32(std)
    return out


def to_bf16_valued(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even) and return them as fp32."""
    import torch

    return torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).to(torch.float32).numpy()


def activations(seed: int, layer: int, T: int, d_model: int, act_dtype: str, batch_tag: int = 0) -> np.ndarray:
    """x[T][d_model] ~ N(0,1): the post-norm input of a transformer block's FFN.
    bf16 workloads get bf16-representable values (still returned as fp32)."""
    x = normal_f32(seed, _tensor_id(_KIND_X, layer, batch_tag & 0xFFFF), T * d_model).reshape(T, d_model)
    return to_bf16_valued(x) if act_dtype == "bf16" else x


def router_weight(seed: int, layer: int, d_model: int, n_experts: int, std: float = 0.02) -> np.ndarray:
    """Router weight Wr[d_model][n_experts] ~ N(0, std^2), fp32."""
    return normal_f32(seed, _tensor_id(_KIND_ROUTER, layer), d_model * n_experts, std).reshape(d_model, n_experts)


def expert_matrix(seed: int, layer: int, expert: int, matrix: int, N: int, K: int, std: float = 0.02) -> np.ndarray:
    """One expert weight matrix W[N][K] ~ N(0, std^2), fp32, rows = output channels."""
    return normal_f32(seed, _tensor_id(_KIND_EXPERT, layer, expert, matrix), N * K, std).reshape(N, K)


def expert_bits(w: Workload, layer: int) -> List[int]:
    """Bitwidth of every expert of one layer (the output of the paper's offline
    bitwidth selection, Section 3.2, taken here as an input)."""
    E = w.shape.n_experts
    if w.bits_rule == "fixed":
        assert len(w.fixed_bits) == E
        return list(w.fixed_bits)
    gen = np.random.Generator(np.random.Philox(key=[w.seed, _tensor_id(_KIND_BITS, layer)]))
    if w.bits_rule == "iid_25_50_25":
        return [int(b) for b in gen.choice([2, 4, 8], size=E, p=[0.25, 0.5, 0.25])]
    if w.bits_rule == "exact_1_2_1":
        assert E % 4 == 0
        bits = np.array([2] * (E // 4) + [4] * (E // 2) + [8] * (E // 4))
        gen.shuffle(bits)
        return [int(b) for b in bits]
    raise ValueError(w.bits_rule)


def zipf_targets(n_experts: int, s: float) -> np.ndarray:
    """Target load share of expert e: proportional to (e+1)^-s."""
    p = np.arange(1, n_experts + 1, dtype=np.float64) ** (-s)
    return p / p.sum()


def zipf_router_bias(x: np.ndarray, Wr: np.ndarray, s: float, iters: int = 400, eta: float = 0.1) -> np.ndarray:
    """Additive per-expert router bias that makes the realised top-1 loads of the seeded batch x
    follow Zipf(s).  Damped fixed-point iteration b += eta * (log target - log observed); the
    iterate with the smallest worst-case load error is kept.  This shapes an *input* (the bias
    vector); the layer under test recomputes its own logits from x, Wr and this bias."""
    T, E = x.shape[0], Wr.shape[1]
    z = x.astype(np.float64) @ Wr.astype(np.float64)
    target = zipf_targets(E, s) * T
    b = np.log(target / T)
    best, best_err = b.copy(), np.inf
    for _ in range(iters):
        load = np.bincount(np.argmax(z + b, axis=1), minlength=E).astype(np.float64)
        err = np.max(np.abs(load - target))
        if err < best_err:
            best, best_err = b.copy(), err
        b = b + eta * (np.log(target + 0.5) - np.log(load + 0.5))
    return best.astype(np.float32)


def transition_prior(seed: int, n_experts: int, concentration: float = 0.3) -> np.ndarray:
    """Row-stochastic [E][E] layer-transition prior P(next expert | previous expert),
    the first-order stand-in for the paper's activation dictionary (Section 3.3.1)."""
    gen = np.random.Generator(np.random.Philox(key=[seed, _tensor_id(_KIND_PRIOR)]))
    return gen.dirichlet([concentration] * n_experts, size=n_experts).astype(np.float64)


def layer_tensors(w: Workload, layer: int, T: int, batch_tag: int = 0):
    """(x, Wr, bias-or-None) of one layer of a workload at batch size T."""
    sh = w.shape
    x = activations(w.seed, layer, T, sh.d_model, sh.act_dtype, batch_tag)
    Wr = router_weight(w.seed, layer, sh.d_model, sh.n_experts)
    bias = zipf_router_bias(x, Wr, w.zipf_s) if w.zipf_s is not None else None
    return x, Wr, bias


def small_shape(act: str = "relu", act_dtype: str = "f32", group: int = 0, scale_dtype: str = "f32",
                d_model: int = 64, d_ff: int = 128, n_experts: int = 4, top_k: int = 1,
                gate_mode: str = "softmax") -> LayerShape:
    """Convenience constructor for the small layers the tests sweep."""
    return LayerShape(d_model, d_ff, n_experts, top_k, act, gate_mode, group, scale_dtype, act_dtype)


def expert_set(seed: int, layer: int, shape: LayerShape, std: float = 0.02) -> List[List[np.ndarray]]:
    """All experts' fp32 matrices of one layer: result[e][m] is W[N][K]."""
    out = []
    for e in range(shape.n_experts):
        mats = []
        for m in range(shape.n_matrices):
            N, K = shape.matrix_shape(m)
            mats.append(expert_matrix(seed, layer, e, m, N, K, std))
        out.append(mats)
    return out
