"""A stack of MoE layers whose packed experts live in pinned host memory and are staged into the
library's HBM expert cache: the predict-then-prefetch pipeline of the paper's Section 3.3
("Preloading and pipeline", "Cache eviction policy") on a B200.  Everything here is plumbing
(memory, streams, the order of the library calls); the arithmetic runs in the library's kernels
and the cache decisions in its host code.

Per layer and token batch:
  ids, gates = emoe_router_topk(x, Wr, bias)           # bias ties the routing to the prior
  emoe_prefetch_experts(ranked experts of the next layer)   # copy stream, overlaps this layer
  emoe_cache_acquire(activated experts)                # compute stream waits on the device
  emoe_moe_forward_routed(...); emoe_cache_release(...)
"""
from __future__ import annotations

import ctypes
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from .inputs import LayerShape
from .layer import make_desc

_SDT = {"f32": B.DTYPE_F32, "f16": B.DTYPE_F16}


class CachedStack:
    def __init__(self, shape: LayerShape, n_layers: int, bits: Sequence[int], n_slots: int, device: int = 0,
                 max_tokens: int = 1, seed: int = 4, policy: int = B.EVICT_FORWARD, beta: float = 4.0,
                 n_prefetch: Optional[int] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("CachedStack needs a CUDA device: there is no CPU path")
        assert shape.act_dtype == "bf16"
        self.shape, self.n_layers, self.bits = shape, n_layers, list(bits)
        self.dev = torch.device("cuda", device)
        torch.cuda.set_device(self.dev)
        self.desc = make_desc(shape)
        self.max_tokens = max_tokens
        self.beta = beta
        self.n_prefetch = shape.top_k if n_prefetch is None else n_prefetch
        self.ctx = B.emoe_create(device, B.emoe_workspace_bytes(self.desc, max_tokens))
        self.compute = torch.cuda.Stream(device=self.dev)
        self.copy = torch.cuda.Stream(device=self.dev)
        E = shape.n_experts
        self.seed = seed
        self._gen = torch.Generator(device=self.dev)
        sdt = torch.float16 if shape.scale_dtype == "f16" else torch.float32
        # experts: seeded N(0, 0.02^2) fp32 on the device -> packed by the library -> pinned host memory
        self.host: List[List[tuple]] = []
        self.expert_bytes = 0
        slot_bytes = 0
        for l in range(n_layers):
            row = []
            for e in range(E):
                pm, sm = [], []
                for m in range(shape.n_matrices):
                    N, K = shape.matrix_shape(m)
                    G = shape.group if shape.group > 0 else K
                    W = self.draw_matrix(l, e, m)
                    p = torch.empty(N * K * self.bits[e] // 8, dtype=torch.uint8, device=self.dev)
                    s = torch.empty(N * (K // G), dtype=sdt, device=self.dev)
                    B.emoe_pack_expert(self.ctx, W.data_ptr(), N, K, self.bits[e], shape.group, _SDT[shape.scale_dtype],
                                       p.data_ptr(), s.data_ptr(), 0)
                    pm.append(p.cpu().pin_memory())
                    sm.append(s.cpu().pin_memory())
                    del W, p, s
                row.append((pm, sm))
                nb = self._nbytes(pm, sm)
                self.expert_bytes += sum(nb)
                slot_bytes = max(slot_bytes, sum((b + 255) // 256 * 256 for b in nb))
            self.host.append(row)
        self.slot_bytes = slot_bytes
        self.n_slots = n_slots
        B.emoe_cache_create(self.ctx, n_slots, slot_bytes, n_layers, policy)
        for l in range(n_layers):
            for e in range(E):
                pm, sm = self.host[l][e]
                pad = [0] * (3 - len(pm))
                B.emoe_register_expert(self.ctx, self.expert_id(l, e), l, self.bits[e], [t.data_ptr() for t in pm] + pad,
                                       [t.data_ptr() for t in sm] + pad, self._nbytes(pm, sm))
        # routers and the layer-transition prior (row-stochastic, seeded)
        rng = np.random.default_rng(seed)
        self.Wr = [torch.from_numpy((rng.standard_normal((shape.d_model, E)) * 0.02).astype(np.float32)).to(self.dev)
                   for _ in range(n_layers)]
        prior = rng.random((E, E)) ** 4          # peaked rows: a few likely successors per expert
        self.prior = (prior / prior.sum(axis=1, keepdims=True)).astype(np.float32)
        self._exposed_ns_seen = 0
        self.ids = torch.empty(max_tokens, shape.top_k, dtype=torch.int32, device=self.dev)
        self.gates = torch.empty(max_tokens, shape.top_k, dtype=torch.float32, device=self.dev)
        self.bias = torch.zeros(max_tokens, E, dtype=torch.float32, device=self.dev)
        self.y = torch.empty(max_tokens, shape.d_model, dtype=torch.float32, device=self.dev)
        torch.cuda.synchronize(self.dev)

    def draw_matrix(self, l: int, e: int, m: int) -> torch.Tensor:
        """The fp32 weight matrix m of expert e of layer l (seeded N(0, 0.02^2), drawn on the device)."""
        N, K = self.shape.matrix_shape(m)
        self._gen.manual_seed((self.seed << 32) ^ (l << 16) ^ (e << 4) ^ m)
        return torch.randn(N, K, generator=self._gen, device=self.dev, dtype=torch.float32) * 0.02

    @staticmethod
    def _nbytes(pm, sm):
        nb = [t.numel() * t.element_size() for t in pm] + [0] * (3 - len(pm))
        return nb + [t.numel() * t.element_size() for t in sm] + [0] * (3 - len(sm))

    def expert_id(self, layer: int, e: int) -> int:
        return layer * self.shape.n_experts + e

    def close(self):
        if self.ctx is not None:
            torch.cuda.synchronize(self.dev)
            B.emoe_destroy(self.ctx)
            self.ctx = None

    def h2d_rate_gbs(self) -> float:
        """Pinned host -> device copy rate of this machine, on one expert's largest matrix."""
        src = max((t for t in self.host[0][0][0]), key=lambda t: t.numel())
        dst = torch.empty(src.numel(), dtype=torch.uint8, device=self.dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(self.copy):
            dst.copy_(src, non_blocking=True)
            e0.record()
            for _ in range(4):
                dst.copy_(src, non_blocking=True)
            e1.record()
        e1.synchronize()
        return 4 * src.numel() / (e0.elapsed_time(e1) * 1e-3) / 1e9

    def forward_stack(self, xs: Sequence[torch.Tensor], measure: bool = False, prefetch: bool = True,
                      outputs: Optional[list] = None):
        """One pass of the token batch through all layers.  xs[l]: [T][d] bf16 on the device.
        Returns the picks of every layer (host arrays).  With measure=True the library brackets
        every acquire by two events on the compute stream (emoe_cache_set_timing): their distance is
        the time the compute stream stood still for a load (the exposed copy time).  If `outputs` is a list, every
        layer appends (gates, y) of the batch to it (device copies)."""
        sh, E = self.shape, self.shape.n_experts
        T = xs[0].shape[0]
        cs, cps = self.compute.cuda_stream, self.copy.cuda_stream
        picks = []
        prev = None
        with torch.cuda.stream(self.compute):
            for l in range(self.n_layers):
                bias_ptr, stride = None, 0
                if prev is not None:
                    # routing follows the prior: bias[t] = beta * log(mean of the prior rows of t's previous picks)
                    b = self.beta * np.log(self.prior[prev].mean(axis=1) + 1e-9)
                    self.bias[:T].copy_(torch.from_numpy(b.astype(np.float32)), non_blocking=True)
                    bias_ptr, stride = self.bias.data_ptr(), E
                B.emoe_router_topk(self.ctx, xs[l].data_ptr(), B.DTYPE_BF16, T, sh.d_model, self.Wr[l].data_ptr(), bias_ptr,
                                   stride, E, sh.top_k, B.GATE_SOFTMAX_RENORM if sh.gate_mode == "softmax_renorm" else B.GATE_SOFTMAX,
                                   self.ids.data_ptr(), self.gates.data_ptr(), None, cs)
                ids = self.ids[:T].cpu().numpy()      # the picks decide which experts are needed: read back
                picks.append(ids)
                active = sorted(set(ids.reshape(-1).tolist()))
                if prefetch and l + 1 < self.n_layers:
                    order = B.emoe_rank_experts(self.prior, np.array(active, dtype=np.int32))
                    n = E if T > 1 else self.n_prefetch
                    B.emoe_prefetch_experts(self.ctx, [self.expert_id(l + 1, int(e)) for e in order[:n]], l, cps)
                eids = [self.expert_id(l, e) for e in active]
                B.emoe_cache_set_timing(self.ctx, measure)
                acq = B.emoe_cache_acquire(self.ctx, eids, l, cs, cps)
                by_e = {e: acq[i] for i, e in enumerate(active)}
                first = acq[0]
                table = (B.emoe_expert * E)()
                for e in range(E):
                    # entries of experts nobody picked are never read; they borrow an acquired expert
                    # whole (pointers AND width, so that whatever is derived from an entry stays
                    # inside that expert's slot)
                    src = by_e.get(e, first)
                    table[e].bits = self.bits[e] if e in by_e else self.bits[active[0]]
                    for m in range(3):
                        table[e].packed[m] = src.packed[m]
                        table[e].scales[m] = src.scales[m]
                B.emoe_moe_forward_routed(self.ctx, self.desc, xs[l].data_ptr(), T, self.ids.data_ptr(), self.gates.data_ptr(),
                                          table, self.y.data_ptr(), None, cs)
                B.emoe_cache_release(self.ctx, eids, cs)
                if outputs is not None:
                    outputs.append((self.gates[:T].clone(), self.y[:T].clone()))
                prev = ids
        return picks

    def exposed_ms(self) -> float:
        """Sum of the compute-stream stalls the library measured since the last call (synchronises)."""
        self.compute.synchronize()
        ns = B.emoe_cache_get_stats(self.ctx)["exposed_copy_ns"]
        ms = (ns - self._exposed_ns_seen) * 1e-6
        self._exposed_ns_seen = ns
        return ms
