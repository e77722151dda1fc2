"""Device-memory plumbing around the C ABI: a small holder for one MoE layer's packed
experts and a context, used by the tests and the benchmark.  PyTorch is used here only to
allocate device memory and to move tensors; every step of the computation is a call into
libemoe through ``binding``.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from .inputs import LayerShape

_ACT = {"relu": B.ACT_RELU, "swiglu": B.ACT_SWIGLU}
_GATE = {"softmax": B.GATE_SOFTMAX, "softmax_renorm": B.GATE_SOFTMAX_RENORM}
_SDT = {"f32": B.DTYPE_F32, "f16": B.DTYPE_F16}
_ADT = {"f32": B.DTYPE_F32, "bf16": B.DTYPE_BF16}


def make_desc(shape: LayerShape) -> B.emoe_layer_desc:
    return B.emoe_layer_desc(shape.d_model, shape.d_ff, shape.n_experts, shape.top_k, _ACT[shape.act],
                             _GATE[shape.gate_mode], shape.group, _SDT[shape.scale_dtype], _ADT[shape.act_dtype])


class MoELayer:
    """Packed experts of one layer on one GPU plus an emoe context sized for `max_tokens`."""

    def __init__(self, shape: LayerShape, bits: Sequence[int], device: int = 0, max_tokens: int = 64,
                 ctx: Optional[int] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("MoELayer needs a CUDA device: there is no CPU path")
        B.lib()
        self.shape = shape
        self.bits = list(bits)
        assert len(self.bits) == shape.n_experts
        self.device = torch.device("cuda", device)
        self.desc = make_desc(shape)
        self._own_ctx = ctx is None
        torch.cuda.set_device(self.device)
        torch.cuda.init()
        torch.zeros(1, device=self.device)  # make sure the primary context exists
        self.max_tokens = max_tokens
        self.ctx = ctx if ctx is not None else B.emoe_create(device, B.emoe_workspace_bytes(self.desc, max_tokens))
        self.packed: List[List[torch.Tensor]] = []
        self.scales: List[List[torch.Tensor]] = []
        sdt = torch.float16 if shape.scale_dtype == "f16" else torch.float32
        for e in range(shape.n_experts):
            pe, se = [], []
            for m in range(shape.n_matrices):
                N, K = shape.matrix_shape(m)
                G = shape.group if shape.group > 0 else K
                pe.append(torch.empty(N * K * self.bits[e] // 8, dtype=torch.uint8, device=self.device))
                se.append(torch.empty(N * (K // G), dtype=sdt, device=self.device))
            self.packed.append(pe)
            self.scales.append(se)
        self.table = B.make_expert_table([
            (self.bits[e], [t.data_ptr() for t in self.packed[e]], [t.data_ptr() for t in self.scales[e]])
            for e in range(shape.n_experts)])

    # -- context manager ---------------------------------------------------------------------
    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def close(self):
        if self.ctx is not None and self._own_ctx:
            torch.cuda.synchronize(self.device)
            B.emoe_destroy(self.ctx)
        self.ctx = None

    # -- packing -----------------------------------------------------------------------------
    def pack_matrix(self, e: int, m: int, W_dev: torch.Tensor, stream: int = 0, full_range: bool = False) -> None:
        """Quantise + pack one fp32 device matrix [N][K] into this layer's storage."""
        N, K = self.shape.matrix_shape(m)
        assert W_dev.dtype == torch.float32 and W_dev.is_contiguous() and tuple(W_dev.shape) == (N, K)
        B.emoe_pack_expert_mode(self.ctx, W_dev.data_ptr(), N, K, self.bits[e], self.shape.group,
                                _SDT[self.shape.scale_dtype], B.RANGE_FULL if full_range else B.RANGE_SYMMETRIC,
                                self.packed[e][m].data_ptr(), self.scales[e][m].data_ptr(), stream)

    def pack_from_host(self, W: Sequence[Sequence[np.ndarray]], full_range: bool = False) -> None:
        for e in range(self.shape.n_experts):
            for m in range(self.shape.n_matrices):
                w = torch.from_numpy(np.ascontiguousarray(W[e][m], dtype=np.float32)).to(self.device)
                self.pack_matrix(e, m, w, full_range=full_range)
        torch.cuda.synchronize(self.device)

    def change_width(self, e: int, bits_out: int, stream: int = 0, full_range: bool = False) -> None:
        """Moves expert `e` to `bits_out` on the device, from its stored codes and scales (no fp32
        original needed), and points the expert table at the new buffers."""
        b_in = self.bits[e]
        new_packed, new_scales = [], []
        for m in range(self.shape.n_matrices):
            N, K = self.shape.matrix_shape(m)
            p = torch.empty(N * K * bits_out // 8, dtype=torch.uint8, device=self.device)
            s = torch.empty_like(self.scales[e][m])
            B.emoe_requantize_expert_mode(self.ctx, self.packed[e][m].data_ptr(), self.scales[e][m].data_ptr(), N, K,
                                          b_in, bits_out, self.shape.group, _SDT[self.shape.scale_dtype],
                                          B.RANGE_FULL if full_range else B.RANGE_SYMMETRIC, p.data_ptr(),
                                          s.data_ptr(), stream)
            new_packed.append(p)
            new_scales.append(s)
        torch.cuda.synchronize(self.device)  # the old buffers are released below
        self.packed[e], self.scales[e], self.bits[e] = new_packed, new_scales, bits_out
        self.table = B.make_expert_table([
            (self.bits[i], [t.data_ptr() for t in self.packed[i]], [t.data_ptr() for t in self.scales[i]])
            for i in range(self.shape.n_experts)])

    def packed_host(self, e: int, m: int) -> np.ndarray:
        N, K = self.shape.matrix_shape(m)
        return self.packed[e][m].cpu().numpy().reshape(N, K * self.bits[e] // 8)

    def scales_host(self, e: int, m: int) -> np.ndarray:
        N, K = self.shape.matrix_shape(m)
        G = self.shape.group if self.shape.group > 0 else K
        return self.scales[e][m].cpu().numpy().reshape(N, K // G)

    # -- forward -----------------------------------------------------------------------------
    def to_device_x(self, x: np.ndarray) -> torch.Tensor:
        t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(self.device)
        return t.to(torch.bfloat16) if self.shape.act_dtype == "bf16" else t

    def forward_device(self, x_dev: torch.Tensor, Wr_dev: torch.Tensor, bias_dev: Optional[torch.Tensor],
                       y_dev: torch.Tensor, ids_dev=None, gates_dev=None, perm_dev=None, stream: int = 0) -> None:
        T = x_dev.shape[0]
        stride = 0
        if bias_dev is not None and bias_dev.dim() == 2:
            stride = self.shape.n_experts
        B.emoe_moe_forward(self.ctx, self.desc, x_dev.data_ptr(), T, Wr_dev.data_ptr(),
                           None if bias_dev is None else bias_dev.data_ptr(), stride, self.table, y_dev.data_ptr(),
                           None if ids_dev is None else ids_dev.data_ptr(),
                           None if gates_dev is None else gates_dev.data_ptr(),
                           None if perm_dev is None else perm_dev.data_ptr(), stream)

    def forward(self, x: np.ndarray, Wr: np.ndarray, bias: Optional[np.ndarray] = None):
        """Host-array convenience: returns (y, ids, gates, perm) as numpy arrays."""
        T = x.shape[0]
        k = self.shape.top_k
        xd = self.to_device_x(x)
        Wrd = torch.from_numpy(np.ascontiguousarray(Wr, dtype=np.float32)).to(self.device)
        bd = None if bias is None else torch.from_numpy(np.ascontiguousarray(bias, dtype=np.float32)).to(self.device)
        y = torch.empty(T, self.shape.d_model, dtype=torch.float32, device=self.device)
        ids = torch.empty(T, k, dtype=torch.int32, device=self.device)
        gates = torch.empty(T, k, dtype=torch.float32, device=self.device)
        perm = torch.empty(T * k, dtype=torch.int32, device=self.device)
        self.forward_device(xd, Wrd, bd, y, ids, gates, perm)
        torch.cuda.synchronize(self.device)
        st = B.emoe_device_status(self.ctx)
        if st != B.OK:
            raise B.EmoeError(st, "emoe_moe_forward (device check)")
        return y.cpu().numpy(), ids.cpu().numpy(), gates.cpu().numpy(), perm.cpu().numpy()

    def forward_routed(self, x: np.ndarray, ids: np.ndarray, gates: np.ndarray):
        T = x.shape[0]
        xd = self.to_device_x(x)
        idd = torch.from_numpy(np.ascontiguousarray(ids, dtype=np.int32)).to(self.device)
        gd = torch.from_numpy(np.ascontiguousarray(gates, dtype=np.float32)).to(self.device)
        y = torch.empty(T, self.shape.d_model, dtype=torch.float32, device=self.device)
        perm = torch.empty(T * self.shape.top_k, dtype=torch.int32, device=self.device)
        B.emoe_moe_forward_routed(self.ctx, self.desc, xd.data_ptr(), T, idd.data_ptr(), gd.data_ptr(), self.table,
                                  y.data_ptr(), perm.data_ptr(), 0)
        torch.cuda.synchronize(self.device)
        return y.cpu().numpy(), perm.cpu().numpy()
