"""CPU checker for the sparse-MoE layer on mixed-bitwidth packed experts.

TEST INFRASTRUCTURE ONLY: a thin ctypes wrapper over ``emoe_oracle.cpp`` (plain C++,
fp64 accumulation).  The tests compare the GPU library with it, and the benchmark may
time it as a CPU baseline; the product package never imports it, and it imports nothing
from the product package.

Every function below only marshals numpy arrays; the arithmetic is in the C++ file,
which cites the passages of the paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "emoe_oracle.cpp")
_LIB = os.path.join(_HERE, "libemoe_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker with g++ (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["g++", "-O2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-o", _LIB, _SRC])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_round_f16.restype = ctypes.c_float
        _lib.orc_round_f16.argtypes = [ctypes.c_float]
        _lib.orc_round_bf16.restype = ctypes.c_double
        _lib.orc_round_bf16.argtypes = [ctypes.c_double]
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(_load().orc_num_threads())


def round_f16(v: float) -> float:
    return float(_load().orc_round_f16(ctypes.c_float(v)))


def round_bf16(v: float) -> float:
    return float(_load().orc_round_bf16(ctypes.c_double(v)))


def quantize(W: np.ndarray, bits: int, group: int, scale_dtype: str, full_range: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """Codes q[N][K] (int8) and stored scales [N][K/G] (fp32 values).  full_range: the reading of
    Section 3.2's "range expressible by the bitwidth" that uses every code of the field
    (-2^(b-1) .. 2^(b-1)-1, scale = max-abs / 2^(b-1)) instead of the symmetric one."""
    W = _c(W, np.float32)
    N, K = W.shape
    G = group if group > 0 else K
    q = np.empty((N, K), dtype=np.int8)
    s = np.empty((N, K // G), dtype=np.float32)
    rc = _load().orc_quantize_mode(_p(W), N, K, bits, group, int(scale_dtype == "f16"), int(full_range), _p(q), _p(s))
    if rc != 0:
        raise ValueError(f"orc_quantize_mode failed ({rc})")
    return q, s


def pack(q: np.ndarray, bits: int) -> np.ndarray:
    q = _c(q, np.int8)
    N, K = q.shape
    out = np.empty((N, K * bits // 8), dtype=np.uint8)
    rc = _load().orc_pack(_p(q), N, K, bits, _p(out))
    if rc != 0:
        raise ValueError(f"orc_pack failed ({rc})")
    return out


def unpack(packed: np.ndarray, K: int, bits: int) -> np.ndarray:
    packed = _c(packed, np.uint8)
    N = packed.shape[0]
    q = np.empty((N, K), dtype=np.int8)
    rc = _load().orc_unpack(_p(packed), N, K, bits, _p(q))
    if rc != 0:
        raise ValueError(f"orc_unpack failed ({rc})")
    return q


def dequantize(packed: np.ndarray, scales: np.ndarray, K: int, bits: int, group: int) -> np.ndarray:
    packed = _c(packed, np.uint8)
    scales = _c(scales, np.float32)
    N = packed.shape[0]
    Wt = np.empty((N, K), dtype=np.float64)
    rc = _load().orc_dequantize(_p(packed), _p(scales), N, K, bits, group, _p(Wt))
    if rc != 0:
        raise ValueError(f"orc_dequantize failed ({rc})")
    return Wt


def pack_expert(W: np.ndarray, bits: int, group: int, scale_dtype: str, full_range: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """quantise + pack one matrix: (packed bytes [N][K*b/8], stored scales fp32 [N][K/G])."""
    q, s = quantize(W, bits, group, scale_dtype, full_range)
    return pack(q, bits), s


def requantize(packed: np.ndarray, scales: np.ndarray, K: int, bits_in: int, bits_out: int, group: int,
               scale_dtype: str, full_range: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """An expert matrix stored at `bits_in` moved to `bits_out` without the original weights
    (paper Section 3.2: the bitwidth selection lowers the width of chosen experts): decompress
    to FP32 as the paper does (w~ = q * s, rounded once to fp32; exact with fp16 scales, which
    have 11 significant bits against the codes' 8), then the same channel-wise linear
    quantisation as for an fp32 matrix.  Returns (packed bytes, stored scales)."""
    Wt = dequantize(packed, scales, K, bits_in, group)
    return pack_expert(Wt.astype(np.float32), bits_out, group, scale_dtype, full_range)


def scales_storage(scales: np.ndarray, scale_dtype: str) -> np.ndarray:
    """The scale channel in its storage type (values are already representable)."""
    return scales.astype(np.float16) if scale_dtype == "f16" else scales.astype(np.float32)


def route(x: np.ndarray, Wr: np.ndarray, bias: Optional[np.ndarray], top_k: int, renorm: bool):
    """ids[T][k] int32, gates[T][k] fp32, logits[T][E] fp32."""
    x = _c(x, np.float32)
    Wr = _c(Wr, np.float32)
    T, d = x.shape
    E = Wr.shape[1]
    stride = 0
    if bias is not None:
        bias = _c(bias, np.float32)
        stride = E if bias.ndim == 2 else 0
    ids = np.empty((T, top_k), dtype=np.int32)
    gates = np.empty((T, top_k), dtype=np.float32)
    logits = np.empty((T, E), dtype=np.float32)
    rc = _load().orc_route(_p(x), T, d, _p(Wr), _p(bias), stride, E, top_k, int(renorm), _p(ids), _p(gates), _p(logits))
    if rc != 0:
        raise ValueError(f"orc_route failed ({rc})")
    return ids, gates, logits


def permute(ids: np.ndarray, E: int):
    """counts[E], off[E+1], perm[T*k] of the stable sort of pair indices by expert."""
    flat = _c(ids, np.int32).reshape(-1)
    counts = np.empty(E, dtype=np.int32)
    off = np.empty(E + 1, dtype=np.int32)
    perm = np.empty(flat.size, dtype=np.int32)
    rc = _load().orc_permute(_p(flat), flat.size, E, _p(counts), _p(off), _p(perm))
    if rc != 0:
        raise ValueError(f"orc_permute failed ({rc})")
    return counts, off, perm


def _ptr_table(arrs: Sequence[Sequence[np.ndarray]], dtype):
    """E*3 pointer table (entry e*3+m) plus the arrays kept alive."""
    keep = []
    tab = (ctypes.c_void_p * (len(arrs) * 3))()
    for e, mats in enumerate(arrs):
        for m, a in enumerate(mats):
            a = _c(a, dtype)
            keep.append(a)
            tab[e * 3 + m] = a.ctypes.data
    return tab, keep


def moe_ffn_combine(x: np.ndarray, d_ff: int, act: str, group: int, hidden_bf16: bool,
                    bits: Sequence[int], packed: Sequence[Sequence[np.ndarray]],
                    scales: Sequence[Sequence[np.ndarray]], ids: np.ndarray, gates: np.ndarray,
                    want_intermediates: bool = False):
    """Expert FFNs on the dequantised weights and the weighted combine.
    packed[e][m], scales[e][m]: matrix m of expert e.  Returns y (and h, o if asked)."""
    x = _c(x, np.float32)
    T, d = x.shape
    E = len(bits)
    ids = _c(ids, np.int32).reshape(T, -1)
    gates = _c(gates, np.float32).reshape(T, -1)
    k = ids.shape[1]
    ptab, keep1 = _ptr_table(packed, np.uint8)
    stab, keep2 = _ptr_table(scales, np.float32)
    bits_a = _c(bits, np.int32)
    y = np.empty((T, d), dtype=np.float32)
    h = np.zeros((T * k, d_ff), dtype=np.float32) if want_intermediates else None
    o = np.zeros((T * k, d), dtype=np.float64) if want_intermediates else None
    rc = _load().orc_moe_ffn_combine(_p(x), T, d, d_ff, E, k, int(act == "swiglu"), group, int(hidden_bf16),
                                     _p(bits_a), ptab, stab, _p(ids), _p(gates), _p(y), _p(h), _p(o))
    if rc != 0:
        raise ValueError(f"orc_moe_ffn_combine failed ({rc})")
    del keep1, keep2
    return (y, h, o) if want_intermediates else y


def moe_forward(x, Wr, bias, top_k: int, renorm: bool, d_ff: int, act: str, group: int, hidden_bf16: bool,
                bits, packed, scales):
    """route -> permute -> expert FFNs -> combine.  Returns (y, ids, gates)."""
    ids, gates, _ = route(x, Wr, bias, top_k, renorm)
    y = moe_ffn_combine(x, d_ff, act, group, hidden_bf16, bits, packed, scales, ids, gates)
    return y, ids, gates


def hidden_for_pair(xt: np.ndarray, d_ff: int, act: str, group: int, hidden_bf16: bool, bits: int,
                    packed3: Sequence[np.ndarray], scales3: Sequence[np.ndarray]) -> np.ndarray:
    """Hidden vector h[f] (fp64 values) of one (token, expert) pair."""
    xt = _c(xt, np.float32)
    ptab, k1 = _ptr_table([packed3], np.uint8)
    stab, k2 = _ptr_table([scales3], np.float32)
    h = np.empty(d_ff, dtype=np.float64)
    rc = _load().orc_hidden_for_pair(_p(xt), xt.size, d_ff, int(act == "swiglu"), group, int(hidden_bf16), bits,
                                     ptab, stab, _p(h))
    if rc != 0:
        raise ValueError(f"orc_hidden_for_pair failed ({rc})")
    return h


def output_channels(h: np.ndarray, group: int, bits: int, packed_out: np.ndarray, scales_out: np.ndarray,
                    channels: Sequence[int]) -> np.ndarray:
    """o[c] = sum_j h[j] * W~out[channels[c]][j]."""
    h = _c(h, np.float64)
    packed_out = _c(packed_out, np.uint8)
    scales_out = _c(scales_out, np.float32)
    ch = _c(channels, np.int32)
    o = np.empty(ch.size, dtype=np.float64)
    rc = _load().orc_output_channels(_p(h), h.size, group, bits, _p(packed_out), _p(scales_out), _p(ch), ch.size, _p(o))
    if rc != 0:
        raise ValueError(f"orc_output_channels failed ({rc})")
    return o
