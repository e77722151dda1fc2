"""ctypes binding of libemoe.so: one Python function per C entry point of include/emoe.h,
same names, argument marshalling only.  Tensors are passed as raw device pointers
(``tensor.data_ptr()``), streams as ``torch.cuda.Stream.cuda_stream`` integers.

There is no fallback: if the library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libemoe.so")

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED = -2
ERR_ALIGNMENT = -3
ERR_WORKSPACE = -4
ERR_CUDA = -5
ERR_DEVICE_CHECK = -6
ERR_CACHE_FULL = -7
ERR_TIMEOUT = -8
ERR_RANGE = -9
EVICT_FORWARD, EVICT_PRINTED, EVICT_LRU, EVICT_LFU, EVICT_FIFO = 0, 1, 2, 3, 4

DTYPE_F32, DTYPE_F16, DTYPE_BF16 = 0, 1, 2
ACT_RELU, ACT_SWIGLU = 0, 1
GATE_SOFTMAX, GATE_SOFTMAX_RENORM = 0, 1
RANGE_SYMMETRIC, RANGE_FULL = 0, 1

EXPORTS = (
    "emoe_create", "emoe_destroy", "emoe_workspace_bytes", "emoe_last_cuda_error", "emoe_device_status",
    "emoe_status_string", "emoe_packed_bytes", "emoe_scales_bytes", "emoe_pack_expert", "emoe_requantize_expert",
    "emoe_pack_expert_mode", "emoe_requantize_expert_mode",
    "emoe_router_topk",
    "emoe_permute", "emoe_moe_forward", "emoe_moe_forward_routed", "emoe_set_ffn_path", "emoe_set_timing",
    "emoe_read_timing", "emoe_moe_forward_routed_static", "emoe_static_device_status", "emoe_set_dependent_launch",
    "emoe_set_fused_projections", "emoe_set_fused_routing", "emoe_set_fused_layer", "emoe_kernels_last_forward", "emoe_set_wait_limit",
    "emoe_debug_expect_extra_completions",
    "emoe_cache_create", "emoe_register_expert", "emoe_prefetch_experts", "emoe_cache_acquire", "emoe_cache_release",
    "emoe_cache_slot_of", "emoe_cache_get_stats", "emoe_cache_set_timing", "emoe_last_expert_counts", "emoe_policy_create", "emoe_policy_destroy", "emoe_policy_register",
    "emoe_policy_prefetch", "emoe_policy_acquire", "emoe_policy_release", "emoe_policy_get_stats", "emoe_rank_experts",
    "emoe_build_profile2", "emoe_rank_experts2",
)


class EmoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class emoe_expert(ctypes.Structure):
    _fields_ = [("bits", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("packed", ctypes.c_void_p * 3), ("scales", ctypes.c_void_p * 3)]


class emoe_layer_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("d_model", "d_ff", "n_experts", "top_k", "act", "gate_mode", "group", "scale_dtype", "act_dtype")]


class emoe_cache_stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in
                ("hits", "misses", "prefetch_hits", "prefetched", "prefetch_redundant", "prefetch_refused", "evictions",
                 "bytes_copied", "exposed_copy_ns", "timed_acquires")]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it is missing (no CPU fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} not found: build it with `python -m paper_2308_14352_b200.build` "
                "(needs nvcc); this package has no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.emoe_create.restype = vp
        L.emoe_create.argtypes = [i32, sz, ctypes.POINTER(ctypes.c_int)]
        L.emoe_destroy.argtypes = [vp]
        L.emoe_workspace_bytes.restype = sz
        L.emoe_workspace_bytes.argtypes = [ctypes.POINTER(emoe_layer_desc), i32]
        L.emoe_last_cuda_error.argtypes = [vp]
        L.emoe_device_status.argtypes = [vp, vp]
        L.emoe_status_string.restype = ctypes.c_char_p
        L.emoe_status_string.argtypes = [i32]
        L.emoe_packed_bytes.restype = sz
        L.emoe_packed_bytes.argtypes = [i32, i32, i32]
        L.emoe_scales_bytes.restype = sz
        L.emoe_scales_bytes.argtypes = [i32, i32, i32, i32]
        L.emoe_pack_expert.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp]
        L.emoe_requantize_expert.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp]
        L.emoe_pack_expert_mode.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp]
        L.emoe_requantize_expert_mode.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, vp, vp]
        L.emoe_router_topk.argtypes = [vp, vp, i32, i32, i32, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp]
        L.emoe_permute.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp, vp]
        L.emoe_moe_forward.argtypes = [vp, ctypes.POINTER(emoe_layer_desc), vp, i32, vp, vp, i32,
                                       ctypes.POINTER(emoe_expert), vp, vp, vp, vp, vp]
        L.emoe_moe_forward_routed.argtypes = [vp, ctypes.POINTER(emoe_layer_desc), vp, i32, vp, vp,
                                              ctypes.POINTER(emoe_expert), vp, vp, vp]
        L.emoe_set_ffn_path.argtypes = [vp, i32]
        L.emoe_set_timing.argtypes = [vp, i32]
        L.emoe_set_dependent_launch.argtypes = [vp, i32]
        L.emoe_set_fused_projections.argtypes = [vp, i32]
        L.emoe_set_fused_routing.argtypes = [vp, i32]
        L.emoe_set_fused_layer.argtypes = [vp, i32]
        L.emoe_kernels_last_forward.argtypes = [vp]
        L.emoe_set_wait_limit.argtypes = [vp, ctypes.c_uint]
        L.emoe_debug_expect_extra_completions.argtypes = [vp, i32]
        i64 = ctypes.c_int64
        L.emoe_cache_create.argtypes = [vp, i32, sz, i32, i32]
        L.emoe_register_expert.argtypes = [vp, i64, i32, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(sz)]
        L.emoe_prefetch_experts.argtypes = [vp, ctypes.POINTER(i64), i32, i32, vp]
        L.emoe_cache_acquire.argtypes = [vp, ctypes.POINTER(i64), i32, i32, vp, vp, ctypes.POINTER(emoe_expert)]
        L.emoe_cache_release.argtypes = [vp, ctypes.POINTER(i64), i32, vp]
        L.emoe_cache_slot_of.argtypes = [vp, i64]
        L.emoe_cache_get_stats.argtypes = [vp, ctypes.POINTER(emoe_cache_stats)]
        L.emoe_cache_set_timing.argtypes = [vp, i32]
        L.emoe_last_expert_counts.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), i32, vp]
        L.emoe_policy_create.restype = vp
        L.emoe_policy_create.argtypes = [i32, i32, i32]
        L.emoe_policy_destroy.restype = None
        L.emoe_policy_destroy.argtypes = [vp]
        L.emoe_policy_register.argtypes = [vp, i64, i32, i64]
        L.emoe_policy_prefetch.argtypes = [vp, i64, i32, ctypes.POINTER(i64)]
        L.emoe_policy_acquire.argtypes = [vp, i64, i32, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(i64)]
        L.emoe_policy_release.argtypes = [vp, i64]
        L.emoe_policy_get_stats.argtypes = [vp, ctypes.POINTER(emoe_cache_stats)]
        L.emoe_rank_experts.argtypes = [ctypes.POINTER(ctypes.c_float), i32, ctypes.POINTER(ctypes.c_int32), i32,
                                        ctypes.POINTER(ctypes.c_int32)]
        pf, pi = ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)
        L.emoe_build_profile2.argtypes = [pi, i32, i32, i32, i32, pf]
        L.emoe_rank_experts2.argtypes = [pf, i32, pi, i32, pi, i32, pi]
        L.emoe_moe_forward_routed_static.argtypes = [i32, ctypes.POINTER(emoe_layer_desc), vp, i32, vp, vp,
                                                     ctypes.POINTER(emoe_expert), vp, vp]
        L.emoe_static_device_status.argtypes = [i32, vp]
        L.emoe_read_timing.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float),
                                       ctypes.POINTER(ctypes.c_int)]
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != OK:
        raise EmoeError(status, where)


def status_string(status: int) -> str:
    return lib().emoe_status_string(status).decode()


def emoe_create(device: int, workspace_bytes: int) -> int:
    st = ctypes.c_int(0)
    ctx = lib().emoe_create(device, workspace_bytes, ctypes.byref(st))
    if not ctx:
        raise EmoeError(st.value, "emoe_create")
    return ctx


def emoe_destroy(ctx: int) -> None:
    _check(lib().emoe_destroy(ctx), "emoe_destroy")


def emoe_workspace_bytes(desc: emoe_layer_desc, T: int) -> int:
    return int(lib().emoe_workspace_bytes(ctypes.byref(desc), T))


def emoe_last_cuda_error(ctx: int) -> int:
    return int(lib().emoe_last_cuda_error(ctx))


def emoe_device_status(ctx: int, stream: int = 0) -> int:
    return int(lib().emoe_device_status(ctx, stream))


def emoe_packed_bytes(N: int, K: int, bits: int) -> int:
    return int(lib().emoe_packed_bytes(N, K, bits))


def emoe_scales_bytes(N: int, K: int, group: int, scale_dtype: int) -> int:
    return int(lib().emoe_scales_bytes(N, K, group, scale_dtype))


def emoe_pack_expert(ctx, W_ptr, N, K, bits, group, scale_dtype, out_packed_ptr, out_scales_ptr, stream=0) -> None:
    _check(lib().emoe_pack_expert(ctx, W_ptr, N, K, bits, group, scale_dtype, out_packed_ptr, out_scales_ptr, stream),
           "emoe_pack_expert")


def emoe_pack_expert_mode(ctx, W_ptr, N, K, bits, group, scale_dtype, range_mode, out_packed_ptr, out_scales_ptr,
                          stream=0) -> None:
    _check(lib().emoe_pack_expert_mode(ctx, W_ptr, N, K, bits, group, scale_dtype, range_mode, out_packed_ptr,
                                       out_scales_ptr, stream), "emoe_pack_expert_mode")


def emoe_requantize_expert_mode(ctx, in_packed_ptr, in_scales_ptr, N, K, bits_in, bits_out, group, scale_dtype,
                                range_mode, out_packed_ptr, out_scales_ptr, stream=0) -> None:
    _check(lib().emoe_requantize_expert_mode(ctx, in_packed_ptr, in_scales_ptr, N, K, bits_in, bits_out, group,
                                             scale_dtype, range_mode, out_packed_ptr, out_scales_ptr, stream),
           "emoe_requantize_expert_mode")


def emoe_requantize_expert(ctx, in_packed_ptr, in_scales_ptr, N, K, bits_in, bits_out, group, scale_dtype,
                           out_packed_ptr, out_scales_ptr, stream=0) -> None:
    _check(lib().emoe_requantize_expert(ctx, in_packed_ptr, in_scales_ptr, N, K, bits_in, bits_out, group, scale_dtype,
                                        out_packed_ptr, out_scales_ptr, stream), "emoe_requantize_expert")


def emoe_router_topk(ctx, x_ptr, act_dtype, T, d, router_W_ptr, bias_ptr, bias_token_stride, E, top_k, gate_mode,
                     out_ids_ptr, out_gates_ptr, out_logits_ptr=None, stream=0) -> None:
    _check(lib().emoe_router_topk(ctx, x_ptr, act_dtype, T, d, router_W_ptr, bias_ptr, bias_token_stride, E, top_k,
                                  gate_mode, out_ids_ptr, out_gates_ptr, out_logits_ptr, stream), "emoe_router_topk")


def emoe_permute(ctx, ids_ptr, n_pairs, E, out_counts_ptr, out_off_ptr, out_perm_ptr, out_slot_of_pair_ptr=None,
                 stream=0) -> None:
    _check(lib().emoe_permute(ctx, ids_ptr, n_pairs, E, out_counts_ptr, out_off_ptr, out_perm_ptr,
                              out_slot_of_pair_ptr, stream), "emoe_permute")


def make_expert_table(entries: Sequence[tuple]):
    """entries[e] = (bits, [packed ptrs], [scale ptrs]) -> ctypes array of emoe_expert."""
    tab = (emoe_expert * len(entries))()
    for e, (bits, packed, scales) in enumerate(entries):
        tab[e].bits = bits
        tab[e].reserved = 0
        for m in range(3):
            tab[e].packed[m] = packed[m] if m < len(packed) else None
            tab[e].scales[m] = scales[m] if m < len(scales) else None
    return tab


def emoe_moe_forward(ctx, desc: emoe_layer_desc, x_ptr, T, router_W_ptr, bias_ptr, bias_token_stride, expert_table,
                     y_ptr, out_ids_ptr=None, out_gates_ptr=None, out_perm_ptr=None, stream=0) -> None:
    _check(lib().emoe_moe_forward(ctx, ctypes.byref(desc), x_ptr, T, router_W_ptr, bias_ptr, bias_token_stride,
                                  expert_table, y_ptr, out_ids_ptr, out_gates_ptr, out_perm_ptr, stream),
           "emoe_moe_forward")


def emoe_moe_forward_routed(ctx, desc: emoe_layer_desc, x_ptr, T, ids_ptr, gates_ptr, expert_table, y_ptr,
                            out_perm_ptr=None, stream=0) -> None:
    _check(lib().emoe_moe_forward_routed(ctx, ctypes.byref(desc), x_ptr, T, ids_ptr, gates_ptr, expert_table, y_ptr,
                                         out_perm_ptr, stream), "emoe_moe_forward_routed")


def emoe_set_ffn_path(ctx, path: int) -> None:
    _check(lib().emoe_set_ffn_path(ctx, path), "emoe_set_ffn_path")


def emoe_set_timing(ctx, enabled: bool) -> None:
    _check(lib().emoe_set_timing(ctx, int(enabled)), "emoe_set_timing")


def emoe_read_timing(ctx):
    """(first-projection ms, second-projection ms, forward calls covered) since the last read."""
    a, b, n = ctypes.c_float(0), ctypes.c_float(0), ctypes.c_int(0)
    _check(lib().emoe_read_timing(ctx, ctypes.byref(a), ctypes.byref(b), ctypes.byref(n)), "emoe_read_timing")
    return a.value, b.value, n.value


def emoe_moe_forward_routed_static(device: int, desc: emoe_layer_desc, x_ptr, T, ids_ptr, gates_ptr, expert_table,
                                   y_ptr, stream=0) -> None:
    """Routed forward without a context and without any device allocation (fixed 8 MiB scratch
    inside the library; T * top_k <= 64).  For callers that may not allocate."""
    _check(lib().emoe_moe_forward_routed_static(device, ctypes.byref(desc), x_ptr, T, ids_ptr, gates_ptr,
                                                expert_table, y_ptr, stream), "emoe_moe_forward_routed_static")


def emoe_static_device_status(device: int, stream: int = 0) -> int:
    """Status word of the context-free forward calls enqueued so far on `device` (synchronises)."""
    return int(lib().emoe_static_device_status(device, stream))


def emoe_set_dependent_launch(ctx, enabled: bool) -> None:
    _check(lib().emoe_set_dependent_launch(ctx, int(enabled)), "emoe_set_dependent_launch")


def emoe_set_fused_projections(ctx, enabled: bool) -> None:
    _check(lib().emoe_set_fused_projections(ctx, int(enabled)), "emoe_set_fused_projections")


def emoe_set_fused_routing(ctx, enabled: bool) -> None:
    _check(lib().emoe_set_fused_routing(ctx, int(enabled)), "emoe_set_fused_routing")


def emoe_set_fused_layer(ctx, mode) -> None:
    """0 / False: never; 1 / True: every call inside the limits; 2: the default (one or two pairs)."""
    _check(lib().emoe_set_fused_layer(ctx, int(mode)), "emoe_set_fused_layer")


def emoe_set_wait_limit(ctx, polls: int) -> None:
    _check(lib().emoe_set_wait_limit(ctx, polls), "emoe_set_wait_limit")


def emoe_debug_expect_extra_completions(ctx, extra: int) -> None:
    _check(lib().emoe_debug_expect_extra_completions(ctx, extra), "emoe_debug_expect_extra_completions")


def emoe_kernels_last_forward(ctx) -> int:
    return int(lib().emoe_kernels_last_forward(ctx))


# ---- expert cache and prefetch ------------------------------------------------------------------
def _i64_array(ids):
    arr = (ctypes.c_int64 * len(ids))(*[int(i) for i in ids])
    return arr


def emoe_cache_create(ctx, n_slots: int, slot_bytes: int, n_layers: int, policy: int = EVICT_FORWARD) -> None:
    _check(lib().emoe_cache_create(ctx, n_slots, slot_bytes, n_layers, policy), "emoe_cache_create")


def emoe_register_expert(ctx, expert_id: int, layer: int, bits: int, host_packed, host_scales, nbytes) -> None:
    """host_packed / host_scales: 3 host addresses each (0 for an absent matrix); nbytes: 6 sizes."""
    vp = ctypes.c_void_p
    hp = (vp * 3)(*[vp(int(a)) if a else vp(None) for a in host_packed])
    hs = (vp * 3)(*[vp(int(a)) if a else vp(None) for a in host_scales])
    nb = (ctypes.c_size_t * 6)(*[int(b) for b in nbytes])
    _check(lib().emoe_register_expert(ctx, expert_id, layer, bits, hp, hs, nb), "emoe_register_expert")


def emoe_prefetch_experts(ctx, ids, current_layer: int, copy_stream: int) -> None:
    if len(ids) == 0:
        return
    _check(lib().emoe_prefetch_experts(ctx, _i64_array(ids), len(ids), current_layer, copy_stream), "emoe_prefetch_experts")


def emoe_cache_acquire(ctx, ids, current_layer: int, compute_stream: int, copy_stream: int):
    out = (emoe_expert * len(ids))()
    _check(lib().emoe_cache_acquire(ctx, _i64_array(ids), len(ids), current_layer, compute_stream, copy_stream, out),
           "emoe_cache_acquire")
    return out


def emoe_cache_release(ctx, ids, compute_stream: int) -> None:
    _check(lib().emoe_cache_release(ctx, _i64_array(ids), len(ids), compute_stream), "emoe_cache_release")


def emoe_cache_slot_of(ctx, expert_id: int) -> int:
    return int(lib().emoe_cache_slot_of(ctx, expert_id))


def emoe_cache_get_stats(ctx) -> dict:
    st = emoe_cache_stats()
    _check(lib().emoe_cache_get_stats(ctx, ctypes.byref(st)), "emoe_cache_get_stats")
    return st.as_dict()


def emoe_cache_set_timing(ctx, enabled: bool) -> None:
    _check(lib().emoe_cache_set_timing(ctx, int(enabled)), "emoe_cache_set_timing")


def emoe_last_expert_counts(ctx, n_experts: int, stream=0):
    import numpy as np

    out = np.empty(n_experts, dtype=np.int32)
    _check(lib().emoe_last_expert_counts(ctx, out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), n_experts, stream),
           "emoe_last_expert_counts")
    return out


def emoe_policy_create(n_slots: int, n_layers: int, policy: int = EVICT_FORWARD):
    h = lib().emoe_policy_create(n_slots, n_layers, policy)
    if not h:
        raise EmoeError(ERR_INVALID_ARG, "emoe_policy_create")
    return h


def emoe_policy_destroy(h) -> None:
    lib().emoe_policy_destroy(h)


def emoe_policy_register(h, expert_id: int, layer: int, nbytes: int = 0) -> None:
    _check(lib().emoe_policy_register(h, expert_id, layer, nbytes), "emoe_policy_register")


def emoe_policy_prefetch(h, expert_id: int, current_layer: int):
    """-> (slot the load goes to or -1, id that was evicted or -1)"""
    ev = ctypes.c_int64(-1)
    s = lib().emoe_policy_prefetch(h, expert_id, current_layer, ctypes.byref(ev))
    if s == -2:
        raise EmoeError(ERR_INVALID_ARG, "emoe_policy_prefetch")
    return int(s), int(ev.value)


def emoe_policy_acquire(h, expert_id: int, current_layer: int):
    """-> (slot or -1 when every slot is protected, loaded now?, id that was evicted or -1)"""
    ev = ctypes.c_int64(-1)
    loaded = ctypes.c_int(0)
    s = lib().emoe_policy_acquire(h, expert_id, current_layer, ctypes.byref(loaded), ctypes.byref(ev))
    if s == -2:
        raise EmoeError(ERR_INVALID_ARG, "emoe_policy_acquire")
    return int(s), bool(loaded.value), int(ev.value)


def emoe_policy_release(h, expert_id: int) -> int:
    return int(lib().emoe_policy_release(h, expert_id))


def emoe_policy_get_stats(h) -> dict:
    st = emoe_cache_stats()
    _check(lib().emoe_policy_get_stats(h, ctypes.byref(st)), "emoe_policy_get_stats")
    return st.as_dict()


def emoe_rank_experts(prior, prev_ids):
    import numpy as np

    prior = np.ascontiguousarray(prior, dtype=np.float32)
    prev = np.ascontiguousarray(prev_ids, dtype=np.int32).reshape(-1)
    E = prior.shape[0]
    out = np.empty(E, dtype=np.int32)
    _check(lib().emoe_rank_experts(prior.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), E,
                                   prev.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), len(prev),
                                   out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))), "emoe_rank_experts")
    return out


def emoe_build_profile2(trace, n_experts: int):
    """trace: int array [n_tokens][n_layers][top_k]; returns float32 [n_layers][E][E][E]."""
    import numpy as np

    tr = np.ascontiguousarray(trace, dtype=np.int32)
    n_tokens, n_layers, top_k = tr.shape
    out = np.empty((n_layers, n_experts, n_experts, n_experts), dtype=np.float32)
    _check(lib().emoe_build_profile2(tr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), n_tokens, n_layers, top_k,
                                     n_experts, out.ctypes.data_as(ctypes.POINTER(ctypes.c_float))),
           "emoe_build_profile2")
    return out


def emoe_rank_experts2(prior2_layer, prev2_ids, prev1_ids):
    import numpy as np

    tab = np.ascontiguousarray(prior2_layer, dtype=np.float32)
    p2 = np.ascontiguousarray(prev2_ids, dtype=np.int32).reshape(-1)
    p1 = np.ascontiguousarray(prev1_ids, dtype=np.int32).reshape(-1)
    E = tab.shape[0]
    out = np.empty(E, dtype=np.int32)
    pi = ctypes.POINTER(ctypes.c_int32)
    _check(lib().emoe_rank_experts2(tab.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), E, p2.ctypes.data_as(pi), len(p2),
                                    p1.ctypes.data_as(pi), len(p1), out.ctypes.data_as(pi)), "emoe_rank_experts2")
    return out
