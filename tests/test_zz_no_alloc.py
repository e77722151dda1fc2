"""GPU test of emoe_moe_forward_routed_static, the entry point for callers that may not
allocate device memory (a framework that owns the device heap, a plug-in with a fixed pool,
a latency-critical loop).  It takes no context and keeps its intermediates in a fixed array
inside the library, so this test builds the inputs with plain torch tensors, never creates an
emoe context for the call under test, and checks the result against the CPU checker and
against the ordinary emoe_moe_forward_routed on the same inputs.  Two calls in a row with different inputs show
that what the first call left in the shared array does not leak into the second.

The file name sorts last on purpose: a run that stops at the first failure has then already
run every other test."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2308_14352_b200 import binding as B, inputs, layer
from tests.helpers import oracle_pack_layer, rel_to_max

pytestmark = pytest.mark.gpu


def _case(shape, bits, T, seed):
    W = inputs.expert_set(seed, 0, shape)
    x = inputs.activations(seed, 0, T, shape.d_model, shape.act_dtype)
    rng = np.random.default_rng(seed)
    ids = np.stack([rng.permutation(shape.n_experts)[: shape.top_k] for _ in range(T)]).astype(np.int32)
    gates = rng.random((T, shape.top_k)).astype(np.float32)
    return W, x, ids, gates


@pytest.mark.parametrize("act,adt,group,sdt", [("swiglu", "bf16", 128, "f16"), ("relu", "f32", 0, "f32")])
def test_static_entry_point_matches_the_context_one_twice_in_a_row(act, adt, group, sdt):
    shape = inputs.LayerShape(256, 512, 4, 2, act, "softmax_renorm", group, sdt, adt)
    bits = [4, 2, 8, 4]
    tol = 2e-3 if adt == "bf16" else 1e-5
    with layer.MoELayer(shape, bits, max_tokens=16) as moe:        # only to pack weights and for the reference
        W, _, _, _ = _case(shape, bits, 1, 40)
        moe.pack_from_host(W)
        packed, scales = oracle_pack_layer(W, shape, bits)
        for call, (T, seed) in enumerate([(16, 41), (5, 42)]):
            _, x, ids, gates = _case(shape, bits, T, seed)
            y_ref, _ = moe.forward_routed(x, ids, gates)
            xd = moe.to_device_x(x)
            idd = torch.from_numpy(ids).cuda()
            gd = torch.from_numpy(gates).cuda()
            y = torch.full((T, shape.d_model), float("nan"), dtype=torch.float32, device="cuda")
            B.emoe_moe_forward_routed_static(0, moe.desc, xd.data_ptr(), T, idd.data_ptr(), gd.data_ptr(), moe.table,
                                             y.data_ptr(), 0)
            torch.cuda.synchronize()
            y = y.cpu().numpy()
            assert np.isfinite(y).all()
            y_cpu = oracle.moe_ffn_combine(x, shape.d_ff, shape.act, shape.group, adt == "bf16", bits, packed, scales,
                                           ids, gates)
            assert rel_to_max(y, y_cpu) <= tol, (call, rel_to_max(y, y_cpu))     # against the CPU checker
            err = np.abs(y - y_ref).max() / np.abs(y_ref).max()
            assert err <= tol, (call, err)                                       # against the context entry point
            assert B.emoe_static_device_status(0) == B.OK


def test_static_entry_point_reports_an_expert_id_out_of_range():
    """Ids outside [0, E) are dropped (their terms are missing from y) and leave a flag that the
    status call returns; the next call clears it."""
    shape = inputs.LayerShape(256, 512, 4, 2, "relu", "softmax", 128, "f16", "bf16")
    bits = [4, 2, 8, 4]
    with layer.MoELayer(shape, bits, max_tokens=8) as moe:
        W, x, ids, gates = _case(shape, bits, 6, 43)
        moe.pack_from_host(W)
        packed, scales = oracle_pack_layer(W, shape, bits)
        xd = moe.to_device_x(x)
        gd = torch.from_numpy(gates).cuda()
        y = torch.zeros((6, shape.d_model), dtype=torch.float32, device="cuda")
        bad = ids.copy()
        bad[2, 1] = 7                      # E = 4
        idd = torch.from_numpy(bad).cuda()
        B.emoe_moe_forward_routed_static(0, moe.desc, xd.data_ptr(), 6, idd.data_ptr(), gd.data_ptr(), moe.table,
                                         y.data_ptr(), 0)
        assert B.emoe_static_device_status(0) == B.ERR_DEVICE_CHECK
        # the dropped pair contributes nothing: same as a zero gate on a valid expert
        ids_eq, gates_eq = ids.copy(), gates.copy()
        gates_eq[2, 1] = 0.0
        y_cpu = oracle.moe_ffn_combine(x, shape.d_ff, "relu", 128, True, bits, packed, scales, ids_eq, gates_eq)
        assert rel_to_max(y.cpu().numpy(), y_cpu) <= 2e-3
        idd = torch.from_numpy(ids).cuda()
        B.emoe_moe_forward_routed_static(0, moe.desc, xd.data_ptr(), 6, idd.data_ptr(), gd.data_ptr(), moe.table,
                                         y.data_ptr(), 0)
        assert B.emoe_static_device_status(0) == B.OK


def test_static_entry_point_rejects_what_does_not_fit():
    lib = B.lib()
    shape = inputs.LayerShape(256, 512, 4, 2, "relu", "softmax", 128, "f16", "bf16")
    with layer.MoELayer(shape, [4, 2, 8, 4], max_tokens=4) as moe:
        x = torch.zeros(64, 256, dtype=torch.bfloat16, device="cuda")
        ids = torch.zeros(64, 2, dtype=torch.int32, device="cuda")
        g = torch.zeros(64, 2, dtype=torch.float32, device="cuda")
        y = torch.zeros(64, 256, device="cuda")
        call = lambda desc, T: lib.emoe_moe_forward_routed_static(
            0, ctypes.byref(desc), x.data_ptr(), T, ids.data_ptr(), g.data_ptr(), moe.table, y.data_ptr(), None)
        assert call(moe.desc, 33) == B.ERR_WORKSPACE          # 66 pairs > 64
        assert call(moe.desc, 0) == B.ERR_INVALID_ARG
        big = layer.make_desc(inputs.LayerShape(8192, 65536, 4, 2, "relu", "softmax", 128, "f16", "bf16"))
        assert call(big, 32) == B.ERR_WORKSPACE               # hidden vectors alone exceed the fixed array
        assert call(moe.desc, 32) == B.OK
        torch.cuda.synchronize()
