"""GPU parity: the whole layer (emoe_moe_forward / emoe_moe_forward_routed) against the CPU
checker through the C ABI, on small layers that still span several tiles and ragged tails.
Bars: permutation bit-exact; ids exact outside the 1e-4 logit margin; outputs within
max|y - y_ref| / max|y_ref| <= 2e-3 (bf16 activations) or 1e-5 (fp32 activations).  The
reference is always evaluated with the ids the GPU picked, so a legal tie-break difference
does not leak into the output comparison."""
import numpy as np
import pytest
import torch

import oracle
from paper_2308_14352_b200 import binding as B, inputs, layer
from tests.helpers import check_ids, oracle_pack_layer, output_tolerance, rel_to_max

pytestmark = pytest.mark.gpu


def _run_case(shape, bits, T, seed, path, bias=None, std=0.02, max_tokens=None, fused=True, want_y=False,
              full_range=False):
    W = inputs.expert_set(seed, 0, shape, std)
    x = inputs.activations(seed, 0, T, shape.d_model, shape.act_dtype)
    Wr = inputs.router_weight(seed, 0, shape.d_model, shape.n_experts, std=0.05)
    packed, scales = oracle_pack_layer(W, shape, bits, full_range)
    with layer.MoELayer(shape, bits, max_tokens=max_tokens or T) as moe:
        B.emoe_set_ffn_path(moe.ctx, path)
        B.emoe_set_fused_projections(moe.ctx, fused)
        moe.pack_from_host(W, full_range)
        for e in range(shape.n_experts):          # packed bytes and scales are bit-exact
            for m in range(shape.n_matrices):
                assert np.array_equal(moe.packed_host(e, m), packed[e][m])
                assert np.array_equal(moe.scales_host(e, m).astype(np.float32), scales[e][m])
        y, ids, gates, perm = moe.forward(x, Wr, bias)
    renorm = shape.gate_mode == "softmax_renorm"
    ids_ref, gates_ref, logits_ref = oracle.route(x, Wr, bias, shape.top_k, renorm)
    check_ids(ids, logits_ref, shape.top_k)
    same = np.all(ids == ids_ref, axis=1)
    np.testing.assert_allclose(gates[same], gates_ref[same], rtol=2e-5, atol=1e-7)
    _, _, perm_ref = oracle.permute(ids, shape.n_experts)
    assert np.array_equal(perm, perm_ref)
    y_ref = oracle.moe_ffn_combine(x, shape.d_ff, shape.act, shape.group, shape.act_dtype == "bf16", bits, packed,
                                   scales, ids, gates)
    err = rel_to_max(y, y_ref)
    assert err <= output_tolerance(shape.act_dtype), err
    return (err, y) if want_y else err


GEMV_CASES = [
    # act, act_dtype, group, scale_dtype, d, f, E, k, gate, bits, T
    ("relu", "f32", 0, "f32", 128, 256, 4, 1, "softmax", [8, 4, 2, 4], 9),
    ("relu", "f32", 64, "f32", 192, 320, 3, 2, "softmax_renorm", [2, 8, 4], 7),
    ("swiglu", "f32", 0, "f16", 256, 448, 4, 2, "softmax_renorm", [4, 2, 8, 4], 11),
    ("relu", "bf16", 32, "f16", 64, 160, 5, 1, "softmax", [8, 8, 4, 4, 8], 13),     # shapes the MMA path refuses
    ("swiglu", "bf16", 64, "f16", 192, 320, 2, 2, "softmax", [4, 2], 5),
    ("relu", "bf16", 128, "f16", 256, 512, 4, 1, "softmax", [2, 4, 8, 4], 10),
]


@pytest.mark.parametrize("act,adt,group,sdt,d,f,E,k,gate,bits,T", GEMV_CASES)
def test_forward_cuda_core_path(act, adt, group, sdt, d, f, E, k, gate, bits, T):
    shape = inputs.LayerShape(d, f, E, k, act, gate, group, sdt, adt)
    _run_case(shape, bits, T, seed=21, path=1)


MMA_CASES = [
    ("relu", 128, "f16", 256, 512, 4, 1, "softmax", [2, 4, 8, 4], 10),
    ("relu", 128, "f16", 768, 3072, 8, 1, "softmax", [8, 4, 2, 4, 8, 2, 4, 8], 64),
    ("relu", 0, "f16", 384, 640, 4, 2, "softmax_renorm", [4, 2, 8, 2], 19),        # per-channel scales, ragged row tiles
    ("relu", 128, "f32", 256, 1152, 3, 1, "softmax", [8, 2, 4], 37),                # 37 tokens: two 32-token passes possible
    ("swiglu", 128, "f16", 512, 1408, 4, 2, "softmax_renorm", [4, 8, 2, 4], 16),
    ("swiglu", 256, "f16", 1024, 2560, 8, 2, "softmax_renorm", [4, 4, 8, 2, 4, 8, 2, 4], 33),
    ("swiglu", 128, "f16", 128, 128, 2, 2, "softmax", [2, 8], 1),
    ("relu", 128, "f16", 128, 4224, 2, 1, "softmax", [4, 2], 3),                    # long K in the second projection: split-K
]


@pytest.mark.parametrize("act,group,sdt,d,f,E,k,gate,bits,T", MMA_CASES)
def test_forward_tensor_core_path(act, group, sdt, d, f, E, k, gate, bits, T):
    shape = inputs.LayerShape(d, f, E, k, act, gate, group, sdt, "bf16")
    _run_case(shape, bits, T, seed=22, path=2)


TMA_CASES = [
    ("relu", 128, "f16", 768, 3072, 8, 1, "softmax", [8, 4, 2, 4, 8, 2, 4, 8], 64),   # 1.5 stages at 2 bits
    ("relu", 128, "f16", 768, 3072, 8, 1, "softmax", [2, 2, 4, 4, 8, 8, 2, 4], 5),    # one 8-token tile
    ("relu", 0, "f16", 512, 1152, 4, 2, "softmax_renorm", [4, 2, 8, 2], 9),           # per-channel scales, 16-token tiles
    ("relu", 128, "f32", 640, 1664, 3, 1, "softmax", [8, 2, 4], 37),                  # K tails at every width, two passes
    ("swiglu", 128, "f16", 512, 1408, 4, 2, "softmax_renorm", [4, 8, 2, 4], 16),
    ("swiglu", 256, "f16", 1024, 2560, 8, 2, "softmax_renorm", [4, 4, 8, 2, 4, 8, 2, 4], 33),
    ("swiglu", 128, "f16", 512, 512, 2, 2, "softmax", [2, 8], 1),
    ("relu", 128, "f16", 512, 8704, 2, 1, "softmax", [4, 2], 3),                      # long K: split-K and many ring wraps
]


@pytest.mark.parametrize("act,group,sdt,d,f,E,k,gate,bits,T", TMA_CASES)
def test_forward_tma_pipeline_path(act, group, sdt, d, f, E, k, gate, bits, T):
    """Both projections in one launch (the default) and as two launches: each within the bar, and
    bit-identical to each other (same arithmetic in the same order, only the scheduling differs)."""
    shape = inputs.LayerShape(d, f, E, k, act, gate, group, sdt, "bf16")
    _, y_fused = _run_case(shape, bits, T, seed=25, path=3, want_y=True)
    _, y_split = _run_case(shape, bits, T, seed=25, path=3, fused=False, want_y=True)
    assert np.array_equal(y_fused, y_split)


I8_CASES = TMA_CASES + [
    ("relu", 128, "f16", 768, 3072, 32, 1, "softmax", [2, 4, 8, 4] * 8, 64),                # many experts, 2 tokens each
    ("swiglu", 128, "f16", 512, 1024, 8, 2, "softmax_renorm", [8, 8, 4, 4, 2, 2, 4, 8], 4),
    ("relu", 256, "f16", 1024, 512, 2, 1, "softmax", [2, 4], 40),                          # 32-token tiles, two passes
]


@pytest.mark.parametrize("act,group,sdt,d,f,E,k,gate,bits,T", I8_CASES)
def test_forward_int8_tensor_core_streaming_path(act, group, sdt, d, f, E, k, gate, bits, T):
    """The decode kernel (codes as 8-bit integer tcgen05 operands, activations as two-limb block-scaled
    integers): both projections in one launch and as two launches, each within the bar and
    bit-identical to each other."""
    shape = inputs.LayerShape(d, f, E, k, act, gate, group, sdt, "bf16")
    _, y_fused = _run_case(shape, bits, T, seed=25, path=6, want_y=True)
    _, y_split = _run_case(shape, bits, T, seed=25, path=6, fused=False, want_y=True)
    assert np.array_equal(y_fused, y_split)


def test_int8_streaming_path_keeps_the_bf16_range():
    """Activations far outside the fp16 range (|x| up to 3e38 would overflow a 16-bit float operand)
    and weights whose products are tiny: the block-scaled integer operands follow the bf16
    exponent range, so the result stays inside the bar."""
    shape = inputs.LayerShape(512, 1024, 4, 1, "relu", "softmax", 128, "f16", "bf16")
    bits = [8, 4, 2, 4]
    for scale_x, std in ((3.0e4, 0.02), (1.0e-3, 1.0e-4), (1.0e6, 1.0e-3)):
        W = inputs.expert_set(28, 0, shape, std)
        x = inputs.to_bf16_valued(inputs.activations(28, 0, 9, shape.d_model, "bf16") * np.float32(scale_x))
        Wr = inputs.router_weight(28, 0, shape.d_model, shape.n_experts, std=0.05 / scale_x)
        packed, scales = oracle_pack_layer(W, shape, bits)
        with layer.MoELayer(shape, bits, max_tokens=9) as moe:
            B.emoe_set_ffn_path(moe.ctx, 6)
            moe.pack_from_host(W)
            y, ids, gates, _ = moe.forward(x, Wr)
        y_ref = oracle.moe_ffn_combine(x, shape.d_ff, shape.act, shape.group, True, bits, packed, scales, ids, gates)
        assert np.isfinite(y).all() and np.abs(y_ref).max() > 0
        assert rel_to_max(y, y_ref) <= 2e-3, (scale_x, std, rel_to_max(y, y_ref))


FULL_RANGE_CASES = [
    # path, act, act_dtype, group, sdt, d, f, E, k, gate, bits, T
    (1, "relu", "f32", 64, "f32", 192, 320, 3, 2, "softmax_renorm", [2, 8, 4], 7),            # CUDA-core kernel
    (2, "swiglu", "bf16", 128, "f16", 256, 384, 4, 2, "softmax", [2, 4, 8, 2], 9),              # register-staged mma.sync
    (3, "relu", "bf16", 128, "f16", 512, 1024, 4, 1, "softmax", [2, 4, 8, 2], 12),              # streaming, offset codes
    (3, "swiglu", "bf16", 128, "f16", 512, 1024, 4, 2, "softmax_renorm", [2, 2, 4, 8], 40),     # streaming, exact codes
    (6, "relu", "bf16", 128, "f16", 512, 1024, 4, 1, "softmax", [2, 4, 8, 2], 12),              # int8 tcgen05 streaming
    (6, "swiglu", "bf16", 128, "f16", 512, 1024, 4, 2, "softmax_renorm", [2, 2, 4, 8], 9),
    (4, "relu", "bf16", 128, "f16", 512, 1024, 2, 1, "softmax", [2, 4], 300),                   # tcgen05 grouped GEMM
    (4, "swiglu", "bf16", 128, "f16", 512, 1024, 2, 2, "softmax", [8, 2], 200),
]


@pytest.mark.parametrize("path,act,adt,group,sdt,d,f,E,k,gate,bits,T", FULL_RANGE_CASES)
def test_forward_with_experts_packed_over_the_full_code_range(path, act, adt, group, sdt, d, f, E, k, gate, bits, T):
    """Experts quantised with the reading that uses every code of the field (-2^(b-1) included: the
    fourth INT2 level, -8, -128) run through every kernel family: the kernels decode whole
    two's-complement fields, so only the quantiser differs."""
    shape = inputs.LayerShape(d, f, E, k, act, gate, group, sdt, adt)
    _run_case(shape, bits, T, seed=29, path=path, full_range=True)


ROUTE_CASES = [
    # act, d, f, E, k, gate, T list (one context, calls back to back: the grid counters must come back to zero)
    ("relu", 768, 3072, 32, 1, "softmax", [64, 1, 7, 64]),
    ("swiglu", 512, 1024, 8, 2, "softmax_renorm", [4, 33, 1, 128]),
    ("relu", 512, 512, 128, 1, "softmax", [96, 3]),
]


@pytest.mark.parametrize("act,d,f,E,k,gate,Ts", ROUTE_CASES)
@pytest.mark.parametrize("path", [3, 6])
def test_router_topk_permutation_and_scatter_in_one_launch(act, d, f, E, k, gate, Ts, path):
    """Small batches take router, Top-K, permutation, scatter and plan in one launch (three launches
    per layer with the expert kernel and the combine).  Its ids, gates, permutation and outputs are
    bit-identical to those of the path with one launch per step, call after call on one context."""
    shape = inputs.LayerShape(d, f, E, k, act, gate, 128, "f16", "bf16")
    bits = ([8, 4, 2, 4] * E)[:E]
    W = inputs.expert_set(41, 0, shape)
    Wr = inputs.router_weight(41, 0, d, E, std=0.05)
    with layer.MoELayer(shape, bits, max_tokens=max(Ts)) as moe:
        B.emoe_set_ffn_path(moe.ctx, path)
        moe.pack_from_host(W)
        for i, T in enumerate(Ts):
            x = inputs.activations(41, i, T, d, "bf16")
            B.emoe_set_fused_projections(moe.ctx, True)
            B.emoe_set_fused_routing(moe.ctx, True)
            one = moe.forward(x, Wr)
            assert B.emoe_kernels_last_forward(moe.ctx) == 3
            B.emoe_set_fused_routing(moe.ctx, False)
            chain = moe.forward(x, Wr)
            assert B.emoe_kernels_last_forward(moe.ctx) == 4
            B.emoe_set_fused_projections(moe.ctx, False)
            many = moe.forward(x, Wr)
            assert B.emoe_kernels_last_forward(moe.ctx) >= 6
            for a, b in zip(one, chain):
                assert np.array_equal(a, b)
            for a, b in zip(one, many):
                assert np.array_equal(a, b)
            ids_ref, _, logits_ref = oracle.route(x, Wr, None, k, gate == "softmax_renorm")
            check_ids(one[1], logits_ref, k)
            _, _, perm_ref = oracle.permute(one[1], E)
            assert np.array_equal(one[3], perm_ref)


LAYER_CASES = [
    # act, act_dtype, group, scale_dtype, d, f, E, k, gate, T list (one context, calls back to back)
    ("relu", "bf16", 128, "f16", 768, 3072, 32, 1, "softmax", [1, 4, 16, 1, 2]),
    ("swiglu", "bf16", 128, "f16", 512, 1536, 8, 2, "softmax_renorm", [1, 8, 3]),
    ("relu", "f32", 0, "f32", 128, 256, 4, 1, "softmax", [5, 1]),
    ("swiglu", "f32", 64, "f16", 192, 320, 3, 2, "softmax_renorm", [7, 2]),
    ("relu", "bf16", 64, "f16", 512, 512, 128, 1, "softmax", [3, 16]),
]


@pytest.mark.parametrize("act,adt,group,sdt,d,f,E,k,gate,Ts", LAYER_CASES)
def test_whole_layer_in_one_launch(act, adt, group, sdt, d, f, E, k, gate, Ts):
    """A handful of tokens on a small layer: router, Top-K, both projections and the gate-weighted
    sum in ONE launch.  Picks and permutation are those of the chain of launches, the gates agree
    to rounding (the router product is summed in another order); the
    output matches the CPU checker within the path's tolerance and the chain's output within the
    difference of two fp32 summation orders; the same through the call with given picks; call
    after call on one context (the grid counters must come back to zero)."""
    shape = inputs.LayerShape(d, f, E, k, act, gate, group, sdt, adt)
    bits = ([8, 4, 2, 4] * E)[:E]
    W = inputs.expert_set(47, 0, shape)
    Wr = inputs.router_weight(47, 0, d, E, std=0.05)
    packed, scales = oracle_pack_layer(W, shape, bits)
    with layer.MoELayer(shape, bits, max_tokens=max(Ts)) as moe:
        moe.pack_from_host(W)
        for i, T in enumerate(Ts):
            x = inputs.activations(47, i, T, d, adt)
            B.emoe_set_fused_layer(moe.ctx, True)
            y, ids, gates, perm = moe.forward(x, Wr)
            assert B.emoe_kernels_last_forward(moe.ctx) == 1
            y_r, perm_r = moe.forward_routed(x, ids, gates)
            assert B.emoe_kernels_last_forward(moe.ctx) == 1
            B.emoe_set_fused_layer(moe.ctx, False)
            y_c, ids_c, gates_c, perm_c = moe.forward(x, Wr)
            assert B.emoe_kernels_last_forward(moe.ctx) > 1
            # the router product is summed slice by slice here: same picks, gates equal to rounding
            assert np.array_equal(ids, ids_c) and np.array_equal(perm, perm_c)
            np.testing.assert_allclose(gates, gates_c, rtol=2e-5, atol=1e-7)
            _, _, logits_ref = oracle.route(x, Wr, None, k, gate == "softmax_renorm")
            check_ids(ids, logits_ref, k)
            assert np.array_equal(perm_r, perm) and np.array_equal(y_r, y)
            y_ref = oracle.moe_ffn_combine(x, f, act, group, adt == "bf16", bits, packed, scales, ids, gates)
            assert rel_to_max(y, y_ref) <= output_tolerance(adt)
            assert rel_to_max(y, y_c) <= output_tolerance(adt)
            assert np.array_equal(B.emoe_last_expert_counts(moe.ctx, E), np.bincount(ids.ravel(), minlength=E))


def test_whole_layer_in_one_launch_with_a_router_bias_and_with_a_bad_pick():
    """A per-token router bias (the form the skewed workloads use) goes into the picks of the
    one-launch layer as it does into the router kernel's; a pick outside [0, E) in the call with
    given picks is reported by the device check, contributes nothing, and the context stays usable."""
    shape = inputs.LayerShape(512, 1024, 8, 2, "relu", "softmax_renorm", 128, "f16", "bf16")
    bits = [8, 4, 2, 4] * 2
    T = 4
    W = inputs.expert_set(53, 0, shape)
    Wr = inputs.router_weight(53, 0, 512, 8, std=0.05)
    x = inputs.activations(53, 0, T, 512, "bf16")
    bias = np.random.default_rng(53).normal(0.0, 2.0, size=(T, 8)).astype(np.float32)
    packed, scales = oracle_pack_layer(W, shape, bits)
    with layer.MoELayer(shape, bits, max_tokens=T) as moe:
        moe.pack_from_host(W)
        y, ids, gates, perm = moe.forward(x, Wr, bias)
        assert B.emoe_kernels_last_forward(moe.ctx) == 1
        ids_ref, gates_ref, logits_ref = oracle.route(x, Wr, bias, 2, True)
        check_ids(ids, logits_ref, 2)
        assert not np.array_equal(ids_ref, oracle.route(x, Wr, None, 2, True)[0])   # the bias decides picks here
        same = np.all(ids == ids_ref, axis=1)
        np.testing.assert_allclose(gates[same], gates_ref[same], rtol=2e-5, atol=1e-7)
        y_ref = oracle.moe_ffn_combine(x, 1024, "relu", 128, True, bits, packed, scales, ids, gates)
        assert rel_to_max(y, y_ref) <= 2e-3
        bad = ids.copy()
        bad[1, 0] = 8
        xd = moe.to_device_x(x)
        idd = torch.from_numpy(bad).to(moe.device)
        gd = torch.from_numpy(gates).to(moe.device)
        yd = torch.empty(T, 512, dtype=torch.float32, device=moe.device)
        B.emoe_moe_forward_routed(moe.ctx, moe.desc, xd.data_ptr(), T, idd.data_ptr(), gd.data_ptr(), moe.table,
                                  yd.data_ptr(), None, 0)
        torch.cuda.synchronize(moe.device)
        assert B.emoe_kernels_last_forward(moe.ctx) == 1
        assert B.emoe_device_status(moe.ctx) == B.ERR_DEVICE_CHECK
        # the other tokens are untouched by the bad pick, and token 1 keeps its valid expert's share
        g2 = gates.copy()
        g2[1, 0] = 0.0
        y_ref2 = oracle.moe_ffn_combine(x, 1024, "relu", 128, True, bits, packed, scales, ids, g2)
        assert rel_to_max(yd.cpu().numpy(), y_ref2) <= 2e-3
        y3, ids3, _, _ = moe.forward(x, Wr, bias)
        assert np.array_equal(y3, y) and np.array_equal(ids3, ids)


def test_one_launch_layer_leaves_larger_calls_to_the_other_kernels():
    """Calls beyond 16 token-expert pairs, or with a forced kernel family, run as before."""
    shape = inputs.LayerShape(512, 1024, 8, 2, "relu", "softmax", 128, "f16", "bf16")
    bits = [8, 4, 2, 4] * 2
    W = inputs.expert_set(49, 0, shape)
    Wr = inputs.router_weight(49, 0, 512, 8, std=0.05)
    with layer.MoELayer(shape, bits, max_tokens=16) as moe:
        moe.pack_from_host(W)
        B.emoe_set_fused_layer(moe.ctx, True)
        moe.forward(inputs.activations(49, 0, 8, 512, "bf16"), Wr)
        assert B.emoe_kernels_last_forward(moe.ctx) == 1
        moe.forward(inputs.activations(49, 1, 9, 512, "bf16"), Wr)
        assert B.emoe_kernels_last_forward(moe.ctx) > 1
        B.emoe_set_ffn_path(moe.ctx, 3)
        moe.forward(inputs.activations(49, 0, 8, 512, "bf16"), Wr)
        assert B.emoe_kernels_last_forward(moe.ctx) > 1
        # the default: only calls of up to eight pairs, where the single launch was measured faster
        B.emoe_set_ffn_path(moe.ctx, 0)
        B.emoe_set_fused_layer(moe.ctx, 2)
        moe.forward(inputs.activations(49, 2, 1, 512, "bf16"), Wr)
        assert B.emoe_kernels_last_forward(moe.ctx) == 1
        moe.forward(inputs.activations(49, 3, 4, 512, "bf16"), Wr)
        assert B.emoe_kernels_last_forward(moe.ctx) == 1
        moe.forward(inputs.activations(49, 4, 5, 512, "bf16"), Wr)
        assert B.emoe_kernels_last_forward(moe.ctx) > 1


def test_grid_wide_waits_of_the_one_launch_layer_run_out_without_a_hang():
    """The CTAs are told to wait for one more arrival than will ever come, with a short limit: the
    waits give up, the kernel returns, the status call says "timeout", and the next call on the
    context is right again."""
    shape = inputs.LayerShape(512, 1024, 8, 1, "relu", "softmax", 128, "f16", "bf16")
    bits, T = [8, 4, 2, 4] * 2, 4
    W = inputs.expert_set(51, 0, shape)
    x = inputs.activations(51, 0, T, 512, "bf16")
    Wr = inputs.router_weight(51, 0, 512, 8, std=0.05)
    with layer.MoELayer(shape, bits, max_tokens=T) as moe:
        moe.pack_from_host(W)
        B.emoe_set_fused_layer(moe.ctx, True)
        good = moe.forward(x, Wr)
        B.emoe_set_wait_limit(moe.ctx, 2000)
        B.emoe_debug_expect_extra_completions(moe.ctx, 1)
        with pytest.raises(B.EmoeError) as ei:
            moe.forward(x, Wr)
        assert ei.value.status == B.ERR_TIMEOUT
        B.emoe_set_wait_limit(moe.ctx, 0)
        B.emoe_debug_expect_extra_completions(moe.ctx, 0)
        again = moe.forward(x, Wr)
        for a, b in zip(good, again):
            assert np.array_equal(a, b)


def test_grid_wide_wait_of_the_one_launch_routing_runs_out_without_a_hang():
    """The CTAs are told to wait for one more arrival than the grid has, with a short limit: every
    wait gives up, every kernel still returns, the status call says "timeout", and the next call on
    the context is right again."""
    shape = inputs.LayerShape(512, 1024, 8, 1, "relu", "softmax", 128, "f16", "bf16")
    bits, T = [8, 4, 2, 4] * 2, 128
    W = inputs.expert_set(43, 0, shape)
    x = inputs.activations(43, 0, T, shape.d_model, "bf16")
    Wr = inputs.router_weight(43, 0, shape.d_model, shape.n_experts, std=0.05)
    with layer.MoELayer(shape, bits, max_tokens=T) as moe:
        B.emoe_set_ffn_path(moe.ctx, 3)
        moe.pack_from_host(W)
        good = moe.forward(x, Wr)
        B.emoe_set_fused_routing(moe.ctx, True)
        B.emoe_set_wait_limit(moe.ctx, 2000)
        B.emoe_debug_expect_extra_completions(moe.ctx, 1)
        with pytest.raises(B.EmoeError) as ei:
            moe.forward(x, Wr)
        assert ei.value.status == B.ERR_TIMEOUT
        B.emoe_set_wait_limit(moe.ctx, 0)
        B.emoe_debug_expect_extra_completions(moe.ctx, 0)
        again = moe.forward(x, Wr)
        for a, b in zip(good, again):
            assert np.array_equal(a, b)


def test_bounded_wait_inside_the_kernel_runs_out_and_the_context_stays_usable():
    """Failure detection without a fault: the second projection is told to expect one more
    completion of the first than will ever be counted, with a short wait limit.  The wait must give
    up, the kernels must return, the status call must say "timeout", and the next ordinary forward
    on the same context must be right again."""
    shape = inputs.LayerShape(512, 1024, 4, 1, "relu", "softmax", 128, "f16", "bf16")
    bits, T = [8, 4, 2, 4], 6
    W = inputs.expert_set(35, 0, shape)
    x = inputs.activations(35, 0, T, shape.d_model, "bf16")
    Wr = inputs.router_weight(35, 0, shape.d_model, shape.n_experts, std=0.05)
    packed, scales = oracle_pack_layer(W, shape, bits)
    with layer.MoELayer(shape, bits, max_tokens=T) as moe:
        B.emoe_set_ffn_path(moe.ctx, 6)
        moe.pack_from_host(W)
        y, ids, gates, _ = moe.forward(x, Wr)
        y_ref = oracle.moe_ffn_combine(x, shape.d_ff, shape.act, shape.group, True, bits, packed, scales, ids, gates)
        assert rel_to_max(y, y_ref) <= 2e-3
        B.emoe_set_wait_limit(moe.ctx, 20000)
        B.emoe_debug_expect_extra_completions(moe.ctx, 1)
        with pytest.raises(B.EmoeError) as ei:
            moe.forward(x, Wr)                      # returns (no hang); the device check reports the timeout
        assert ei.value.status == B.ERR_TIMEOUT
        assert B.emoe_device_status(moe.ctx) == B.OK   # the word was cleared by the read above
        B.emoe_debug_expect_extra_completions(moe.ctx, 0)
        B.emoe_set_wait_limit(moe.ctx, 0)
        y2, ids2, gates2, _ = moe.forward(x, Wr)
        assert np.array_equal(ids2, ids) and np.array_equal(y2, y)


@pytest.mark.parametrize("path", [0, 3, 4])
def test_fp16_operand_kernels_report_values_outside_their_range(path):
    """The default tensor-core kernels carry activations as fp16.  Inputs (or hidden values) beyond
    65504 are saturated there, and the many-token kernel also loses bits of q * s below 2^-14: neither
    may pass silently.  The device status must say so; the same inputs on kernel family 6 stay
    inside the bar (previous test)."""
    shape = inputs.LayerShape(512, 1024, 4, 1, "relu", "softmax", 128, "f16", "bf16")
    bits, T = [8, 4, 2, 4], 9
    cases = [(3.0e4, 0.02)]                    # x beyond 65504
    if path == 4:
        cases.append((1.0, 1.0e-5))            # scales below 2^-14: q * s is subnormal as fp16
    for scale_x, std in cases:
        W = inputs.expert_set(28, 0, shape, std)
        x = inputs.to_bf16_valued(inputs.activations(28, 0, T, shape.d_model, "bf16") * np.float32(scale_x))
        Wr = inputs.router_weight(28, 0, shape.d_model, shape.n_experts, std=0.05 / scale_x)
        with layer.MoELayer(shape, bits, max_tokens=T) as moe:
            B.emoe_set_ffn_path(moe.ctx, path)
            moe.pack_from_host(W)
            with pytest.raises(B.EmoeError) as ei:
                moe.forward(x, Wr)
            assert ei.value.status == B.ERR_RANGE, (path, scale_x)
            # ordinary inputs afterwards: no flag is left over
            x_ok = inputs.activations(28, 0, T, shape.d_model, "bf16")
            W_ok = inputs.expert_set(28, 0, shape, 0.02)
            moe.pack_from_host(W_ok)
            moe.forward(x_ok, inputs.router_weight(28, 0, shape.d_model, shape.n_experts, std=0.05))


UMMA_CASES = [
    ("relu", 128, "f16", 512, 1024, 4, 1, "softmax", [8, 4, 2, 4], 200),              # ~50 tokens per expert
    ("relu", 128, "f16", 512, 1024, 2, 1, "softmax", [4, 2], 300),                    # two token tiles per expert
    ("relu", 0, "f16", 1024, 512, 3, 2, "softmax_renorm", [2, 8, 4], 97),             # per-channel scales
    ("swiglu", 128, "f16", 512, 1536, 4, 2, "softmax_renorm", [4, 8, 2, 4], 150),     # two accumulators
    ("swiglu", 256, "f32", 1024, 2048, 8, 2, "softmax_renorm", [4, 4, 8, 2, 4, 8, 2, 4], 64),
    ("relu", 128, "f16", 512, 512, 2, 1, "softmax", [2, 8], 1),                       # a single token
]


@pytest.mark.parametrize("act,group,sdt,d,f,E,k,gate,bits,T", UMMA_CASES)
def test_forward_tcgen05_path(act, group, sdt, d, f, E, k, gate, bits, T):
    shape = inputs.LayerShape(d, f, E, k, act, gate, group, sdt, "bf16")
    _run_case(shape, bits, T, seed=27, path=4)


HYBRID_CASES = [
    # loads shaped by a router bias so that some experts hold more than 32 tokens and others fewer
    ("relu", 128, "f16", 512, 1024, 8, 1, "softmax", [8, 4, 2, 4, 2, 8, 4, 2], 220, 1.1),
    ("swiglu", 128, "f16", 512, 1536, 6, 2, "softmax_renorm", [4, 8, 2, 4, 2, 8], 90, 1.3),
    ("relu", 0, "f32", 1024, 512, 5, 1, "softmax", [2, 8, 4, 4, 8], 64, 1.5),
    ("relu", 128, "f16", 512, 512, 4, 1, "softmax", [2, 8, 4, 4], 12, 0.0),          # nobody above 32 tokens
    ("relu", 128, "f16", 512, 1024, 2, 1, "softmax", [4, 2], 300, 0.0),               # everybody above 32 tokens
    ("swiglu", 128, "f16", 512, 512, 2, 2, "softmax_renorm", [8, 2], 700, 0.0),       # 700 tokens per expert: several token groups
]


@pytest.mark.parametrize("act,group,sdt,d,f,E,k,gate,bits,T,zipf", HYBRID_CASES)
def test_forward_both_kernel_families_in_one_call(act, group, sdt, d, f, E, k, gate, bits, T, zipf):
    """Skewed loads: experts with few tokens stream, the others run on tcgen05, one forward call."""
    shape = inputs.LayerShape(d, f, E, k, act, gate, group, sdt, "bf16")
    bias = None
    if zipf > 0:
        bias = (-zipf * 2.0 * np.log(np.arange(1, E + 1))).astype(np.float32)  # strongly decreasing loads
    x = inputs.activations(29, 0, T, d, "bf16")
    Wr = inputs.router_weight(29, 0, d, E, std=0.05)
    ids, _, _ = oracle.route(x, Wr, bias, k, gate == "softmax_renorm")
    counts = np.bincount(ids.reshape(-1), minlength=E)
    if zipf > 0:
        assert counts.max() > 32 and 0 < counts[counts > 0].min() <= 32, counts   # the case covers both families
    _run_case(shape, bits, T, seed=29, path=5, bias=bias)
    _run_case(shape, bits, T, seed=29, path=5, bias=bias, fused=False)


def test_tma_path_is_refused_for_narrow_rows():
    shape = inputs.LayerShape(256, 512, 4, 1, "relu", "softmax", 128, "f16", "bf16")
    with pytest.raises(B.EmoeError) as ei:
        _run_case(shape, [2, 4, 8, 4], 4, seed=26, path=3)
    assert ei.value.status == B.ERR_UNSUPPORTED


def test_both_paths_agree_and_default_picks_tensor_cores():
    shape = inputs.LayerShape(256, 512, 4, 2, "swiglu", "softmax_renorm", 128, "f16", "bf16")
    e_auto = _run_case(shape, [2, 4, 8, 4], 12, seed=23, path=0)
    e_gemv = _run_case(shape, [2, 4, 8, 4], 12, seed=23, path=1)
    e_mma = _run_case(shape, [2, 4, 8, 4], 12, seed=23, path=2)
    assert e_auto == e_mma and e_gemv <= 2e-3
    big = inputs.LayerShape(512, 1024, 4, 2, "swiglu", "softmax_renorm", 128, "f16", "bf16")
    # wide enough for the weight-streaming kernels: the default is the TMA-staged mma.sync one
    assert _run_case(big, [2, 4, 8, 4], 12, seed=23, path=0) == _run_case(big, [2, 4, 8, 4], 12, seed=23, path=3)
    assert _run_case(big, [2, 4, 8, 4], 12, seed=23, path=6) <= 2e-3


def test_zipf_bias_and_many_tokens_on_one_expert():
    """All tokens of a batch on one expert (several token passes) plus idle experts."""
    shape = inputs.LayerShape(256, 512, 8, 1, "relu", "softmax", 128, "f16", "bf16")
    bias = np.full(8, -30.0, dtype=np.float32)
    bias[5] = 30.0
    for path in (1, 2):
        _run_case(shape, [2, 4, 8, 4, 2, 4, 8, 2], 70, seed=24, path=path, bias=bias)
    wide = inputs.LayerShape(512, 1024, 8, 1, "relu", "softmax", 128, "f16", "bf16")
    _run_case(wide, [2, 4, 8, 4, 2, 4, 8, 2], 70, seed=24, path=3, bias=bias)


def test_forward_routed_and_unselected_experts():
    shape = inputs.LayerShape(256, 384, 4, 2, "relu", "softmax", 128, "f16", "bf16")
    bits = [4, 2, 8, 4]
    W = inputs.expert_set(30, 0, shape)
    x = inputs.activations(30, 0, 6, shape.d_model, "bf16")
    ids = np.array([[0, 2], [2, 0], [0, 2], [2, 0], [0, 2], [2, 0]], dtype=np.int32)
    gates = np.random.default_rng(0).random((6, 2)).astype(np.float32)
    packed, scales = oracle_pack_layer(W, shape, bits)
    y_ref = oracle.moe_ffn_combine(x, shape.d_ff, "relu", 128, True, bits, packed, scales, ids, gates)
    for path in (1, 2):
        with layer.MoELayer(shape, bits, max_tokens=6) as moe:
            B.emoe_set_ffn_path(moe.ctx, path)
            moe.pack_from_host(W)
            y, perm = moe.forward_routed(x, ids, gates)
            assert np.array_equal(perm, oracle.permute(ids, 4)[2])
            assert rel_to_max(y, y_ref) <= 2e-3
            # experts 1 and 3 are never selected: overwriting their weights changes nothing
            moe.packed[1][0].fill_(0x5A)
            moe.scales[3][1].fill_(3.0)
            y2, _ = moe.forward_routed(x, ids, gates)
            assert np.array_equal(y, y2)
            # two runs are bit-identical
            y3, _ = moe.forward_routed(x, ids, gates)
            assert np.array_equal(y2, y3)


def test_forward_argument_errors():
    shape = inputs.LayerShape(256, 384, 4, 2, "relu", "softmax", 128, "f16", "bf16")
    lib = B.lib()
    with layer.MoELayer(shape, [4, 2, 8, 4], max_tokens=4) as moe:
        x = torch.zeros(8, 256, dtype=torch.bfloat16, device="cuda")
        Wr = torch.zeros(256, 4, device="cuda")
        y = torch.zeros(8, 256, device="cuda")
        import ctypes
        fwd = lambda desc, T, tab, xp=x.data_ptr(): lib.emoe_moe_forward(
            moe.ctx, ctypes.byref(desc), xp, T, Wr.data_ptr(), None, 0, tab, y.data_ptr(), None, None, None, None)
        assert fwd(moe.desc, 8, moe.table) == B.ERR_WORKSPACE          # context sized for 4 tokens
        assert fwd(moe.desc, 0, moe.table) == B.ERR_INVALID_ARG
        assert fwd(moe.desc, 4, moe.table, x.data_ptr() + 2) == B.ERR_ALIGNMENT
        bad = layer.make_desc(shape)
        bad.top_k = 5
        assert fwd(bad, 4, moe.table) == B.ERR_INVALID_ARG
        tab = B.make_expert_table([(3, [t.data_ptr() for t in moe.packed[e]], [t.data_ptr() for t in moe.scales[e]])
                                   for e in range(4)])
        assert fwd(moe.desc, 4, tab) == B.ERR_UNSUPPORTED
        assert fwd(moe.desc, 4, moe.table) == B.OK
        torch.cuda.synchronize()
