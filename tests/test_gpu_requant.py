"""GPU parity: emoe_requantize_expert against the CPU checker, bit for bit (packed bytes and
the scale channel), through the C ABI.  The stored input comes from the checker, so the two
sides see the same bytes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2308_14352_b200 import binding as B

pytestmark = pytest.mark.gpu

SDT = {"f32": (B.DTYPE_F32, torch.float32, np.uint32), "f16": (B.DTYPE_F16, torch.float16, np.uint16)}


@pytest.fixture(scope="module")
def ctx():
    torch.zeros(1, device="cuda")
    c = B.emoe_create(0, 1 << 20)
    yield c
    torch.cuda.synchronize()
    B.emoe_destroy(c)


def _gpu_requant(ctx, packed, scales, K, bits_in, bits_out, group, sdt, full_range=False):
    N = packed.shape[0]
    G = group if group else K
    code, tdt, _ = SDT[sdt]
    pin = torch.from_numpy(np.ascontiguousarray(packed)).cuda()
    sin = torch.from_numpy(oracle.scales_storage(scales, sdt)).cuda()
    pout = torch.zeros(B.emoe_packed_bytes(N, K, bits_out), dtype=torch.uint8, device="cuda")
    sout = torch.zeros(N * (K // G), dtype=tdt, device="cuda")
    if full_range:
        B.emoe_requantize_expert_mode(ctx, pin.data_ptr(), sin.data_ptr(), N, K, bits_in, bits_out, group, code,
                                      B.RANGE_FULL, pout.data_ptr(), sout.data_ptr(), 0)
    else:
        B.emoe_requantize_expert(ctx, pin.data_ptr(), sin.data_ptr(), N, K, bits_in, bits_out, group, code,
                                 pout.data_ptr(), sout.data_ptr(), 0)
    torch.cuda.synchronize()
    return pout.cpu().numpy().reshape(N, -1), sout.cpu().numpy().reshape(N, K // G)


@pytest.mark.parametrize("bits_in,bits_out", [(8, 4), (8, 2), (4, 2), (8, 8), (4, 4), (2, 2), (2, 4), (4, 8), (2, 8)])
@pytest.mark.parametrize("group,sdt", [(0, "f32"), (0, "f16"), (128, "f16"), (32, "f16"), (64, "f32")])
@pytest.mark.parametrize("N,K", [(37, 384), (5, 4096), (130, 128)])
def test_requantize_bit_exact(ctx, bits_in, bits_out, group, sdt, N, K):
    rng = np.random.default_rng(bits_in * 100 + bits_out * 10 + group + N)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    W[1, :] = 0.0                      # all-zero channel: scale 0 in, scale 0 out
    W[2, : K // 2] *= 1e-6             # groups whose fp16 scale is subnormal
    packed, scales = oracle.pack_expert(W, bits_in, group, sdt)
    p_ref, s_ref = oracle.requantize(packed, scales, K, bits_in, bits_out, group, sdt)
    p_gpu, s_gpu = _gpu_requant(ctx, packed, scales, K, bits_in, bits_out, group, sdt)
    view = SDT[sdt][2]
    assert np.array_equal(s_gpu.view(view), oracle.scales_storage(s_ref, sdt).view(view))
    assert np.array_equal(p_gpu, p_ref)
    if bits_in == bits_out and sdt == "f16":   # the same width reproduces the stored matrix
        assert np.array_equal(p_gpu, packed)


def test_requantize_equals_pack_of_the_decompressed_matrix(ctx):
    """The definition, end to end on the GPU: requantise == quantise(decompress(stored))."""
    rng = np.random.default_rng(77)
    N, K, G = 64, 1024, 128
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    packed, scales = oracle.pack_expert(W, 8, G, "f16")
    Wt = oracle.dequantize(packed, scales, K, 8, G).astype(np.float32)
    Wd = torch.from_numpy(Wt).cuda()
    p2 = torch.zeros(B.emoe_packed_bytes(N, K, 4), dtype=torch.uint8, device="cuda")
    s2 = torch.zeros(N * (K // G), dtype=torch.float16, device="cuda")
    B.emoe_pack_expert(ctx, Wd.data_ptr(), N, K, 4, G, B.DTYPE_F16, p2.data_ptr(), s2.data_ptr(), 0)
    p_gpu, s_gpu = _gpu_requant(ctx, packed, scales, K, 8, 4, G, "f16")
    torch.cuda.synchronize()
    assert np.array_equal(p_gpu.ravel(), p2.cpu().numpy())
    assert np.array_equal(s_gpu.ravel().view(np.uint16), s2.cpu().numpy().view(np.uint16))


def test_requantize_full_size_matrix_sampled_rows(ctx):
    """One matrix of the Mixtral-like layer (14336 x 4096, INT8 -> INT4, group-128 fp16 scales): the
    whole result against the checker on sampled rows."""
    N, K, G = 14336, 4096, 128
    g = torch.Generator(device="cuda")
    g.manual_seed(3)
    Wd = torch.randn(N, K, device="cuda", generator=g) * 0.02
    p8 = torch.zeros(B.emoe_packed_bytes(N, K, 8), dtype=torch.uint8, device="cuda")
    s8 = torch.zeros(N * (K // G), dtype=torch.float16, device="cuda")
    B.emoe_pack_expert(ctx, Wd.data_ptr(), N, K, 8, G, B.DTYPE_F16, p8.data_ptr(), s8.data_ptr(), 0)
    p4 = torch.zeros(B.emoe_packed_bytes(N, K, 4), dtype=torch.uint8, device="cuda")
    s4 = torch.zeros(N * (K // G), dtype=torch.float16, device="cuda")
    B.emoe_requantize_expert(ctx, p8.data_ptr(), s8.data_ptr(), N, K, 8, 4, G, B.DTYPE_F16, p4.data_ptr(), s4.data_ptr(), 0)
    torch.cuda.synchronize()
    rows = np.array([0, 1, 63, 64, 777, 8191, 14335])
    p8h = p8.view(N, K)[rows].cpu().numpy()
    s8h = s8.view(N, K // G)[rows].cpu().numpy().astype(np.float32)
    p_ref, s_ref = oracle.requantize(p8h, s8h, K, 8, 4, G, "f16")
    assert np.array_equal(p4.view(N, K // 2)[rows].cpu().numpy(), p_ref)
    assert np.array_equal(s4.view(N, K // G)[rows].cpu().numpy().view(np.uint16),
                          oracle.scales_storage(s_ref, "f16").view(np.uint16))


def test_requantize_argument_errors(ctx):
    lib = B.lib()
    pin = torch.zeros(8 * 128, dtype=torch.uint8, device="cuda")
    sin = torch.zeros(8, dtype=torch.float32, device="cuda")
    pout = torch.zeros(8 * 64, dtype=torch.uint8, device="cuda")
    sout = torch.zeros(8, dtype=torch.float32, device="cuda")
    call = lambda *a: lib.emoe_requantize_expert(ctx, *a)
    ok = (pin.data_ptr(), sin.data_ptr(), 8, 128, 8, 4, 0, B.DTYPE_F32, pout.data_ptr(), sout.data_ptr(), None)
    assert call(*ok) == B.OK
    bad = lambda i, v: tuple(v if j == i else a for j, a in enumerate(ok))
    assert call(*bad(4, 3)) == B.ERR_UNSUPPORTED          # bits_in
    assert call(*bad(5, 16)) == B.ERR_UNSUPPORTED         # bits_out
    assert call(*bad(6, 48)) == B.ERR_INVALID_ARG         # group does not divide K
    assert call(*bad(0, None)) == B.ERR_INVALID_ARG
    assert call(*bad(2, 0)) == B.ERR_INVALID_ARG
    assert call(*bad(8, pin.data_ptr())) == B.ERR_INVALID_ARG   # in place
    assert call(*bad(0, pin.data_ptr() + 4)) == B.ERR_ALIGNMENT
    assert call(*bad(7, B.DTYPE_BF16)) == B.ERR_UNSUPPORTED
    torch.cuda.synchronize()


def test_forward_after_lowering_the_width_of_two_experts():
    """The bitwidth adaptation end to end: a layer packed at INT8, two experts then moved to INT4
    and INT2 on the device; packed bytes and scales equal the checker's, and the forward on the
    new storage equals the checker's forward on it."""
    from paper_2308_14352_b200 import inputs, layer
    from tests.helpers import rel_to_max

    shape = inputs.LayerShape(512, 1024, 4, 2, "swiglu", "softmax_renorm", 128, "f16", "bf16")
    bits = [8, 8, 8, 8]
    W = inputs.expert_set(41, 0, shape)
    x = inputs.activations(41, 0, 12, shape.d_model, "bf16")
    Wr = inputs.router_weight(41, 0, shape.d_model, shape.n_experts, std=0.05)
    packed, scales = [], []
    for e in range(4):
        ps = [oracle.pack_expert(W[e][m], 8, 128, "f16") for m in range(3)]
        packed.append([p for p, _ in ps])
        scales.append([s for _, s in ps])
    new_bits = [8, 4, 8, 2]
    for e in (1, 3):
        for m in range(3):
            K = shape.matrix_shape(m)[1]
            packed[e][m], scales[e][m] = oracle.requantize(packed[e][m], scales[e][m], K, 8, new_bits[e], 128, "f16")
    with layer.MoELayer(shape, bits, max_tokens=12) as moe:
        moe.pack_from_host(W)
        moe.change_width(1, 4)
        moe.change_width(3, 2)
        assert moe.bits == new_bits
        for e in range(4):
            for m in range(3):
                assert np.array_equal(moe.packed_host(e, m), packed[e][m])
                assert np.array_equal(moe.scales_host(e, m).astype(np.float32), scales[e][m])
        y, ids, gates, _ = moe.forward(x, Wr)
    y_ref = oracle.moe_ffn_combine(x, shape.d_ff, "swiglu", 128, True, new_bits, packed, scales, ids, gates)
    assert rel_to_max(y, y_ref) <= 2e-3


@pytest.mark.parametrize("bits_in,bits_out", [(8, 4), (8, 2), (4, 2), (2, 2), (2, 8)])
@pytest.mark.parametrize("group,sdt", [(0, "f32"), (128, "f16"), (32, "f16")])
def test_requantize_full_range_bit_exact(ctx, bits_in, bits_out, group, sdt):
    """A stored matrix (itself packed with the full code range) moved to another width, again with
    the full range (Section 3.2): bytes and scales bit for bit."""
    N, K = 37, 384
    rng = np.random.default_rng(bits_in * 31 + bits_out + group)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    W[1, :] = 0.0
    packed, scales = oracle.pack_expert(W, bits_in, group, sdt, full_range=True)
    p_ref, s_ref = oracle.requantize(packed, scales, K, bits_in, bits_out, group, sdt, full_range=True)
    p_gpu, s_gpu = _gpu_requant(ctx, packed, scales, K, bits_in, bits_out, group, sdt, full_range=True)
    view = SDT[sdt][2]
    assert np.array_equal(s_gpu.view(view), oracle.scales_storage(s_ref, sdt).view(view))
    assert np.array_equal(p_gpu, p_ref)
