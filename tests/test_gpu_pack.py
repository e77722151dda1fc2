"""GPU parity: emoe_pack_expert against the CPU checker, bit for bit (packed bytes and the
scale channel), through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2308_14352_b200 import binding as B

pytestmark = pytest.mark.gpu

SDT = {"f32": (B.DTYPE_F32, torch.float32), "f16": (B.DTYPE_F16, torch.float16)}


@pytest.fixture(scope="module")
def ctx():
    torch.zeros(1, device="cuda")
    c = B.emoe_create(0, 1 << 20)
    yield c
    torch.cuda.synchronize()
    B.emoe_destroy(c)


def _gpu_pack(ctx, W, bits, group, sdt, full_range=False):
    N, K = W.shape
    G = group if group else K
    code, tdt = SDT[sdt]
    Wd = torch.from_numpy(W).cuda()
    packed = torch.zeros(B.emoe_packed_bytes(N, K, bits), dtype=torch.uint8, device="cuda")
    scales = torch.zeros(N * (K // G), dtype=tdt, device="cuda")
    assert B.emoe_scales_bytes(N, K, group, code) == scales.numel() * scales.element_size()
    if full_range:
        B.emoe_pack_expert_mode(ctx, Wd.data_ptr(), N, K, bits, group, code, B.RANGE_FULL, packed.data_ptr(),
                                scales.data_ptr(), 0)
    else:
        B.emoe_pack_expert(ctx, Wd.data_ptr(), N, K, bits, group, code, packed.data_ptr(), scales.data_ptr(), 0)
    torch.cuda.synchronize()
    return packed.cpu().numpy().reshape(N, -1), scales.cpu().numpy().reshape(N, K // G)


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("group,sdt", [(0, "f32"), (0, "f16"), (128, "f16"), (32, "f16"), (128, "f32"), (64, "f32")])
@pytest.mark.parametrize("N,K", [(37, 384), (5, 4096), (130, 128)])
def test_pack_bit_exact(ctx, bits, group, sdt, N, K):
    rng = np.random.default_rng(bits * 1000 + group + N)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    W[1, :] = 0.0                                 # all-zero channel
    W[2, : K // 2] *= 1e-6                          # groups whose fp16 scale is subnormal
    W[3, ::7] = np.float32(0.02)                    # repeated values
    if N > 4:
        W[4] = np.round(W[4] * 400) / 400           # values that land on rounding ties more often
    p_ref, s_ref = oracle.pack_expert(W, bits, group, sdt)
    p_gpu, s_gpu = _gpu_pack(ctx, W, bits, group, sdt)
    assert np.array_equal(s_gpu.view(np.uint16 if sdt == "f16" else np.uint32),
                          oracle.scales_storage(s_ref, sdt).view(np.uint16 if sdt == "f16" else np.uint32))
    assert np.array_equal(p_gpu, p_ref)


def test_pack_exact_ties_and_extremes(ctx):
    # scale exactly 1 (amax = qmax): quotients are the inputs themselves, halves go to even
    w = np.zeros((1, 128), dtype=np.float32)
    w[0, :8] = [7.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5]
    p_gpu, s_gpu = _gpu_pack(ctx, w, 4, 0, "f32")
    assert s_gpu[0, 0] == 1.0
    assert oracle.unpack(p_gpu, 128, 4)[0, :8].tolist() == [7, 0, 2, 2, 0, -2, -2, 4]
    p_ref, _ = oracle.pack_expert(w, 4, 0, "f32")
    assert np.array_equal(p_gpu, p_ref)


def test_pack_argument_errors(ctx):
    lib = B.lib()
    W = torch.zeros(8, 128, device="cuda")
    out = torch.zeros(8 * 128, dtype=torch.uint8, device="cuda")
    sc = torch.zeros(8 * 4, dtype=torch.float32, device="cuda")
    call = lambda *a: lib.emoe_pack_expert(ctx, *a)
    assert call(W.data_ptr(), 8, 128, 3, 0, B.DTYPE_F32, out.data_ptr(), sc.data_ptr(), None) == B.ERR_UNSUPPORTED
    assert call(W.data_ptr(), 8, 128, 4, 48, B.DTYPE_F32, out.data_ptr(), sc.data_ptr(), None) == B.ERR_INVALID_ARG
    assert call(None, 8, 128, 4, 0, B.DTYPE_F32, out.data_ptr(), sc.data_ptr(), None) == B.ERR_INVALID_ARG
    assert call(W.data_ptr(), 0, 128, 4, 0, B.DTYPE_F32, out.data_ptr(), sc.data_ptr(), None) == B.ERR_INVALID_ARG
    assert call(W.data_ptr() + 4, 8, 128, 4, 0, B.DTYPE_F32, out.data_ptr(), sc.data_ptr(), None) == B.ERR_ALIGNMENT
    assert call(W.data_ptr(), 8, 128, 4, 0, B.DTYPE_BF16, out.data_ptr(), sc.data_ptr(), None) == B.ERR_UNSUPPORTED


def _assert_same(p_gpu, s_gpu, p_ref, s_ref, sdt):
    view = np.uint16 if sdt == "f16" else np.uint32
    assert np.array_equal(s_gpu.view(view), oracle.scales_storage(s_ref, sdt).view(view))
    assert np.array_equal(p_gpu, p_ref)


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("group,sdt", [(0, "f32"), (128, "f16"), (32, "f16"), (128, "f32")])
@pytest.mark.parametrize("N,K", [(37, 384), (130, 128)])
def test_pack_full_range_bit_exact(ctx, bits, group, sdt, N, K):
    """The reading that uses every code of the field (Section 3.2): bytes and scales bit for bit."""
    rng = np.random.default_rng(bits * 77 + group + N)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    W[1, :] = 0.0
    W[2, : K // 2] *= 1e-6
    W[3, 5] = -np.abs(W[3]).max() * 2                # the negative extreme takes the extra code
    W[4, 9] = np.abs(W[4]).max() * 2                 # the positive extreme is clamped
    p_ref, s_ref = oracle.pack_expert(W, bits, group, sdt, full_range=True)
    p_gpu, s_gpu = _gpu_pack(ctx, W, bits, group, sdt, full_range=True)
    _assert_same(p_gpu, s_gpu, p_ref, s_ref, sdt)
    q = oracle.unpack(p_gpu, K, bits)
    assert q.min() == -(1 << (bits - 1)) and q.max() == (1 << (bits - 1)) - 1


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("group,sdt", [(128, "f16"), (128, "f32"), (0, "f32"), (64, "f16")])
@pytest.mark.parametrize("full_range", [False, True])
def test_pack_weights_on_and_next_to_rounding_ties(ctx, bits, group, sdt, full_range):
    """The kernel forms w * (1/s) and falls back to the definition's division near a half-integer.
    Weights placed on the ties of their group's stored scale and one to three fp32 steps on either
    side of them, at ordinary, tiny and huge magnitudes, must still give the definition's codes."""
    rng = np.random.default_rng(9 + bits + group)
    N, K = 48, 512
    G = group or K
    half = 1 << (bits - 1)
    W = np.zeros((N, K), dtype=np.float32)
    for n in range(N):
        mag = [0.02, 1.0, 3e-7, 1e-36, 3e34, 777.0][n % 6]
        for g in range(K // G):
            amax = np.float32(mag * (1.0 + rng.random()))
            rng_div = np.float32(half if full_range else half - 1)
            s = np.float32(amax / rng_div)
            if sdt == "f16":
                with np.errstate(over="ignore"):
                    s = np.float32(np.float16(s))
            if not np.isfinite(s) or s == 0:
                s = np.float32(amax / rng_div)
            h = rng.integers(-half, half, size=G).astype(np.float64) + 0.5      # half-integers in range
            w = (h * np.float64(s)).astype(np.float32)
            steps = rng.integers(-3, 4, size=G)
            for i in range(G):
                for _ in range(abs(int(steps[i]))):
                    w[i] = np.nextafter(w[i], np.float32(np.inf if steps[i] > 0 else -np.inf))
            w[0] = amax                                                          # fixes the group's max-abs
            w = np.clip(w, -amax, amax)
            W[n, g * G:(g + 1) * G] = w
    p_ref, s_ref = oracle.pack_expert(W, bits, group, sdt, full_range)
    p_gpu, s_gpu = _gpu_pack(ctx, W, bits, group, sdt, full_range)
    _assert_same(p_gpu, s_gpu, p_ref, s_ref, sdt)
