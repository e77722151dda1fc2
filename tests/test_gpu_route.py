"""GPU parity: emoe_router_topk and emoe_permute against the CPU checker through the C ABI.
Expert ids are compared exactly wherever the decisive logit gaps exceed 1e-4; the permutation
(counts, offsets, order) is compared bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2308_14352_b200 import binding as B, inputs
from tests.helpers import check_ids

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    torch.zeros(1, device="cuda")
    c = B.emoe_create(0, 1 << 20)
    yield c
    torch.cuda.synchronize()
    B.emoe_destroy(c)


def _route_gpu(ctx, x, bf16, Wr, bias, k, renorm):
    T, d = x.shape
    E = Wr.shape[1]
    xd = torch.from_numpy(x).cuda()
    if bf16:
        xd = xd.to(torch.bfloat16)
    Wd = torch.from_numpy(Wr).cuda()
    bd = None if bias is None else torch.from_numpy(bias).cuda()
    stride = E if (bias is not None and bias.ndim == 2) else 0
    ids = torch.full((T, k), -1, dtype=torch.int32, device="cuda")
    gates = torch.zeros(T, k, dtype=torch.float32, device="cuda")
    logits = torch.zeros(T, E, dtype=torch.float32, device="cuda")
    B.emoe_router_topk(ctx, xd.data_ptr(), B.DTYPE_BF16 if bf16 else B.DTYPE_F32, T, d, Wd.data_ptr(),
                       None if bd is None else bd.data_ptr(), stride, E, k,
                       B.GATE_SOFTMAX_RENORM if renorm else B.GATE_SOFTMAX, ids.data_ptr(), gates.data_ptr(),
                       logits.data_ptr(), 0)
    torch.cuda.synchronize()
    return ids.cpu().numpy(), gates.cpu().numpy(), logits.cpu().numpy()


CASES = [
    # T, d, E, k, renorm, bf16, bias
    (1, 768, 32, 1, False, True, None),
    (64, 768, 32, 1, False, True, None),
    (16, 768, 8, 1, False, False, None),
    (33, 4096, 8, 2, True, True, None),
    (5, 64, 200, 3, True, False, "vec"),
    (600, 1024, 128, 1, False, True, "vec"),      # 8-token CTAs with a ragged last CTA
    (515, 1100, 7, 2, True, False, "tok"),         # d not a multiple of the chunk, odd E, per-token bias
    (9, 96, 1, 1, False, False, None),
    (4, 128, 8, 8, True, True, None),
    (2048, 1024, 128, 1, False, True, "vec"),     # long batches
    (1037, 1100, 200, 2, True, False, "tok"),      # ... ragged last CTA, d not a multiple of the chunk, E above 128
    (1500, 4096, 8, 2, True, True, None),
]


@pytest.mark.parametrize("T,d,E,k,renorm,bf16,bias_kind", CASES)
def test_router_topk(ctx, T, d, E, k, renorm, bf16, bias_kind):
    seed = T * 7 + E
    x = inputs.activations(seed, 0, T, d, "bf16" if bf16 else "f32")
    Wr = inputs.router_weight(seed, 0, d, E, std=0.05)
    rng = np.random.default_rng(seed)
    bias = None
    if bias_kind == "vec":
        bias = rng.standard_normal(E).astype(np.float32)
    elif bias_kind == "tok":
        bias = rng.standard_normal((T, E)).astype(np.float32)
    ids_ref, gates_ref, logits_ref = oracle.route(x, Wr, bias, k, renorm)
    ids, gates, logits = _route_gpu(ctx, x, bf16, Wr, bias, k, renorm)
    np.testing.assert_allclose(logits, logits_ref, rtol=0, atol=2e-5)
    strict = check_ids(ids, logits_ref, k)
    assert strict >= 0.9 * T
    same = np.all(ids == ids_ref, axis=1)
    np.testing.assert_allclose(gates[same], gates_ref[same], rtol=2e-5, atol=1e-7)
    if renorm:
        np.testing.assert_allclose(gates.sum(axis=1), 1.0, rtol=1e-5)


def test_router_ties_go_to_the_lower_index(ctx):
    # identical router columns give identical logits: the lower index must win
    d, E = 64, 6
    x = inputs.activations(1, 0, 10, d, "f32")
    col = inputs.router_weight(1, 0, d, 1, std=0.1)
    Wr = np.repeat(col, E, axis=1).copy()
    ids, gates, _ = _route_gpu(ctx, x, False, Wr, None, 3, False)
    assert np.array_equal(ids, np.tile(np.array([0, 1, 2], dtype=np.int32), (10, 1)))
    np.testing.assert_allclose(gates, 1.0 / E, rtol=1e-6)


def _permute_gpu(ctx, ids, E):
    flat = np.ascontiguousarray(ids.reshape(-1), dtype=np.int32)
    n = flat.size
    idd = torch.from_numpy(flat).cuda()
    counts = torch.full((E,), -1, dtype=torch.int32, device="cuda")
    off = torch.full((E + 1,), -1, dtype=torch.int32, device="cuda")
    perm = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    slot = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    B.emoe_permute(ctx, idd.data_ptr(), n, E, counts.data_ptr(), off.data_ptr(), perm.data_ptr(), slot.data_ptr(), 0)
    torch.cuda.synchronize()
    return counts.cpu().numpy(), off.cpu().numpy(), perm.cpu().numpy(), slot.cpu().numpy()


@pytest.mark.parametrize("n,E,skew", [(1, 32, 0), (64, 32, 0), (16, 8, 0), (4096, 8, 0), (2048, 128, 1.1),
                                      (1023, 3, 0), (1025, 256, 0), (5000, 1, 0), (3000, 200, 2.0)])
def test_permute_bit_exact(ctx, n, E, skew):
    rng = np.random.default_rng(n + E)
    if skew:
        p = np.arange(1, E + 1, dtype=np.float64) ** -skew
        ids = rng.choice(E, size=n, p=p / p.sum()).astype(np.int32)
    else:
        ids = rng.integers(0, E, size=n).astype(np.int32)
    c_ref, o_ref, p_ref = oracle.permute(ids, E)
    c, o, p, slot = _permute_gpu(ctx, ids, E)
    assert np.array_equal(c, c_ref) and np.array_equal(o, o_ref) and np.array_equal(p, p_ref)
    assert np.array_equal(slot[p], np.arange(n))
    assert B.emoe_device_status(ctx) == B.OK


def test_permute_flags_out_of_range_ids(ctx):
    ids = np.array([0, 1, 7, 1, -1, 2], dtype=np.int32)      # 7 and -1 are outside [0, 4)
    c, o, p, slot = _permute_gpu(ctx, ids, 4)
    assert B.emoe_device_status(ctx) == B.ERR_DEVICE_CHECK
    assert B.emoe_device_status(ctx) == B.OK                  # reading clears the word
    assert c.tolist() == [1, 2, 1, 0] and o.tolist() == [0, 1, 3, 4, 4]
    assert p[:4].tolist() == [0, 1, 3, 5] and slot[2] == -1 and slot[4] == -1
