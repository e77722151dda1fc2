"""Pins for the CPU checker's expert-FFN + combine (paper Sections 1, 2.1, 3.2: only the
Top-K experts of a token are evaluated, each an independent FFN on weights decompressed
as q*s).  Expected values: fp64 dense evaluation with numpy matmul, written without
permutation or grouping; textbook special cases; analytic quantisation bounds."""
import numpy as np
import pytest

import oracle
from paper_2308_14352_b200 import inputs


def _layer(shape, bits, seed, T, std=0.05):
    W = inputs.expert_set(seed, 0, shape, std)
    packed, scales = [], []
    for e in range(shape.n_experts):
        pe, se = [], []
        for m in range(shape.n_matrices):
            p, s = oracle.pack_expert(W[e][m], bits[e], shape.group, shape.scale_dtype)
            pe.append(p)
            se.append(s)
        packed.append(pe)
        scales.append(se)
    x = inputs.activations(seed, 0, T, shape.d_model, shape.act_dtype)
    Wr = inputs.router_weight(seed, 0, shape.d_model, shape.n_experts, std=0.3)
    return W, packed, scales, x, Wr


def _bf16(a):
    import torch

    return torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()


def _dense_expert(xt, mats, act, hidden_bf16):
    """FFN of one expert on fp64 dense matrices mats[m][N][K] for a block of tokens."""
    xt = xt.astype(np.float64)
    if act == "relu":
        h = np.maximum(xt @ mats[0].T, 0.0)
    else:
        a = xt @ mats[0].T
        h = a / (1.0 + np.exp(-a)) * (xt @ mats[1].T)
    h = _bf16(h) if hidden_bf16 else h.astype(np.float32).astype(np.float64)
    return h @ mats[-1].T


def _brute_force(x, shape, bits, packed, scales, ids, gates):
    """Every expert on every token from the dequantised dense weights, masked by the Top-K
    set: no permutation, no grouping."""
    T = x.shape[0]
    dense = [[oracle.dequantize(packed[e][m], scales[e][m], shape.matrix_shape(m)[1], bits[e], shape.group)
              for m in range(shape.n_matrices)] for e in range(shape.n_experts)]
    weight = np.zeros((T, shape.n_experts))
    for t in range(T):
        for j in range(shape.top_k):
            weight[t, ids[t, j]] += float(gates[t, j])
    y = np.zeros((T, shape.d_model))
    for e in range(shape.n_experts):
        y += weight[:, e:e + 1] * _dense_expert(x, dense[e], shape.act, shape.act_dtype == "bf16")
    return y


CASES = [
    ("relu", "f32", 0, "f32", 1, "softmax"),
    ("relu", "bf16", 32, "f16", 1, "softmax"),
    ("relu", "bf16", 32, "f16", 2, "softmax_renorm"),
    ("swiglu", "f32", 0, "f32", 2, "softmax_renorm"),
    ("swiglu", "bf16", 64, "f16", 2, "softmax_renorm"),
    ("swiglu", "bf16", 0, "f16", 3, "softmax"),
]


@pytest.mark.parametrize("act,adt,group,sdt,k,gm", CASES)
def test_against_dense_fp64_brute_force(act, adt, group, sdt, k, gm):
    shape = inputs.small_shape(act, adt, group, sdt, d_model=64, d_ff=128, n_experts=4, top_k=k, gate_mode=gm)
    bits = [2, 4, 8, 4]
    W, packed, scales, x, Wr = _layer(shape, bits, seed=11, T=9)
    y, ids, gates = oracle.moe_forward(x, Wr, None, k, gm == "softmax_renorm", shape.d_ff, act, group,
                                       adt == "bf16", bits, packed, scales)
    ref = _brute_force(x, shape, bits, packed, scales, ids, gates)
    scale = np.abs(ref).max()
    assert scale > 0
    # identical definition, different summation order: fp64 round-off plus the final fp32
    # rounding of y, plus (bf16 mode) rare one-ulp flips of a hidden value at a rounding tie
    tol = 2e-7 if adt == "f32" else 2e-5
    assert np.abs(y - ref).max() / scale < tol


def test_single_expert_is_a_textbook_dense_ffn():
    for act in ("relu", "swiglu"):
        shape = inputs.small_shape(act, "f32", 0, "f32", d_model=32, d_ff=96, n_experts=1, top_k=1)
        W, packed, scales, x, Wr = _layer(shape, [8], seed=3, T=5)
        y, ids, gates = oracle.moe_forward(x, Wr, None, 1, False, shape.d_ff, act, 0, False, [8], packed, scales)
        assert np.all(ids == 0) and np.all(gates == 1.0)
        dense = [oracle.dequantize(packed[0][m], scales[0][m], shape.matrix_shape(m)[1], 8, 0)
                 for m in range(shape.n_matrices)]
        ref = _dense_expert(x, dense, act, False)
        assert np.abs(y - ref).max() / np.abs(ref).max() < 2e-7


def test_dense_equivalence_int8_all_experts_selected():
    """All experts at 8 bits, k = E, renormalised gates: the layer is the softmax-weighted sum
    of all expert FFNs, and must agree with the same sum on the ORIGINAL fp32 weights up to
    the quantisation error, |dW| <= amax/254 per weight."""
    E = 4
    shape = inputs.small_shape("relu", "f32", 0, "f32", d_model=48, d_ff=64, n_experts=E, top_k=E,
                               gate_mode="softmax_renorm")
    bits = [8] * E
    W, packed, scales, x, Wr = _layer(shape, bits, seed=5, T=6)
    y, ids, gates = oracle.moe_forward(x, Wr, None, E, True, shape.d_ff, "relu", 0, False, bits, packed, scales)
    from scipy.special import softmax

    p = softmax((x.astype(np.float64) @ Wr.astype(np.float64)).astype(np.float32).astype(np.float64), axis=1)
    ref = np.zeros((6, shape.d_model))
    bound = np.zeros((6, shape.d_model))
    xa = np.abs(x.astype(np.float64))
    for e in range(E):
        Win, Wout = W[e][0].astype(np.float64), W[e][1].astype(np.float64)
        h = np.maximum(x.astype(np.float64) @ Win.T, 0.0)
        ref += p[:, e:e + 1] * (h @ Wout.T)
        # first-order propagation of |dW| <= amax_row/254 through ReLU FFN (ReLU is 1-Lipschitz)
        din = np.abs(Win).max(axis=1) / 254.0            # per hidden unit
        dout = np.abs(Wout).max(axis=1) / 254.0          # per output channel
        dh = xa.sum(axis=1, keepdims=True) * din[None, :]
        bound += p[:, e:e + 1] * (dh @ np.abs(Wout).T + (h + dh).sum(axis=1, keepdims=True) * dout[None, :])
    assert np.all(np.abs(y - ref) <= bound * 1.0001 + 1e-7)
    # and the bound is not vacuous: quantisation did change the result, by far less than y
    assert 0 < np.abs(y - ref).max() < 0.05 * np.abs(ref).max()


def test_unselected_expert_does_not_matter():
    shape = inputs.small_shape("relu", "bf16", 32, "f16", d_model=64, d_ff=64, n_experts=4, top_k=1)
    bits = [4, 4, 4, 4]
    W, packed, scales, x, Wr = _layer(shape, bits, seed=8, T=4)
    ids = np.array([[0], [2], [0], [2]], dtype=np.int32)
    gates = np.full((4, 1), 0.5, dtype=np.float32)
    y0 = oracle.moe_ffn_combine(x, shape.d_ff, "relu", 32, True, bits, packed, scales, ids, gates)
    packed[1][0] = (packed[1][0] ^ 0x5A).astype(np.uint8)      # experts 1 and 3 are never selected
    scales[3][1] = scales[3][1] * 3.0
    y1 = oracle.moe_ffn_combine(x, shape.d_ff, "relu", 32, True, bits, packed, scales, ids, gates)
    assert np.array_equal(y0, y1)
    packed[2][0] = (packed[2][0] ^ 0x11).astype(np.uint8)      # a selected expert does matter
    y2 = oracle.moe_ffn_combine(x, shape.d_ff, "relu", 32, True, bits, packed, scales, ids, gates)
    assert not np.array_equal(y0, y2)
    assert np.array_equal(y0[[0, 2]], y2[[0, 2]])


def test_gate_linearity_and_combine_order():
    """y is linear in the gates: doubling them doubles y; with k = 2 and the two picks swapped
    (ids and gates together) the result is unchanged."""
    shape = inputs.small_shape("swiglu", "f32", 0, "f32", d_model=32, d_ff=64, n_experts=3, top_k=2)
    bits = [8, 4, 2]
    W, packed, scales, x, Wr = _layer(shape, bits, seed=9, T=5)
    ids = np.array([[0, 1], [1, 2], [2, 0], [0, 2], [1, 0]], dtype=np.int32)
    gates = np.array([[0.75, 0.25], [0.5, 0.5], [0.125, 0.5], [1.0, 0.0], [0.25, 0.25]], dtype=np.float32)
    y = oracle.moe_ffn_combine(x, shape.d_ff, "swiglu", 0, False, bits, packed, scales, ids, gates)
    y2 = oracle.moe_ffn_combine(x, shape.d_ff, "swiglu", 0, False, bits, packed, scales, ids, 2 * gates)
    np.testing.assert_allclose(y2, 2 * y, rtol=1e-6, atol=1e-9)
    ys = oracle.moe_ffn_combine(x, shape.d_ff, "swiglu", 0, False, bits, packed, scales, ids[:, ::-1], gates[:, ::-1])
    np.testing.assert_allclose(ys, y, rtol=1e-6, atol=1e-9)
    # a zero gate removes that expert's contribution: token 3 equals gate 1.0 * expert 0 alone
    y_single = oracle.moe_ffn_combine(x[3:4], shape.d_ff, "swiglu", 0, False, bits, packed, scales,
                                      np.array([[0, 1]], dtype=np.int32), np.array([[1.0, 0.0]], dtype=np.float32))
    np.testing.assert_allclose(y_single[0], y[3], rtol=1e-6, atol=1e-9)


def test_spot_check_helpers_agree_with_full_evaluation():
    shape = inputs.small_shape("swiglu", "bf16", 32, "f16", d_model=64, d_ff=96, n_experts=2, top_k=1)
    bits = [4, 2]
    W, packed, scales, x, Wr = _layer(shape, bits, seed=10, T=3)
    ids = np.array([[1], [0], [1]], dtype=np.int32)
    gates = np.ones((3, 1), dtype=np.float32)
    y, h, o = oracle.moe_ffn_combine(x, shape.d_ff, "swiglu", 32, True, bits, packed, scales, ids, gates, True)
    hp = oracle.hidden_for_pair(x[2], shape.d_ff, "swiglu", 32, True, 2, packed[1], scales[1])
    assert np.array_equal(hp.astype(np.float32), h[2])
    oc = oracle.output_channels(hp, 32, 2, packed[1][2], scales[1][2], [0, 5, 63])
    assert np.array_equal(oc, o[2, [0, 5, 63]])
