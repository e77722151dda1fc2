"""Pins for the CPU checker's quantise / pack / dequantise functions (paper Section 3.2).

The expected values here come from hand-computed rows (tests/golden/quant_rows.txt), from
closed forms the definition fixes, from numpy's own float16 type, and from exhaustive
enumeration: none comes from the checker itself or from the GPU library."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "quant_rows.txt")


def _golden_rows():
    rows = []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            bits, group, sdt, w, q, s, b = [p.strip() for p in line.split("|")]
            rows.append((int(bits), int(group), sdt,
                         np.array(w.split(), dtype=np.float64).astype(np.float32),
                         np.array(q.split(), dtype=np.int64),
                         np.array(s.split(), dtype=np.float64),
                         np.array([int(v, 16) for v in b.split()], dtype=np.uint8)))
    return rows


@pytest.mark.parametrize("row", _golden_rows(), ids=lambda r: f"int{r[0]}_g{r[1]}_{r[2]}")
def test_hand_computed_rows(row):
    bits, group, sdt, w, q_exp, s_exp, bytes_exp = row
    q, s = oracle.quantize(w[None, :], bits, group, sdt)
    assert np.array_equal(q[0].astype(np.int64), q_exp)
    assert np.array_equal(s[0].astype(np.float64), s_exp)
    packed = oracle.pack(q, bits)
    assert np.array_equal(packed[0], bytes_exp)
    assert np.array_equal(oracle.unpack(bytes_exp[None, :], w.size, bits)[0].astype(np.int64), q_exp)
    Wt = oracle.dequantize(packed, s, w.size, bits, group)
    G = group if group else w.size
    assert np.array_equal(Wt[0], q_exp.astype(np.float64) * np.repeat(s_exp, G))


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_pack_unpack_exhaustive_codes_at_every_position(bits):
    """Every code value at every field position of a byte group survives pack -> unpack, and
    lands in the bit field the storage format names (low bits first)."""
    lo, hi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    per_byte = 8 // bits
    K = 4 * per_byte
    for pos in range(K):
        for code in range(lo, hi + 1):
            q = np.zeros((1, K), dtype=np.int8)
            q[0, pos] = code
            packed = oracle.pack(q, bits)
            expect = np.zeros(K * bits // 8, dtype=np.uint8)
            expect[(pos * bits) // 8] = (code & ((1 << bits) - 1)) << ((pos * bits) % 8)
            assert np.array_equal(packed[0], expect)
            assert np.array_equal(oracle.unpack(packed, K, bits), q)
    rng = np.random.default_rng(0)
    q = rng.integers(lo, hi + 1, size=(5, 64)).astype(np.int8)
    assert np.array_equal(oracle.unpack(oracle.pack(q, bits), 64, bits), q)


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("group,sdt", [(0, "f32"), (0, "f16"), (32, "f16"), (128, "f16"), (128, "f32")])
def test_quantise_closed_forms(bits, group, sdt):
    rng = np.random.default_rng(bits * 100 + group)
    N, K = 7, 256
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    W[3, :] = 0.0  # an all-zero channel
    q, s = oracle.quantize(W, bits, group, sdt)
    qmax = (1 << (bits - 1)) - 1
    G = group if group else K
    Wg = W.reshape(N, K // G, G)
    qg = q.reshape(N, K // G, G).astype(np.int64)
    amax = np.abs(Wg).max(axis=2)
    # scale = max-abs / range, in fp32, then stored in the scale channel's type
    s32 = (amax / np.float32(qmax)).astype(np.float32)
    s_expected = s32.astype(np.float16).astype(np.float32) if sdt == "f16" else s32
    assert np.array_equal(s, s_expected)
    # the max-abs element maps to +-qmax, zero maps to zero, codes stay in range
    idx = np.abs(Wg).argmax(axis=2)
    top = np.take_along_axis(qg, idx[..., None], axis=2)[..., 0]
    sign = np.sign(np.take_along_axis(Wg, idx[..., None], axis=2)[..., 0])
    assert np.array_equal(top, (sign * qmax).astype(np.int64))
    assert np.all(np.abs(qg) <= qmax)
    assert np.all(q[3] == 0) and np.all(s[3] == 0)
    # reconstruction error at most half a step (plus the fp16 rounding of the scale)
    err = np.abs(Wg.astype(np.float64) - qg * s.astype(np.float64)[..., None])
    slack = amax.astype(np.float64)[..., None] * 2.0 ** -11 if sdt == "f16" else 0.0
    assert np.all(err <= 0.5 * s.astype(np.float64)[..., None] * (1 + 1e-6) + slack)
    # dequantisation is exactly q*s; with an fp16 scale (11 significant bits) times a code of
    # at most 7 bits the product is also representable in fp32
    Wt = oracle.dequantize(oracle.pack(q, bits), s, K, bits, group)
    assert np.array_equal(Wt.reshape(N, K // G, G), qg * s.astype(np.float64)[..., None])
    if sdt == "f16":
        assert np.array_equal(Wt.astype(np.float32).astype(np.float64), Wt)


def test_round_half_to_even_codes():
    # scale is exactly 1 (amax = qmax), so w/s = w: halves must go to the even neighbour
    w = np.array([[7.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5]], dtype=np.float32)
    q, s = oracle.quantize(w, 4, 0, "f32")
    assert s[0, 0] == 1.0
    assert q[0].tolist() == [7, 0, 2, 2, 0, -2, -2, 4]


def test_fp16_and_bf16_rounding_against_library_types():
    import torch

    rng = np.random.default_rng(1)
    vals = np.concatenate([
        rng.standard_normal(2000) * 10.0 ** rng.integers(-9, 5, 2000),
        [0.0, 1.0, 65504.0, 65519.9, 2.0 ** -24, 2.0 ** -25, 1.5 * 2.0 ** -24, 2.5 * 2.0 ** -24, 1 + 2.0 ** -11, 1 + 3 * 2.0 ** -11],
    ])
    for v in vals:
        v32 = np.float32(v)
        if abs(v32) < 65520:
            assert oracle.round_f16(float(v32)) == float(np.float16(v32))
    t = torch.tensor(vals, dtype=torch.float64)
    # a double that is exactly a float goes through torch's fp32 -> bf16 rounding unchanged
    t32 = t.to(torch.float32)
    ref = t32.to(torch.bfloat16).to(torch.float64)
    got = torch.tensor([oracle.round_bf16(float(a)) for a in t32.to(torch.float64)], dtype=torch.float64)
    assert torch.equal(ref, got)
    # single rounding from fp64: just above a bf16 tie must round up even though fp32 rounding
    # of the same number lands exactly on the tie (which would then go to even, i.e. down)
    tie = 1.0 + 2.0 ** -8          # halfway between bf16 1.0 and 1.0078125
    assert oracle.round_bf16(tie) == 1.0
    assert oracle.round_bf16(tie + 2.0 ** -40) == 1.0078125
    assert oracle.round_bf16(3.0 * 2.0 ** -134) == 2.0 ** -132   # subnormal tie: 1.5 quanta -> 2


# ---- moving a stored matrix to another bitwidth (Section 3.2, bitwidth selection) -------------
REQUANT_GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "requant_rows.txt")


def _requant_rows():
    rows = []
    with open(REQUANT_GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            bi, bo, group, sdt, b_in, s_in, q_out, s_out, b_out = [p.strip() for p in line.split("|")]
            rows.append((int(bi), int(bo), int(group), sdt,
                         np.array([int(v, 16) for v in b_in.split()], dtype=np.uint8),
                         np.array(s_in.split(), dtype=np.float64).astype(np.float32),
                         np.array(q_out.split(), dtype=np.int64),
                         np.array(s_out.split(), dtype=np.float64),
                         np.array([int(v, 16) for v in b_out.split()], dtype=np.uint8)))
    return rows


@pytest.mark.parametrize("row", _requant_rows(), ids=lambda r: f"int{r[0]}_to_int{r[1]}_g{r[2]}_{r[3]}")
def test_requantize_hand_computed_rows(row):
    bi, bo, group, sdt, b_in, s_in, q_exp, s_exp, b_exp = row
    K = b_in.size * 8 // bi
    packed, scales = oracle.requantize(b_in[None, :], s_in[None, :], K, bi, bo, group, sdt)
    assert np.array_equal(oracle.unpack(packed, K, bo)[0].astype(np.int64), q_exp)
    assert np.array_equal(scales[0].astype(np.float64), s_exp)
    assert np.array_equal(packed[0], b_exp)


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("group", [0, 32])
def test_requantize_to_the_same_width_is_the_identity(bits, group):
    """Every non-zero group of a stored matrix holds a code of magnitude qmax, so its max-abs is
    qmax * s exactly (fp16 scale: 11 + 7 significant bits) and the new scale (qmax * s) / qmax is s
    again; the quotients (q * s) / s are the codes themselves."""
    rng = np.random.default_rng(5 + bits)
    W = (rng.standard_normal((24, 128)) * 0.02).astype(np.float32)
    W[3, :] = 0.0  # an all-zero channel stays all zero
    packed, scales = oracle.pack_expert(W, bits, group, "f16")
    packed2, scales2 = oracle.requantize(packed, scales, 128, bits, bits, group, "f16")
    assert np.array_equal(packed2, packed)
    assert np.array_equal(scales2, scales)


@pytest.mark.parametrize("bits_in,bits_out", [(8, 4), (8, 2), (4, 2), (2, 4), (4, 8)])
@pytest.mark.parametrize("sdt", ["f16", "f32"])
def test_requantize_closed_forms(bits_in, bits_out, sdt):
    """The largest stored weight of a group maps to +-qmax of the new width, the new scale is the
    group's largest decompressed magnitude over that qmax, and no weight moves by more than half
    a new step (plus the fp16 rounding of the scale)."""
    rng = np.random.default_rng(11 * bits_in + bits_out)
    N, K, G = 16, 256, 128
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    packed, scales = oracle.pack_expert(W, bits_in, G, sdt)
    Wt = oracle.dequantize(packed, scales, K, bits_in, G).astype(np.float32).astype(np.float64)
    packed2, scales2 = oracle.requantize(packed, scales, K, bits_in, bits_out, G, sdt)
    q2 = oracle.unpack(packed2, K, bits_out).astype(np.int64)
    qmax = (1 << (bits_out - 1)) - 1
    amax = np.abs(Wt).reshape(N, K // G, G).max(axis=2)
    s32 = (amax.astype(np.float32) / np.float32(qmax)).astype(np.float32)
    expect_s = s32.astype(np.float16).astype(np.float32) if sdt == "f16" else s32
    assert np.array_equal(scales2, expect_s)
    Wt2 = q2 * np.repeat(scales2.astype(np.float64), G, axis=1)
    assert np.all(np.abs(q2) <= qmax)
    at_max = np.abs(Wt) == np.repeat(amax, G, axis=1)
    assert np.all(np.abs(q2[at_max & (np.repeat(amax, G, axis=1) > 0)]) == qmax)
    slack = np.repeat(amax, G, axis=1) * 2.0 ** -11 if sdt == "f16" else 0.0
    assert np.all(np.abs(Wt2 - Wt) <= np.repeat(scales2.astype(np.float64), G, axis=1) / 2 + slack + 1e-12)


# ---- the full-range reading of the code range (Section 3.2) -----------------------------------
FULL_RANGE_GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "full_range_rows.txt")


def _full_range_rows(kind):
    rows = []
    with open(FULL_RANGE_GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = [p.strip() for p in line.split("|")]
            if parts[0] == kind:
                rows.append(parts[1:])
    return rows


@pytest.mark.parametrize("row", _full_range_rows("pack"), ids=lambda r: f"int{r[0]}_g{r[1]}_{r[2]}")
def test_full_range_hand_computed_rows(row):
    bits, group, sdt = int(row[0]), int(row[1]), row[2]
    w = np.array(row[3].split(), dtype=np.float64).astype(np.float32)
    q_exp = np.array(row[4].split(), dtype=np.int64)
    s_exp = np.array(row[5].split(), dtype=np.float64)
    bytes_exp = np.array([int(v, 16) for v in row[6].split()], dtype=np.uint8)
    q, s = oracle.quantize(w[None, :], bits, group, sdt, full_range=True)
    assert np.array_equal(q[0].astype(np.int64), q_exp)
    assert np.array_equal(s[0].astype(np.float64), s_exp)
    packed, s2 = oracle.pack_expert(w[None, :], bits, group, sdt, full_range=True)
    assert np.array_equal(packed[0], bytes_exp) and np.array_equal(s2, s)
    assert np.array_equal(oracle.unpack(packed, w.size, bits)[0].astype(np.int64), q_exp)


@pytest.mark.parametrize("row", _full_range_rows("requant"), ids=lambda r: f"int{r[0]}_to_int{r[1]}")
def test_full_range_requantize_hand_computed_rows(row):
    bi, bo, group, sdt = int(row[0]), int(row[1]), int(row[2]), row[3]
    b_in = np.array([int(v, 16) for v in row[4].split()], dtype=np.uint8)
    s_in = np.array(row[5].split(), dtype=np.float64).astype(np.float32)
    q_exp = np.array(row[6].split(), dtype=np.int64)
    s_exp = np.array(row[7].split(), dtype=np.float64)
    b_exp = np.array([int(v, 16) for v in row[8].split()], dtype=np.uint8)
    K = b_in.size * 8 // bi
    packed, scales = oracle.requantize(b_in[None, :], s_in[None, :], K, bi, bo, group, sdt, full_range=True)
    assert np.array_equal(oracle.unpack(packed, K, bo)[0].astype(np.int64), q_exp)
    assert np.array_equal(scales[0].astype(np.float64), s_exp)
    assert np.array_equal(packed[0], b_exp)


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("group", [0, 32])
def test_full_range_properties(bits, group):
    """What the definition fixes at any size: codes lie in [-2^(b-1), 2^(b-1)-1]; the scale is
    max-abs / 2^(b-1); a channel's most negative weight of magnitude max-abs takes the extra code;
    the reconstruction error of a weight that is not clamped is at most half a step; and a matrix
    whose weights are whole multiples of the step comes back exactly except +max-abs."""
    rng = np.random.default_rng(11 + bits)
    W = (rng.standard_normal((16, 128)) * 0.05).astype(np.float32)
    W[5, :] = 0.0
    half = 1 << (bits - 1)
    q, s = oracle.quantize(W, bits, group, "f32", full_range=True)
    G = group or 128
    assert q.min() >= -half and q.max() <= half - 1
    amax = np.abs(W.reshape(16, 128 // G, G)).max(axis=2)
    assert np.array_equal(s, (amax / np.float32(half)).astype(np.float32))
    step = np.repeat(s, G, axis=1).astype(np.float64)
    Wt = q.astype(np.float64) * step
    clamped = (W.astype(np.float64) > (half - 1 + 0.5) * step)
    err = np.abs(Wt - W.astype(np.float64))
    assert np.all(err[~clamped] <= 0.5 * step[~clamped] * (1 + 1e-6) + 1e-12)
    # the negative extreme of a group maps to -2^(b-1) exactly
    Wg = W.reshape(16, 128 // G, G)
    qg = q.reshape(16, 128 // G, G)
    for n in range(16):
        for g in range(128 // G):
            k = int(np.argmax(np.abs(Wg[n, g])))
            if Wg[n, g, k] < 0:
                assert qg[n, g, k] == -half
    # symmetric and full-range agree on what they share: same codes wherever the symmetric scale
    # is used with the symmetric clamp (sanity: the default did not change)
    q0, s0 = oracle.quantize(W, bits, group, "f32")
    assert q0.min() >= -(half - 1) and np.array_equal(s0, (amax / np.float32(half - 1)).astype(np.float32))


def test_full_range_int2_has_four_levels_and_lower_error_on_gaussian_weights():
    """Ternary INT2 (the default reading) maps most of a Gaussian group to 0; the four-level reading
    halves the step.  On seeded Gaussian weights with groups of 128 its mean squared error is lower."""
    rng = np.random.default_rng(3)
    W = (rng.standard_normal((64, 512)) * 0.02).astype(np.float32)
    q3, s3 = oracle.quantize(W, 2, 128, "f16")
    q4, s4 = oracle.quantize(W, 2, 128, "f16", full_range=True)
    assert set(np.unique(q3)) == {-1, 0, 1} and set(np.unique(q4)) == {-2, -1, 0, 1}
    e3 = np.mean((q3 * np.repeat(s3, 128, axis=1) - W) ** 2)
    e4 = np.mean((q4 * np.repeat(s4, 128, axis=1) - W) ** 2)
    assert e4 < e3
