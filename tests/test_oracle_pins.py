"""Pins of the CPU oracle against things other than itself: hand-computed examples of
Eq. 4, dot products and box sums a person can verify, float64 cross-correlation from a
library routine, exact rational arithmetic, library pooling, and the invariants the paper
states (outputs inside [0, max_int], h_i requantises to max_int, concatenation and
addition operands share one ratio)."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
from scipy import signal

from oracle import layers as L
from oracle import planner as P

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
ONE = ([1], [0], [0])   # mul, shift, h_i of an identity requantisation


def _examples():
    rows = []
    with open(os.path.join(GOLDEN, "round_shift_examples.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if len(line) == 4:
                rows.append(tuple(int(v) for v in line))
    return rows


# ---------------------------------------------------------------- Eq. 4 bracket
def test_round_shift_hand_examples():
    rows = _examples()
    assert len(rows) >= 20
    for Y, mul, shift, V in rows:
        assert L.round_shift(Y * mul, shift) == V, (Y, mul, shift)


def test_round_shift_equals_exact_rational_rounding():
    rng = np.random.default_rng(7)
    for _ in range(2000):
        v = int(rng.integers(-2 ** 40, 2 ** 40))
        s = int(rng.integers(0, 41))
        exact = P.round_half_up(Fraction(v, 1 << s))
        assert L.round_shift(v, s) == exact
        if s:
            assert exact == (v + (1 << (s - 1))) >> s     # python ints: floor shift


def test_layer_applies_hand_examples_through_the_whole_tail():
    """1x1 kernel with weight 1 and C_in = 1: Y = x + b, so the layer output must be the
    golden V for Y reachable with an 8-bit x and an int32 bias."""
    for Y, mul, shift, V in _examples():
        x = np.array([[[[7]]]], dtype=np.uint8)
        W = np.ones((1, 1, 1, 1), dtype=np.int8)
        out, ovf = L.conv(x, W, [Y - 7], [mul], [shift], [2 ** 31 - 1], out_dtype=L.S8,
                          brelu=False, out_lo=-128, out_hi=127)
        assert not ovf
        assert int(out[0, 0, 0, 0]) == max(-128, min(127, V))


# ---------------------------------------------------------------- hand-checkable layers
def test_single_pixel_dot_product():
    x = np.array([[[[3, 0, 255, 17]]]], dtype=np.uint8)
    W = np.array([[[[2, -5, 1, -1]]], [[[-127, 127, 0, 4]]]], dtype=np.int8)
    b = np.array([10, -20], dtype=np.int32)
    # 3*2 + 255 - 17 + 10 = 254 ;  -381 + 68 - 20 = -333
    out, _ = L.conv(x, W, b, *ONE, out_dtype=L.I32, brelu=False)
    assert out.reshape(-1).tolist() == [254, -333]
    # BReLU to [0, 200], then *3/4 rounded half up: 200*3/4 = 150 ; 0
    out, _ = L.conv(x, W, b, [3], [2], [200])
    assert out.reshape(-1).tolist() == [150, 0]
    # raw-128 input: (3-128)*2 + (255-128) - (17-128) + 640 + 10 = 638 ... (0-128)*-5 = 640
    out, _ = L.conv(x, W, b, *ONE, in_dtype=L.U8_RAW128, out_dtype=L.I32, brelu=False)
    assert int(out[0, 0, 0, 0]) == (3 - 128) * 2 + (0 - 128) * -5 + (255 - 128) - (17 - 128) + 10


def test_one_hot_kernel_shifts_and_ones_kernel_box_sums():
    rng = np.random.default_rng(3)
    x = rng.integers(0, 256, size=(1, 3, 3, 1), dtype=np.uint8)
    for r in range(3):
        for s in range(3):
            W = np.zeros((1, 3, 3, 1), dtype=np.int8)
            W[0, r, s, 0] = 1
            out, _ = L.conv(x, W, [0], *ONE, pad=1, out_dtype=L.I32, brelu=False)
            padded = np.zeros((5, 5), dtype=np.int64)
            padded[1:4, 1:4] = x[0, :, :, 0]
            assert np.array_equal(out[0, :, :, 0], padded[r:r + 3, s:s + 3])
    W = np.ones((1, 3, 3, 1), dtype=np.int8)
    out, _ = L.conv(x, W, [0], *ONE, pad=1, out_dtype=L.I32, brelu=False)
    xi = x[0, :, :, 0].astype(np.int64)
    assert int(out[0, 1, 1, 0]) == xi.sum()
    assert int(out[0, 0, 0, 0]) == xi[:2, :2].sum()
    assert int(out[0, 2, 1, 0]) == xi[1:, :].sum()
    # raw-128 input: padding is zero AFTER the re-normalisation, so a corner sums four values
    out, _ = L.conv(x, W, [0], *ONE, pad=1, in_dtype=L.U8_RAW128, out_dtype=L.I32, brelu=False)
    assert int(out[0, 0, 0, 0]) == (xi[:2, :2] - 128).sum()


# ---------------------------------------------------------------- library cross-correlation
def _xcorr_f64(xv, W, stride, pad):
    """float64 cross-correlation of integer values with scipy (exact below 2^53)."""
    n, h, w, c = xv.shape
    co, kh, kw, _ = W.shape
    xp = np.zeros((n, h + 2 * pad, w + 2 * pad, c), dtype=np.float64)
    xp[:, pad:pad + h, pad:pad + w, :] = xv
    full_h, full_w = h + 2 * pad - kh + 1, w + 2 * pad - kw + 1
    out = np.zeros((n, full_h, full_w, co))
    for i in range(n):
        for o in range(co):
            for ch in range(c):
                out[i, :, :, o] += signal.correlate2d(xp[i, :, :, ch], W[o, :, :, ch].astype(np.float64), mode="valid")
    return out[:, ::stride, ::stride, :]


@pytest.mark.parametrize("k,stride,pad,c_in,c_out,h,w", [
    (1, 1, 0, 16, 5, 5, 7), (3, 1, 1, 3, 4, 6, 5), (3, 2, 1, 16, 3, 7, 9), (5, 1, 2, 1, 6, 8, 6),
    (5, 2, 0, 3, 2, 9, 9), (7, 2, 3, 3, 4, 11, 10), (3, 1, 0, 48, 2, 5, 5), (3, 2, 2, 64, 3, 6, 7),
    (1, 2, 0, 16, 4, 6, 6), (7, 1, 3, 1, 2, 7, 7), (3, 1, 3, 2, 2, 4, 4),
])
@pytest.mark.parametrize("in_dtype", [L.U8, L.U8_RAW128, L.S8])
def test_plain_integer_convolution_equals_float64_cross_correlation(k, stride, pad, c_in, c_out, h, w, in_dtype):
    rng = np.random.default_rng(k * 100 + stride * 10 + pad + c_in)
    if in_dtype == L.S8:
        x = rng.integers(-128, 128, size=(2, h, w, c_in), dtype=np.int8)
        xv = x.astype(np.float64)
    else:
        x = rng.integers(0, 256, size=(2, h, w, c_in), dtype=np.uint8)
        xv = x.astype(np.float64) - (128 if in_dtype == L.U8_RAW128 else 0)
    W = rng.integers(-127, 128, size=(c_out, k, k, c_in), dtype=np.int8)
    b = rng.integers(-4096, 4097, size=(c_out,), dtype=np.int32)
    out, ovf = L.conv(x, W, b, *ONE, stride=stride, pad=pad, in_dtype=in_dtype, out_dtype=L.I32,
                      brelu=False, check_partial=True)
    assert not ovf
    ref = _xcorr_f64(xv, W, stride, pad) + b.astype(np.float64)
    assert out.shape == ref.shape
    assert np.array_equal(out.astype(np.float64), ref)


def test_tail_matches_exact_rationals_on_a_random_layer():
    rng = np.random.default_rng(11)
    x = rng.integers(0, 256, size=(1, 6, 6, 16), dtype=np.uint8)
    W = rng.integers(-127, 128, size=(8, 3, 3, 16), dtype=np.int8)
    b = rng.integers(-4096, 4097, size=(8,), dtype=np.int32)
    mul = rng.integers(100, 400, size=8).astype(np.int32)
    shift = rng.integers(14, 18, size=8).astype(np.int32)
    h_i = rng.integers(20000, 90000, size=8).astype(np.int32)
    Y = _xcorr_f64(x.astype(np.float64), W, 1, 1) + b
    out, _ = L.conv(x, W, b, mul, shift, h_i, pad=1)           # per-channel parameters
    for idx in np.ndindex(*Y.shape):
        co = idx[3]
        y = min(max(int(Y[idx]), 0), int(h_i[co]))
        v = P.round_half_up(Fraction(y * int(mul[co]), 1 << int(shift[co])))
        assert int(out[idx]) == min(max(v, 0), 255)


# ---------------------------------------------------------------- invariants
def test_outputs_stay_in_range_and_requant_is_monotone():
    rng = np.random.default_rng(5)
    q = P.brelu_params(6.0, 24498.7, 255)
    assert L.round_shift(q["h_i"] * q["mul"], q["shift"]) == 255
    ys = np.sort(rng.integers(-10 ** 6, 10 ** 6, size=500))
    prev = -1
    for y in ys:
        yc = min(max(int(y), 0), q["h_i"])
        v = L.round_shift(yc * q["mul"], q["shift"])
        assert 0 <= v <= 255 and v >= prev
        prev = v


def test_mul_shift_scaling_and_bias_linearity():
    rng = np.random.default_rng(6)
    x = rng.integers(0, 256, size=(1, 5, 5, 16), dtype=np.uint8)
    W = rng.integers(-127, 128, size=(4, 3, 3, 16), dtype=np.int8)
    b = rng.integers(-4096, 4097, size=(4,), dtype=np.int32)
    a, _ = L.conv(x, W, b, [200], [16], [80000], pad=1)
    c, _ = L.conv(x, W, b, [400], [17], [80000], pad=1)
    assert np.array_equal(a, c)                     # doubling mul and adding 1 to shift
    # adding c * 2^shift / mul (integral) to the bias adds c to the unclamped output
    u0, _ = L.conv(x, W, b, [256], [16], [0], pad=1, brelu=False, out_dtype=L.S8, out_lo=-128, out_hi=127,
                   out_zero=0)
    u1, _ = L.conv(x, W, b + 3 * 256, [256], [16], [0], pad=1, brelu=False, out_dtype=L.S8, out_lo=-128,
                   out_hi=127)
    inside = (u0.astype(int) > -120) & (u0.astype(int) < 120)
    assert inside.any()
    assert np.array_equal(u1.astype(int)[inside], u0.astype(int)[inside] + 3)


def test_clamp_then_requant_equals_requant_then_clamp_when_h_i_maps_to_max_int():
    q = P.brelu_params_from_h_ri(146992, 1.0, 255)
    for y in list(range(-5, 5)) + list(range(q["h_i"] - 2000, q["h_i"] + 2000, 7)):
        pre = L.round_shift(min(max(y, 0), q["h_i"]) * q["mul"], q["shift"])
        post = min(max(L.round_shift(y * q["mul"], q["shift"]), 0), 255)
        assert pre == post


def test_concat_through_channel_offsets_equals_host_concatenation():
    rng = np.random.default_rng(8)
    x = rng.integers(0, 256, size=(2, 6, 7, 64), dtype=np.uint8)
    Wa = rng.integers(-127, 128, size=(16, 5, 5, 64), dtype=np.int8)
    Wb = rng.integers(-127, 128, size=(32, 3, 3, 64), dtype=np.int8)
    ba = rng.integers(-4096, 4097, size=(16,), dtype=np.int32)
    bb = rng.integers(-4096, 4097, size=(32,), dtype=np.int32)
    cat = np.full((2, 6, 7, 48), 77, dtype=np.uint8)
    L.conv(x, Wa, ba, [130], [17], [257103], pad=2, out=cat, out_c_offset=0)
    L.conv(x, Wb, bb, [136], [17], [245760], pad=1, out=cat, out_c_offset=16)
    a, _ = L.conv(x, Wa, ba, [130], [17], [257103], pad=2)
    b, _ = L.conv(x, Wb, bb, [136], [17], [245760], pad=1)
    assert np.array_equal(cat, np.concatenate([a, b], axis=3))
    # reading a channel slice of the concatenated tensor
    Wc = rng.integers(-127, 128, size=(4, 3, 3, 32), dtype=np.int8)
    s1, _ = L.conv(cat, Wc, [0] * 4, *ONE, pad=1, in_c_offset=16, c_in=32, out_dtype=L.I32, brelu=False)
    s2, _ = L.conv(np.ascontiguousarray(cat[..., 16:48]), Wc, [0] * 4, *ONE, pad=1, out_dtype=L.I32, brelu=False)
    assert np.array_equal(s1, s2)


def test_fused_skip_equals_raw_convolution_followed_by_add_requant():
    rng = np.random.default_rng(9)
    x = rng.integers(0, 256, size=(2, 5, 6, 16), dtype=np.uint8)
    W = rng.integers(-127, 128, size=(32, 1, 1, 16), dtype=np.int8)
    b = rng.integers(-4096, 4097, size=(32,), dtype=np.int32)
    for skip_dtype, lo, hi, zero in ((L.U8, 0, 256, 0), (L.I32, -200000, 200000, 0), (L.U8_RAW128, 0, 256, 128)):
        npdt = np.int32 if skip_dtype == L.I32 else np.uint8
        S = rng.integers(lo, hi, size=(2, 5, 6, 32)).astype(npdt)
        fused, _ = L.conv(x, W, b, [150], [17], [220000], skip=S, skip_dtype=skip_dtype, skip_mul=811, skip_shift=3)
        Y, _ = L.conv(x, W, b, *ONE, out_dtype=L.I32, brelu=False)
        two, _ = L.add_requant(S, Y, a_dtype=L.U8 if skip_dtype != L.I32 else L.I32, b_dtype=L.I32, a_zero=zero,
                               mul_a=811, sh_a=3, mul_b=1, sh_b=0, brelu=True, h_i=220000, mul=150, shift=17)
        assert np.array_equal(fused, two)
        # and against exact rationals on a few elements
        for idx in [(0, 0, 0, 0), (1, 4, 5, 31), (0, 2, 3, 7)]:
            s = int(S[idx]) - zero
            y = int(Y[idx]) + P.round_half_up(Fraction(s * 811, 8))
            v = P.round_half_up(Fraction(min(max(y, 0), 220000) * 150, 1 << 17))
            assert int(fused[idx]) == min(max(v, 0), 255)


def test_overflow_is_reported():
    x = np.full((1, 8, 8, 64), 255, dtype=np.uint8)
    W = np.full((1, 7, 7, 64), 127, dtype=np.int8)
    _, ovf = L.conv(x, W, [2 ** 31 - 1 - 255 * 127 * 64 * 49 + 100], *ONE, pad=3, out_dtype=L.I32, brelu=False)
    assert ovf
    _, ovf = L.conv(x, W, [0], *ONE, pad=3, out_dtype=L.I32, brelu=False, check_partial=True)
    assert not ovf
    # partial sums can overflow while the final sum does not: + then - of large products
    x2 = np.full((1, 1, 1, 2 * 70000), 255, dtype=np.uint8)
    W2 = np.concatenate([np.full(70000, 127), np.full(70000, -127)]).astype(np.int8).reshape(1, 1, 1, -1)
    _, ovf = L.conv(x2, W2, [0], *ONE, out_dtype=L.I32, brelu=False)
    assert not ovf
    _, ovf = L.conv(x2, W2, [0], *ONE, out_dtype=L.I32, brelu=False, check_partial=True)
    assert ovf


# ---------------------------------------------------------------- pooling
def test_maxpool_equals_library_maxpool():
    rng = np.random.default_rng(10)
    for (h, w, k, s, p) in [(9, 11, 3, 2, 1), (8, 8, 3, 2, 1), (7, 5, 2, 2, 0), (6, 6, 3, 1, 1)]:
        x = rng.integers(0, 256, size=(2, h, w, 5), dtype=np.uint8)
        ref = torch.nn.functional.max_pool2d(torch.from_numpy(x.astype(np.float32)).permute(0, 3, 1, 2), k, s, p)
        got = L.maxpool(x, k, s, p)
        assert np.array_equal(got, ref.permute(0, 2, 3, 1).numpy().astype(np.uint8))


def test_avgpool_is_rounded_exact_mean():
    rng = np.random.default_rng(12)
    x = rng.integers(0, 256, size=(3, 7, 7, 9), dtype=np.uint8)
    m, s = P.avgpool_mul_shift(49)
    assert (m, s) == (1337, 16)           # 65536/49 = 1337.47
    got = L.avgpool_requant(x, m, s)
    for n in range(3):
        for c in range(9):
            tot = int(x[n, :, :, c].astype(np.int64).sum())
            assert int(got[n, 0, 0, c]) == min(255, P.round_half_up(Fraction(tot * m, 1 << s)))
            assert abs(int(got[n, 0, 0, c]) - tot / 49.0) <= 1.0


# ---------------------------------------------------------------- stand-alone add: both operands, zero points
# Hand-computed rows (Sections 3.4.2, 4.1: both operands rescaled, then the convolution's tail).
#   a' = [(A - a_zero) * mul_a / 2^sh_a],  b' = [(B - b_zero) * mul_b / 2^sh_b],  Y = a' + b',
#   Y = clamp(Y, 0, h_i) if brelu,  V = [Y * mul / 2^shift],  out = clamp(V + out_zero, lo, hi)
# (A, a_zero, mul_a, sh_a, B, b_zero, mul_b, sh_b, brelu, h_i, mul, shift, out_zero, lo, hi) -> out
ADD_ROWS = [
    # the second operand does all the work: 7*3/2 = 10.5 -> 11
    ((0, 0, 1, 0, 7, 0, 3, 1, 0, 0, 1, 0, 0, -128, 127), 11),
    # negative tie of the second operand: -7*3/2 = -10.5 -> -10 (ties go up)
    ((0, 0, 1, 0, -7, 0, 3, 1, 0, 0, 1, 0, 0, -128, 127), -10),
    # b_zero: (5 - 12) * 3 / 2 = -10.5 -> -10; a: (9 - 1) * 5 / 4 = 10 -> Y = 0
    ((9, 1, 5, 2, 5, 12, 3, 1, 0, 0, 1, 0, 0, -128, 127), 0),
    # a distinct shift for each operand: a' = [10*7/8] = [8.75] = 9, b' = [100*500/2^10] = [48.83] = 49; Y = 58
    ((10, 0, 7, 3, 100, 0, 500, 10, 0, 0, 1, 0, 0, -128, 127), 58),
    # ... then Eq. 4 with a tie: 58 * 3 / 4 = 43.5 -> 44, and a zero point of -40 -> 4
    ((10, 0, 7, 3, 100, 0, 500, 10, 0, 0, 3, 2, -40, -128, 127), 4),
    # negative Y with a tie in Eq. 4 and a positive zero point: a' = -9 (=[-8.75]), b' = [-48.83] = -49,
    # Y = -58, V = [-43.5] = -43, out = -43 + 128 = 85
    ((-10, 0, 7, 3, -100, 0, 500, 10, 0, 0, 3, 2, 128, 0, 255), 85),
    # the same through BReLU: Y = -58 clamps to 0, V = 0, out = 128
    ((-10, 0, 7, 3, -100, 0, 500, 10, 1, 1000, 3, 2, 128, 0, 255), 128),
    # BReLU's upper bound acts on Y before Eq. 4: Y = 58 -> h_i = 50 -> [50*3/4] = [37.5] = 38, +out_zero 10 = 48
    ((10, 0, 7, 3, 100, 0, 500, 10, 1, 50, 3, 2, 10, 0, 255), 48),
    # saturation after the zero point: V = 44, out_zero = 250 -> 294 -> 255
    ((10, 0, 7, 3, 100, 0, 500, 10, 0, 0, 3, 2, 250, 0, 255), 255),
    # and at the lower end: V = -43, out_zero = 20 -> -23 -> lo = -5
    ((-10, 0, 7, 3, -100, 0, 500, 10, 0, 0, 3, 2, 20, -5, 127), -5),
    # operands swapped in role (a carries mul 500 / shift 10, b carries 7 / 3) give the same sum
    ((100, 0, 500, 10, 10, 0, 7, 3, 0, 0, 1, 0, 0, -128, 127), 58),
]


def _add_one(row):
    (A, az, ma, sa, Bv, bz, mb, sb, brelu, h_i, mul, shift, oz, lo, hi) = row
    out_dtype = L.S8 if lo < 0 else L.U8
    out, ovf = L.add_requant(np.array([A], np.int32), np.array([Bv], np.int32), a_dtype=L.I32, b_dtype=L.I32,
                             out_dtype=out_dtype, a_zero=az, b_zero=bz, mul_a=ma, sh_a=sa, mul_b=mb, sh_b=sb,
                             brelu=brelu, h_i=h_i, mul=mul, shift=shift, out_zero=oz, out_lo=lo, out_hi=hi)
    assert not ovf
    return int(out[0])


@pytest.mark.parametrize("row,want", ADD_ROWS)
def test_add_requant_hand_computed_rows(row, want):
    assert _add_one(row) == want


def test_add_requant_both_operands_against_exact_rationals():
    """Every field of the descriptor varies (second operand's multiplier, shift and zero included);
    the expected value is the definition in exact rationals, element by element."""
    rng = np.random.default_rng(21)
    for trial in range(40):
        a_dtype = [L.U8, L.S8, L.I32][trial % 3]
        b_dtype = [L.I32, L.U8, L.S8][(trial // 3) % 3]
        n = 64
        draw = {L.U8: lambda: rng.integers(0, 256, n).astype(np.uint8), L.S8: lambda: rng.integers(-128, 128, n).astype(np.int8),
                L.I32: lambda: rng.integers(-300000, 300000, n).astype(np.int32)}
        A, Bv = draw[a_dtype](), draw[b_dtype]()
        az, bz = int(rng.integers(-3, 130)), int(rng.integers(-3, 130))
        ma, mb = int(rng.integers(1, 2000)), int(rng.integers(1, 2000))
        sa, sb = int(rng.integers(0, 12)), int(rng.integers(0, 12))
        brelu = trial % 2
        h_i = int(rng.integers(1, 400000))
        mul, shift = int(rng.integers(1, 300)), int(rng.integers(0, 20))
        oz = int(rng.integers(-100, 200))
        signed = trial % 4 == 3
        lo, hi = (-128 + int(rng.integers(0, 10)), 127 - int(rng.integers(0, 10))) if signed else (int(rng.integers(0, 10)), 255 - int(rng.integers(0, 10)))
        out, ovf = L.add_requant(A, Bv, a_dtype=a_dtype, b_dtype=b_dtype, out_dtype=L.S8 if signed else L.U8, a_zero=az, b_zero=bz,
                                 mul_a=ma, sh_a=sa, mul_b=mb, sh_b=sb, brelu=brelu, h_i=h_i, mul=mul, shift=shift,
                                 out_zero=oz, out_lo=lo, out_hi=hi)
        assert not ovf
        for i in range(n):
            y = P.round_half_up(Fraction((int(A[i]) - az) * ma, 1 << sa)) + P.round_half_up(Fraction((int(Bv[i]) - bz) * mb, 1 << sb))
            if brelu:
                y = min(max(y, 0), h_i)
            v = P.round_half_up(Fraction(y * mul, 1 << shift)) + oz
            assert int(out[i]) == min(max(v, lo), hi), (trial, i)


def test_add_requant_operands_are_not_interchangeable_by_accident():
    """A slip that uses one operand's shift, multiplier or zero for the other changes these sums."""
    base = dict(a_dtype=L.I32, b_dtype=L.I32, out_dtype=L.S8, brelu=False, mul=1, shift=0, out_lo=-128, out_hi=127)
    A, Bv = np.array([40], np.int32), np.array([24], np.int32)
    # a' = [40 * 3 / 2^3] = 15, b' = [24 * 5 / 2^1] = 60
    assert int(L.add_requant(A, Bv, mul_a=3, sh_a=3, mul_b=5, sh_b=1, **base)[0][0]) == 75
    # with the shifts exchanged it would be 60 + 15 = 75 as well, so break the symmetry: zeros
    # a' = [(40-8) * 3 / 8] = 12, b' = [(24-4) * 5 / 2] = 50
    assert int(L.add_requant(A, Bv, a_zero=8, b_zero=4, mul_a=3, sh_a=3, mul_b=5, sh_b=1, **base)[0][0]) == 62
    # b_zero dropped would give 12 + 60 = 72; a_zero used for b would give 12 + 40 = 52; sh_a for b: 12 + [20*5/8] = 12 + 13 = 25


def test_conv_out_zero_exact():
    """Zero point and saturation of a convolution output (the regression networks' last layer)
    against hand-computed values: one pixel, one channel, K = 2."""
    X = np.array([[[[10, 200]]]], dtype=np.uint8)
    W = np.array([[[[3, -1]]]], dtype=np.int8)
    # U = 30 - 200 = -170, Y = U + 50 = -120, no BReLU, V = [-120 * 3 / 8] = [-45] = -45
    for oz, lo, hi, want in ((128, 0, 255, 83), (0, 0, 255, 0), (300, 0, 255, 255), (45, 0, 255, 0), (46, 0, 255, 1), (40, 7, 255, 7)):
        out, ovf = L.conv(X, W, [50], [3], [3], [0], brelu=False, out_zero=oz, out_lo=lo, out_hi=hi)
        assert not ovf and int(out[0, 0, 0, 0]) == want, (oz, lo, hi)
    # a tie below zero: Y = -121 -> -363/8 = -45.375 -> -45; Y = -124 -> -46.5 -> -46 (ties go up)
    out, _ = L.conv(X, W, [46], [3], [3], [0], brelu=False, out_zero=128, out_lo=0, out_hi=255)
    assert int(out[0, 0, 0, 0]) == 128 - 46
    # RAW128 input: x = raw - 128 = (-118, 72): U = -354 - 72 = -426, Y = -426 + 426 = 0 -> out_zero
    out, _ = L.conv(X, W, [426], [3], [3], [0], brelu=False, in_dtype=L.U8_RAW128, out_zero=128, out_lo=0, out_hi=255)
    assert int(out[0, 0, 0, 0]) == 128


# ---------------------------------------------------------------- Eq. 8: the bracket of the exact product
def test_eq8_bracket_is_taken_of_the_exact_product():
    """Pairs (h_rf, ratio_Y) whose product, rounded to a double, lands exactly on k + 0.5 while the
    exact product lies just beside it: the bracket follows the exact product."""
    below = above = 0
    for k in range(1000, 1400):
        b = (k + 0.5) / 3.0
        if 3.0 * b != k + 0.5:
            continue
        exact = Fraction(3) * Fraction(b)
        if exact == Fraction(2 * k + 1, 2):
            continue
        want = k + 1 if exact > Fraction(2 * k + 1, 2) else k
        assert P.brelu_params(3.0, b, 255)["h_ri"] == want
        below += want == k
        above += want == k + 1
    assert below > 5 and above > 5
