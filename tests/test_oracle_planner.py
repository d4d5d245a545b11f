"""Pins of the oracle's parameter arithmetic (Eq. 1-2, Eq. 7-13, Algorithm 2, residual
ratio synchronisation) and of whole small networks: a float "shadow" network built from
the de-quantised parameters must track the integer network, which fails if a ratio is
applied in the wrong direction, a skip is rescaled with the wrong factor or concatenated
branches end up on different scales."""
from fractions import Fraction

import numpy as np
import pytest
from scipy import signal

from oracle import layers as L
from oracle import networks as ON
from oracle import planner as P
from workloads import generators as gen
from workloads import networks as N
from workloads.networks import AvgPool, Conv, MaxPool


def test_weight_quantisation_eq_1_2():
    W_f = np.array([0.5, -1.27, 0.004, 0.006, -0.015, 1.0], dtype=np.float32)
    delta = P.weight_delta(W_f)
    assert delta == pytest.approx(0.01, rel=1e-6)         # max|W| = 1.27 -> step 0.01
    assert P.quantize_weights(W_f, delta).tolist() == [50, -127, 0, 1, -1, 100]   # -1.5 rounds toward +inf
    # a smaller (adjusted) step clips at +-127
    assert P.quantize_weights(W_f, delta / 2).tolist() == [100, -127, 1, 1, -3, 127]


def test_mul_shift_reading():
    # config-1 style: ratio 255/146992 reaches mul >= 2^6 at shift 16
    assert P.mul_shift(Fraction(255, 146992)) == (114, 16)
    assert P.mul_shift(Fraction(255, 300000)) == (111, 17)      # 55.7 at 16 is below 2^6 -> shift 17
    assert P.mul_shift(1.0) == (65536, 16)
    assert P.mul_shift(400.25, shift_min=8) == (102464, 8)
    with pytest.raises(ValueError):
        P.mul_shift(1e9, shift_min=16)                          # mul would not fit int32
    with pytest.raises(ValueError):
        P.mul_shift(0.0)
    rng = np.random.default_rng(1)
    for _ in range(300):
        r = float(np.exp(rng.uniform(np.log(1e-7), np.log(1e3))))
        mul, shift = P.mul_shift(r)
        assert 16 <= shift <= 40 and 64 <= mul < 2 ** 31
        assert abs(mul / 2 ** shift - r) <= 0.5 / 2 ** shift + 1e-18
        if shift > 16:                                          # smallest shift that reaches 2^6
            assert P.round_half_up(Fraction(r) * (1 << (shift - 1))) < 64


def test_quantised_brelu_section_3_3_worked_instance():
    # ratio_Y = 24498.7, h_rf = 6.0: h_ri = [146992.2] = 146992, mul = [255*65536/146992] = 114
    q = P.brelu_params(6.0, 24498.7, 255)
    assert (q["h_ri"], q["mul"], q["shift"]) == (146992, 114, 16)
    # Eq. 10 itself fails for h_ri (146992*114/65536 = 255.69 -> 256): the reason for Eq. 11-13
    assert P.requant_exact(q["h_ri"], q["mul"], q["shift"]) == 256
    assert q["h_i"] == 146594                                   # [255*65536/114] = [146593.68]
    assert P.requant_exact(q["h_i"], q["mul"], q["shift"]) == 255
    assert q["ratio_V"] == pytest.approx(24498.7 * 114 / 65536)
    assert q["h_f"] == pytest.approx(255 / q["ratio_V"])
    assert q["h_i"] == P.round_half_up(q["h_f"] * 24498.7)      # Eq. 13 verbatim agrees


def test_h_i_always_requantises_to_max_int():
    rng = np.random.default_rng(2)
    for max_int in (255, 127, 63, 31, 15):
        for _ in range(200):
            h_ri = int(np.exp(rng.uniform(np.log(1), np.log(2e8))))
            q = P.brelu_params_from_h_ri(h_ri, 1234.5, max_int)
            assert P.requant_exact(q["h_i"], q["mul"], q["shift"]) == max_int
            assert q["mul"] >= 64
            assert q["h_i"] * q["mul"] + (1 << (q["shift"] - 1)) < 2 ** 63


def test_sigma_bound_is_the_kth_largest_value():
    """Section 3.2.2: the bound is characterised without sorting: at least k values reach it,
    fewer than k exceed it (k = the size of the largest 0.15 %), and it is never below 1."""
    rng = np.random.default_rng(11)
    for size, frac in [(1, 0.0015), (7, 0.0015), (1000, 0.0015), (4001, 0.0015), (50000, 0.00023), (300, 0.5), (64, 1.0)]:
        for scale in (3.0, 40000.0):
            Y = np.floor(rng.normal(0, scale, size=size) + 0.5).astype(np.int32)
            b = P.sigma_bound(Y, frac)
            k = max(1, int(np.ceil(size * frac)))
            exact = sorted(Y.tolist(), reverse=True)[k - 1]
            assert b == max(1, exact)
            if exact >= 1:
                assert (Y >= b).sum() >= k and (Y > b).sum() < k
    assert P.sigma_bound(np.array([5, 5, 5, 5], dtype=np.int32), 0.5) == 5
    assert P.sigma_bound(np.array([-9, -3], dtype=np.int32)) == 1
    assert P.sigma_bound(np.zeros(0, dtype=np.int32)) == 1
    # three sigma of a wide normal sample sits near 2.97 standard deviations (the 99.85th percentile)
    Y = np.floor(np.random.default_rng(5).normal(0, 10000.0, size=2_000_000) + 0.5).astype(np.int32)
    assert 2.9 * 10000 < P.sigma_bound(Y) < 3.05 * 10000
    # and it is the rule the calibration of the networks uses
    from oracle import networks as ON
    assert ON._three_sigma_bound(Y) == P.sigma_bound(Y, 0.0015)


def test_bn_fold_equals_batch_norm_after_the_convolution():
    """Section 3.4.3: the merged layer computes what convolution followed by batch normalisation
    computes (checked on data, in float64, against the two operations written apart), and each
    channel's step maps that channel's largest merged weight to 127."""
    rng = np.random.default_rng(21)
    c_out, k, c_in, eps = 6, 3, 4, 1e-5
    W = rng.normal(0, 0.1, size=(c_out, k, k, c_in))
    b = rng.normal(0, 0.05, size=c_out)
    gamma, beta = rng.uniform(0.2, 2.0, size=c_out), rng.normal(0, 0.3, size=c_out)
    mean, var = rng.normal(0, 0.2, size=c_out), rng.uniform(0.05, 3.0, size=c_out)
    gamma[2] = 0.0                                            # a dead channel
    x = rng.normal(0, 1.0, size=(5, k * k * c_in))            # five receptive fields
    conv = x @ W.reshape(c_out, -1).T + b
    want = (conv - mean) / np.sqrt(var + eps) * gamma + beta  # batch normalisation, inference form
    Wp, bp, delta = P.bn_fold(W, b, gamma, beta, mean, var, eps)
    assert np.allclose(x @ Wp.reshape(c_out, -1).T + bp, want, rtol=1e-12, atol=1e-12)
    assert np.allclose(delta, np.abs(Wp.reshape(c_out, -1)).max(axis=1) / 127.0, rtol=0, atol=0)
    assert delta[2] == 0.0 and np.all(Wp[2] == 0) and bp[2] == beta[2]
    for co in (0, 1, 3, 4, 5):
        assert np.abs(P.quantize_weights(Wp[co], delta[co])).max() == 127
    # no bias: the mean still shifts
    Wp2, bp2, _ = P.bn_fold(W, None, gamma, beta, mean, var, eps)
    assert np.array_equal(Wp2, Wp) and np.allclose(bp2, -mean * gamma / np.sqrt(var + eps) + beta)


def test_concat_sync_algorithm_2():
    ry, rv = [30000.0, 52000.0, 41000.0], [90.0, 61.5, 75.25]
    s = P.concat_sync(ry, rv)
    assert s["ratio_V_min"] == 61.5                             # the minimal ratio is the reference
    for i in range(3):
        m, sh = s["mul"][i], s["shift"][i]
        assert abs(m / 2 ** sh - 61.5 / ry[i]) <= 0.5 / 2 ** sh
        # new ratio_Y is defined by (mul, shift): ratio_Y_new * mul / 2^shift == ratio_min
        assert s["ratio_Y_new"][i] * m / 2 ** sh == pytest.approx(61.5, rel=1e-14)
        # the factor on delta equals ratio_Y_old / ratio_Y_new and stays within mul's resolution
        assert s["delta_scale"][i] == pytest.approx(ry[i] / s["ratio_Y_new"][i], rel=1e-14)
        assert abs(s["delta_scale"][i] - 1) <= 0.5 / m + 1e-12
    exact = {Fraction(Fraction(61.5) * (1 << s["shift"][i]), s["mul"][i]) * s["mul"][i] / (1 << s["shift"][i])
             for i in range(3)}
    assert exact == {Fraction(61.5)}                            # one common ratio, exactly


def test_skip_sync_section_4_1():
    s = P.skip_sync(ratio_Y=98765.4, ratio_S=42.5)
    assert (s["skip_mul"], s["skip_shift"]) == P.mul_shift(98765.4 / 42.5, 8)
    assert s["ratio_Y_new"] == pytest.approx(42.5 * s["skip_mul"] / 2 ** s["skip_shift"], rel=1e-15)
    assert s["delta_scale"] == pytest.approx(98765.4 / s["ratio_Y_new"], rel=1e-15)
    assert abs(s["delta_scale"] - 1) < 1e-5


# ---------------------------------------------------------------- whole networks
def _float_shadow(net, params, x):
    """The float network the integer one stands for: X_f = X_i / ratio, W_d = W_i * delta."""
    T = {net.input: (x.astype(np.float64) - 128.0) / net.input_ratio if net.input_kind == "smooth"
         else x.astype(np.float64) / net.input_ratio}
    for op in net.ops:
        if isinstance(op, MaxPool):
            xs = T[op.src]
            n, h, w, c = xs.shape
            ho, wo = L.out_hw(h, w, op.k, op.k, op.stride, op.pad)
            xp = np.full((n, h + 2 * op.pad, w + 2 * op.pad, c), -np.inf)
            xp[:, op.pad:op.pad + h, op.pad:op.pad + w] = xs
            out = np.full((n, ho, wo, c), -np.inf)
            for r in range(op.k):
                for s in range(op.k):
                    out = np.maximum(out, xp[:, r:r + ho * op.stride:op.stride, s:s + wo * op.stride:op.stride])
            T[op.dst] = out
        elif isinstance(op, AvgPool):
            T[op.dst] = T[op.src].mean(axis=(1, 2), keepdims=True)
        else:
            p = params[op.name]
            W, b = ON.layer_weights(net, op, p["delta"])
            xs = T[op.src][..., op.in_c_offset:op.in_c_offset + op.c_in]
            n, h, w, c = xs.shape
            xp = np.zeros((n, h + 2 * op.pad, w + 2 * op.pad, c))
            xp[:, op.pad:op.pad + h, op.pad:op.pad + w] = xs
            Wd = W.astype(np.float64) * p["delta"]
            ho, wo = L.out_hw(h, w, op.k, op.k, op.stride, op.pad)
            y = np.zeros((n, ho, wo, op.c_out))
            for r in range(op.k):
                for s in range(op.k):
                    y += xp[:, r:r + ho * op.stride:op.stride, s:s + wo * op.stride:op.stride] @ Wd[:, r, s, :].T
            y += b / p["ratio_Y"]
            if op.skip:
                y += T[op.skip]
            if op.role == "act":
                y = np.clip(y, 0.0, p["h_i"][0] / p["ratio_Y"])
            if op.dst not in T:
                t = net.tensors[op.dst]
                T[op.dst] = np.zeros((n, t.h, t.w, t.c))
            T[op.dst][..., op.out_c_offset:op.out_c_offset + op.c_out] = y
    return T


def _ratio_of(net, params, name):
    for op in net.ops:
        if op.dst == name and isinstance(op, Conv):
            return params[op.name]["ratio_Y"] if op.role == "raw" else params[op.name]["ratio_V"]
    raise KeyError(name)


@pytest.mark.parametrize("net", [
    N.single_conv(),
    N.vdsr(n=2, h=24, w=20, depth=6),
    N.vrcnn(n=2, h=24, w=28),
    N.resnet(2, (2, 1), h=48, w=40, widths=(16, 32), classes=10, seed=4),
    N.resnet_basic(2, (2, 1), h=48, w=40, widths=(16, 32), classes=10, seed=6),
], ids=lambda n: n.name)
def test_integer_network_tracks_its_float_shadow_and_is_not_vacuous(net):
    params = ON.calibrate(net)
    x = ON.net_input(net)
    T = ON.forward(net, params, x)
    F = _float_shadow(net, params, x)
    for op in net.ops:
        if not isinstance(op, Conv):
            continue
        p = params[op.name]
        t = T[op.dst][..., op.out_c_offset:op.out_c_offset + op.c_out].astype(np.float64)
        f = F[op.dst][..., op.out_c_offset:op.out_c_offset + op.c_out]
        if op.role == "act":
            zeros, sat = (t == 0).mean(), (t == net.max_int).mean()
            assert 0.05 <= zeros <= 0.95 and sat < 0.5, (op.name, zeros, sat)      # vacuity guard
            assert t.min() >= 0 and t.max() <= net.max_int
            deq = t / p["ratio_V"]
        elif op.role == "raw":
            deq = t / p["ratio_Y"]
        else:                                                    # regression: back in pixel units
            deq = (t - 128.0) / p["ratio_V"]
            assert p["ratio_V"] == pytest.approx(net.input_ratio, rel=0.01)
        err = np.sqrt(np.mean((deq - f) ** 2)) / (np.sqrt(np.mean(f ** 2)) + 1e-30)
        assert err < 0.08, (op.name, err)


def test_concat_branches_share_one_ratio_and_residual_operands_match():
    net = N.vrcnn(n=1, h=20, w=20)
    p = ON.calibrate(net)
    assert p["conv2a"]["ratio_V"] == p["conv2b"]["ratio_V"]
    assert p["conv3a"]["ratio_V"] == p["conv3b"]["ratio_V"]
    for a in ("conv2a", "conv2b", "conv3a", "conv3b"):
        q = p[a]
        assert Fraction(q["ratio_Y"]) * q["mul"][0] / (1 << q["shift"][0]) == pytest.approx(q["ratio_V"], rel=1e-14)
        assert P.requant_exact(q["h_i"][0], q["mul"][0], q["shift"][0]) == 255
        assert q["ratio_Y"] == pytest.approx(q["ratio_X"] / q["delta"], rel=1e-12)   # delta realises the ratio
    r = N.resnet(1, (2,), h=32, w=32, widths=(16,), classes=4)
    pr = ON.calibrate(r)
    ident = pr["s1b1_1x1b"]
    assert ident["ratio_Y"] == pytest.approx(pr["s1b0_1x1b"]["ratio_V"] * ident["skip_mul"] / 2 ** ident["skip_shift"], rel=1e-14)
    proj = pr["s1b0_1x1b"]
    assert proj["ratio_Y"] == pytest.approx(pr["s1b0_proj"]["ratio_Y"] * proj["skip_mul"] / 2 ** proj["skip_shift"], rel=1e-14)
    assert proj["ratio_Y"] == pytest.approx(proj["ratio_X"] / proj["delta"], rel=1e-12)


def test_generators_are_seeded_and_image_addressable():
    a = gen.image_batch(4, 3, 16, 12, 3)
    b = gen.image_batch(4, 1, 16, 12, 3, first=2)
    assert np.array_equal(a[2:3], b)
    assert a.std() > 10 and a.min() >= 0
    assert not np.array_equal(gen.weights_f(4, 0, 4, 3, 3, 2), gen.weights_f(4, 1, 4, 3, 3, 2))
    assert np.abs(gen.bias_i32(1, 0, 1000)).max() <= 4096
