"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header
declares, validates descriptors without touching a GPU, and its host-side parameter
arithmetic agrees with the oracle's planner."""
import os
import re

import numpy as np
import pytest

from oracle import planner as P
from paper_2006_11735_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "iconv.h")).read()
    return sorted(set(re.findall(r"^ICONV_API\s+(?:const\s+)?\w+\s*\*?\s*(\w+)\s*\(", text, flags=re.M)))


def test_library_exports_every_declared_symbol():
    names = _declared()
    assert len(names) >= 15
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert hasattr(B.lib, n), n


def _desc_kw(**over):
    kw = dict(n=1, h=8, w=8, c_in=16, c_out=16, kh=3, kw=3, stride=1, pad=1,
              weights=np.ones((16, 3, 3, 16), np.int8), bias=np.zeros(16, np.int32),
              mul=[200], shift=[16], h_i=[80000])
    kw.update(over)
    return kw


@pytest.mark.parametrize("over,status", [
    (dict(h=0), B.ERR_ARG),
    (dict(stride=0), B.ERR_ARG),
    (dict(in_dtype=B.I32), B.ERR_ARG),
    (dict(out_dtype=B.U8_RAW128), B.ERR_ARG),
    (dict(kernel=9), B.ERR_ARG),
    (dict(h=2, w=2, kh=5, kw=5, pad=1, weights=np.ones((16, 5, 5, 16), np.int8)), B.ERR_SHAPE),
    (dict(in_c_total=16, in_c_offset=8), B.ERR_SHAPE),
    (dict(out_c_total=24, out_c_offset=16), B.ERR_SHAPE),
    (dict(skip_dtype=B.U8, skip_c_total=8), B.ERR_SHAPE),
    (dict(mul=[0]), B.ERR_ARG),
    (dict(shift=[41]), B.ERR_ARG),
    (dict(h_i=[-1]), B.ERR_ARG),
    (dict(out_hi=300), B.ERR_ARG),
    (dict(skip_dtype=B.U8, skip_c_total=16, skip_mul=0), B.ERR_ARG),
    (dict(c_in=70000, kh=1, kw=1, pad=0, weights=np.full((16, 1, 1, 70000), 127, np.int8)), B.ERR_OVERFLOW),
    (dict(bias=np.full(16, 2 ** 31 - 1, np.int64).astype(np.int32)), B.ERR_OVERFLOW),
])
def test_plan_rejects_bad_descriptors_before_touching_the_gpu(over, status):
    with pytest.raises(B.IconvError) as e:
        B.iconv_plan(**_desc_kw(**over))
    assert e.value.status == status
    assert B.iconv_last_error()


def test_null_arguments():
    assert B.lib.iconv_plan(None, None) == B.ERR_ARG
    assert B.lib.iconv_forward(None, None, None, None, None, None) == B.ERR_ARG
    assert B.lib.iconv_plan_destroy(None) == B.OK
    assert B.lib.iadd_requant(None, None, None, None, None) == B.ERR_ARG
    assert B.lib.ipool_max(None, None, 1, 8, 8, 15, 3, 2, 1, None) == B.ERR_ALIGN
    import ctypes
    b = ctypes.c_int32(-7)
    assert B.lib.iq_sigma_bound(None, 10, 0.0015, ctypes.byref(b), None) == B.ERR_ARG          # no tensor
    assert B.lib.iq_sigma_bound(None, 0, 0.0015, None, None) == B.ERR_ARG                      # no place for the result
    assert B.lib.iq_sigma_bound(None, 0, 0.0, ctypes.byref(b), None) == B.ERR_ARG              # fraction outside (0, 1]
    assert B.lib.iq_sigma_bound(None, 0, 1.5, ctypes.byref(b), None) == B.ERR_ARG
    assert B.lib.iq_sigma_bound(None, 0, 0.0015, ctypes.byref(b), None) == B.OK and b.value == 1   # an empty map: no GPU touched


def test_weight_quantisation_matches_oracle_planner():
    rng = np.random.default_rng(0)
    w = rng.normal(0, 0.05, size=20000).astype(np.float32)
    d = B.iq_weight_delta(w)
    assert d == P.weight_delta(w)
    for scale in (1.0, 0.9973, 1.0041, 0.5):
        assert np.array_equal(B.iq_quantize_weights(w, d * scale), P.quantize_weights(w, d * scale))


def test_mul_shift_and_brelu_params_match_oracle_planner():
    rng = np.random.default_rng(1)
    for _ in range(500):
        r = float(np.exp(rng.uniform(np.log(1e-8), np.log(3e4))))
        smin = int(rng.integers(0, 20))
        try:
            want = P.mul_shift(r, smin)
        except ValueError:
            with pytest.raises(B.IconvError):
                B.iq_mul_shift(r, smin)
            continue
        assert B.iq_mul_shift(r, smin) == want
    for _ in range(500):
        h_rf = float(np.exp(rng.uniform(np.log(1e-3), np.log(50))))
        ry = float(np.exp(rng.uniform(np.log(10), np.log(1e6))))
        for max_int in (255, 127, 15):
            got = B.iq_brelu_params(h_rf, ry, max_int)
            want = P.brelu_params(h_rf, ry, max_int)
            for k in ("h_ri", "mul", "shift", "h_i"):
                assert got[k] == want[k], (k, h_rf, ry)
            assert got["ratio_V"] == want["ratio_V"] and got["h_f"] == want["h_f"]


def test_brelu_params_bracket_follows_the_exact_product_like_the_oracle():
    """Eq. 8 where the double product of the two arguments lands exactly on a tie while their exact
    product does not: the library decides by the exact product (fused multiply-add residual), as
    the oracle's rationals do."""
    from fractions import Fraction
    seen = set()
    for k in range(1000, 1400):
        for a in (3.0, 7.0, 1.1):
            b = (k + 0.5) / a
            if a * b != k + 0.5 or Fraction(a) * Fraction(b) == Fraction(2 * k + 1, 2):
                continue
            want = P.brelu_params(a, b, 255)
            got = B.iq_brelu_params(a, b, 255)
            assert got["h_ri"] == want["h_ri"] and got["mul"] == want["mul"] and got["h_i"] == want["h_i"], (a, b)
            seen.add(want["h_ri"] - k)
    assert seen == {0, 1}


def test_no_tensor_core_device_table_entry_without_a_gpu_call():
    assert B.iconv_device_initialised(63) == -1 and B.iconv_device_initialised(-5) == -1 and B.iconv_device_initialised(1000) == -1


def test_bn_fold_matches_oracle_planner():
    rng = np.random.default_rng(4)
    c_out = 9
    W = rng.normal(0, 0.1, size=(c_out, 3, 3, 5)).astype(np.float32)
    b = rng.normal(0, 0.05, size=c_out).astype(np.float32)
    gamma, beta = rng.uniform(0.2, 2.0, size=c_out).astype(np.float32), rng.normal(0, 0.3, size=c_out).astype(np.float32)
    mean, var = rng.normal(0, 0.2, size=c_out).astype(np.float32), rng.uniform(0.05, 3.0, size=c_out).astype(np.float32)
    gamma[4] = 0.0
    for bias in (b, None):
        got = B.iq_bn_fold(W, bias, gamma, beta, mean, var, 1e-5)
        want = P.bn_fold(W, bias, gamma, beta, mean, var, 1e-5)
        for g, w in zip(got, want):
            assert np.array_equal(g, w)
    assert got[2][4] == 0.0
    import ctypes
    assert B.lib.iq_bn_fold(None, None, None, None, None, None, 1e-5, 1, 1, None, None, None) == B.ERR_ARG
    with pytest.raises(B.IconvError):
        B.iq_bn_fold(W, b, gamma, beta, mean, -var, 0.0)          # var + eps <= 0


def test_skip_sync_and_concat_plan_match_oracle_planner():
    rng = np.random.default_rng(2)
    for _ in range(200):
        ry = float(np.exp(rng.uniform(np.log(1e3), np.log(1e7))))
        rs = float(np.exp(rng.uniform(np.log(1), np.log(1e4))))
        assert B.iq_skip_sync(ry, rs) == P.skip_sync(ry, rs)
        k = int(rng.integers(1, 5))
        rys = np.exp(rng.uniform(np.log(1e3), np.log(1e6), size=k)).tolist()
        rvs = np.exp(rng.uniform(np.log(10), np.log(500), size=k)).tolist()
        assert B.iconcat_plan(rys, rvs) == P.concat_sync(rys, rvs)
