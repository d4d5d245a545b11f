"""GPU parity of the n-sigma bound (Section 3.2.2) against the oracle's sort-and-pick definition:
the radix select must return the same integer for every input, duplicates, negatives and
extremes included."""
import numpy as np
import pytest
import torch

from oracle import planner as P
from paper_2006_11735_b200 import binding as B

pytestmark = pytest.mark.gpu


def _bound(Y, frac, offset=0):
    """Runs the library on a device copy of Y placed `offset` elements into its buffer."""
    buf = torch.empty(Y.size + offset + 3, dtype=torch.int32, device="cuda")
    buf[offset:offset + Y.size] = torch.from_numpy(Y.reshape(-1)).cuda()
    got = B.iq_sigma_bound(buf.data_ptr() + 4 * offset, Y.size, frac, torch.cuda.current_stream().cuda_stream)
    B.iconv_check(torch.cuda.current_stream().cuda_stream)
    return got


@pytest.mark.parametrize("size", [1, 2, 7, 1000, 4099, 1 << 20, 20_000_003])
@pytest.mark.parametrize("frac", [0.0015, 0.00023, 0.5, 1.0])
def test_sigma_bound_matches_oracle_on_normal_feature_maps(size, frac):
    rng = np.random.default_rng(size % 9973 + int(frac * 1e6))
    Y = np.floor(rng.normal(-2000.0, 90000.0, size=size) + 0.5).astype(np.int32)
    want = P.sigma_bound(Y, frac)
    for offset in (0, 1, 3):                     # the 16-byte fast path starts at every alignment
        assert _bound(Y, frac, offset) == want


def test_sigma_bound_degenerate_inputs():
    cases = [
        np.full(100_000, 77, dtype=np.int32),                                          # every value equal
        np.full(5000, -5, dtype=np.int32),                                             # all negative: clamped to 1
        np.array([np.iinfo(np.int32).min, np.iinfo(np.int32).max, 0, -1, 1] * 2000, dtype=np.int32),
        np.repeat(np.arange(-50, 50, dtype=np.int32), 3000),                           # heavy duplicates
        (np.arange(300_000, dtype=np.int64) * 7919 % 1_000_003 - 500_000).astype(np.int32),   # all distinct
        np.random.default_rng(3).integers(-2 ** 31, 2 ** 31, size=700_001, dtype=np.int64).astype(np.int32),   # full range
    ]
    for Y in cases:
        for frac in (0.0015, 0.01, 0.999):
            assert _bound(Y, frac) == P.sigma_bound(Y, frac)
    assert B.iq_sigma_bound(None, 0) == 1
    with pytest.raises(B.IconvError):
        B.iq_sigma_bound(torch.zeros(4, dtype=torch.int32, device="cuda").data_ptr() + 1, 2)    # misaligned


def test_sigma_bound_calibrates_a_layer_like_the_oracle():
    """The bound of a raw convolution output computed on the GPU feeds Eq. 9-13 to the same
    mul, shift and h_i as the oracle's calibration of that layer."""
    from gpu_util import gpu_conv, oracle_conv
    rng = np.random.default_rng(17)
    X = rng.integers(0, 256, size=(2, 40, 44, 64), dtype=np.uint8)
    W = np.clip(np.floor(rng.normal(0, 40, size=(64, 3, 3, 64)) + 0.5), -127, 127).astype(np.int8)
    b = rng.integers(-4096, 4097, size=(64,), dtype=np.int32)
    Yo = oracle_conv(X, W, b, [1], [0], [0], pad=1, out_dtype=B.I32, brelu=False)
    Yg, _ = gpu_conv(X, W, b, [1], [0], [0], pad=1, out_dtype=B.I32, brelu=False)
    assert np.array_equal(Yg, Yo)
    h_ri = _bound(Yg.astype(np.int32), 0.0015)
    assert h_ri == P.sigma_bound(Yo)
    assert B.iq_brelu_params(float(h_ri), 1.0, 255) == {k: v for k, v in P.brelu_params(float(h_ri), 1.0, 255).items()}


def test_batch_norm_folded_per_channel_layer_end_to_end():
    """A float convolution + batch normalisation + ReLU-like clamp becomes an integer layer with
    one quantisation step per output channel (Section 3.4.3) and per-channel mul / shift / h_i
    from Algorithm 2 with every channel a branch; the GPU equals the oracle bit for bit and the
    dequantised result tracks the float layer."""
    from gpu_util import gpu_conv, oracle_conv
    rng = np.random.default_rng(33)
    n, h, w, c_in, c_out, k, max_int, h_rf = 2, 20, 24, 32, 48, 3, 255, 4.0
    x_f = rng.uniform(0.0, 1.0, size=(n, h, w, c_in))
    ratio_X = 255.0
    X = np.floor(x_f * ratio_X + 0.5).astype(np.uint8)
    W_f = rng.normal(0, 0.08, size=(c_out, k, k, c_in)).astype(np.float32)
    gamma = rng.uniform(0.05, 3.0, size=c_out).astype(np.float32)          # steps differing 60-fold between channels
    beta = rng.normal(0, 0.2, size=c_out).astype(np.float32)
    mean = rng.normal(0, 0.3, size=c_out).astype(np.float32)
    var = rng.uniform(0.2, 2.0, size=c_out).astype(np.float32)
    Wp, bp, delta = B.iq_bn_fold(W_f, None, gamma, beta, mean, var, 1e-5)
    assert delta.max() / delta.min() > 10
    ratio_Y = [ratio_X / d for d in delta]
    ratio_V = [P.brelu_params(h_rf, ry, max_int)["ratio_V"] for ry in ratio_Y]
    sync = P.concat_sync(ratio_Y, ratio_V)                                   # Algorithm 2, one branch per channel
    got_plan = B.iconcat_plan(ratio_Y, ratio_V)
    assert list(got_plan["mul"]) == list(sync["mul"]) and list(got_plan["shift"]) == list(sync["shift"])
    Wq = np.stack([P.quantize_weights(Wp[c], delta[c] * sync["delta_scale"][c]) for c in range(c_out)])
    b_i = np.array([P.round_half_up(bp[c] * sync["ratio_Y_new"][c]) for c in range(c_out)], dtype=np.int32)
    mul = np.array(sync["mul"], dtype=np.int32)
    shift = np.array(sync["shift"], dtype=np.int32)
    h_i = np.array([P.round_half_up(P.Fraction(max_int * (1 << int(s)), int(m))) for m, s in zip(mul, shift)], dtype=np.int32)
    want = oracle_conv(X, Wq, b_i, mul, shift, h_i, pad=1)
    for kernel in (B.KERNEL_AUTO, B.KERNEL_UMMA_IM2COL, B.KERNEL_DIRECT):
        got, _ = gpu_conv(X, Wq, b_i, mul, shift, h_i, pad=1, kernel=kernel)
        assert np.array_equal(got, want)
    # the float layer: convolution, batch normalisation, clamp to [0, h_f]
    xp = np.pad(x_f, ((0, 0), (1, 1), (1, 1), (0, 0)))
    y = np.zeros((n, h, w, c_out))
    for r in range(k):
        for s in range(k):
            y += xp[:, r:r + h, s:s + w, :] @ W_f[:, r, s, :].astype(np.float64).T
    y = (y - mean) / np.sqrt(var.astype(np.float64) + 1e-5) * gamma + beta
    h_f = max_int / sync["ratio_V_min"]
    y = np.clip(y, 0.0, h_f)
    err = np.abs(want.astype(np.float64) / sync["ratio_V_min"] - y)
    assert err.mean() < 0.02 * h_f and (want > 0).mean() > 0.2 and (want == max_int).mean() < 0.5
