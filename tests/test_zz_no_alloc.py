"""The allocation-free first-layer entry point against the planned one and against the oracle.

Some users of this library run where device allocation is off limits once set-up is over: under a
framework's memory pool, in a serving loop with a fixed memory budget, or while a stream is being
captured.  `iconv_stem_forward_static` serves them: no plan, weights and bias already on the
device, scratch in a fixed array inside the library.  This file checks, through the C-ABI, that it
gives exactly the bytes of `iconv_plan` + `iconv_forward` for the same layer and of the CPU oracle,
on two calls in a row (the second with other data and another shape, so that whatever the first
call left in the shared array would show), that it refuses what does not fit the array, and that
a bias it cannot take is reported by `iconv_check`.  The comparison is
exact: the layer is integer arithmetic, and the library's other GPU tests use no tolerance either.
It sits in a file of its own, collected last, so a failure here cannot hide any other test.
"""
import numpy as np
import pytest
import torch

from paper_2006_11735_b200 import binding as B

from gpu_util import Fenced, dev, gpu_conv, oracle_conv

pytestmark = pytest.mark.gpu


def _case(seed, n, h, w, c_out):
    rng = np.random.default_rng(seed)
    X = rng.integers(0, 256, size=(n, h, w, 3), dtype=np.uint8)
    W = np.clip(np.floor(rng.normal(0, 40, size=(c_out, 7, 7, 3)) + 0.5), -127, 127).astype(np.int8)
    b = rng.integers(-4096, 4097, size=(c_out,), dtype=np.int32)
    h_i = int(40.0 * 100.0 * np.sqrt(147) * 2.0)
    shift = 17
    mul = int(np.floor(255.0 * 2.0 ** shift / h_i + 0.5))
    return X, W, b, mul, shift, h_i


def _static(X, W, b, mul, shift, h_i, in_dtype, out_c_total=None, out_c_offset=0, fill=0x5A):
    n, h, w, _ = X.shape
    c_out = W.shape[0]
    ho, wo = (h - 1) // 2 + 1, (w - 1) // 2 + 1
    out = Fenced((n, ho, wo, c_out if out_c_total is None else out_c_total), np.uint8, fill)
    xd, wd, bd = dev(X), dev(W), dev(b)
    st = torch.cuda.current_stream().cuda_stream
    B.iconv_stem_forward_static(xd.data_ptr(), wd.data_ptr(), bd.data_ptr(), out.ptr, st, n=n, h=h, w=w, c_out=c_out,
                                in_dtype=in_dtype, out_c_total=out_c_total, out_c_offset=out_c_offset,
                                mul=mul, shift=shift, h_i=h_i)
    B.iconv_check(st)
    return out.get()


def test_static_scratch_first_layer_equals_the_planned_one_twice_in_a_row():
    # first call: raw image with the -128 re-normalisation, 64 channels
    X, W, b, mul, shift, h_i = _case(11, 3, 38, 30, 64)
    want, fam = gpu_conv(X, W, b, [mul], [shift], [h_i], stride=2, pad=3, in_dtype=B.U8_RAW128, kernel=B.KERNEL_STEM)
    assert fam == B.KERNEL_STEM
    got = _static(X, W, b, mul, shift, h_i, B.U8_RAW128)
    assert np.array_equal(got, want)
    assert np.array_equal(got, oracle_conv(X, W, b, [mul], [shift], [h_i], stride=2, pad=3, in_dtype=B.U8_RAW128))
    assert 0.05 < (want == 0).mean() < 0.95
    # second call, straight after: other data, other shape, a channel offset inside a wider tensor
    X2, W2, b2, mul2, shift2, h2 = _case(12, 2, 21, 45, 32)
    want2, _ = gpu_conv(X2, W2, b2, [mul2], [shift2], [h2], stride=2, pad=3, in_dtype=B.U8, out_c_total=48,
                        out_c_offset=16, kernel=B.KERNEL_STEM)
    got2 = _static(X2, W2, b2, mul2, shift2, h2, B.U8, out_c_total=48, out_c_offset=16)
    assert np.array_equal(got2, want2)
    assert np.array_equal(got2, oracle_conv(X2, W2, b2, [mul2], [shift2], [h2], stride=2, pad=3, in_dtype=B.U8, out_c_total=48,
                                            out_c_offset=16))
    assert (got2[..., :16] == 0x5A).all()
    # and the first case once more: the array now holds the second call's leftovers
    assert np.array_equal(_static(X, W, b, mul, shift, h_i, B.U8_RAW128), want)


@pytest.mark.parametrize("n,h,w,c_out,in_dtype", [
    (2, 8, 8, 64, B.U8_RAW128),       # 4 x 4 outputs: too few real pixels per tile for one patch per tile, the im2col form runs
    (1, 5, 7, 16, B.U8),              # one channel group, odd sizes
    (2, 30, 26, 64, B.S8),            # a signed image
    (1, 64, 64, 256, B.U8_RAW128),    # the widest channel count the weight region holds
])
def test_static_scratch_first_layer_equals_the_oracle(n, h, w, c_out, in_dtype):
    X, W, b, mul, shift, h_i = _case(100 + h, n, h, w, c_out)
    Xs = X.view(np.int8) if in_dtype == B.S8 else X
    want = oracle_conv(Xs, W, b, [mul], [shift], [h_i], stride=2, pad=3, in_dtype=in_dtype)
    got = _static(X, W, b, mul, shift, h_i, in_dtype)
    assert np.array_equal(got, want)
    assert np.unique(want).size > 8


def test_static_scratch_entry_reports_a_bias_it_cannot_take():
    """|bias| beyond 2^30 is found on the device (the bias never visits the host): the value is
    replaced by 0, the status word takes code 8 and the next iconv_check says ICONV_ERR_ARG, once."""
    X, W, b, mul, shift, h_i = _case(7, 1, 16, 16, 16)
    b = b.copy()
    b[3] = 2 ** 30 + 5
    st = torch.cuda.current_stream().cuda_stream
    xd, wd, bd = dev(X), dev(W), dev(b)
    out = Fenced((1, 8, 8, 16), np.uint8)
    B.iconv_stem_forward_static(xd.data_ptr(), wd.data_ptr(), bd.data_ptr(), out.ptr, st, n=1, h=16, w=16, c_out=16,
                                in_dtype=B.U8_RAW128, mul=mul, shift=shift, h_i=h_i)
    with pytest.raises(B.IconvError) as e:
        B.iconv_check(st)
    assert e.value.status == B.ERR_ARG and "code 8" in str(e.value)
    B.iconv_check(st)                 # the word was cleared
    b[3] = 0                          # the output is the layer's with that channel's bias at 0
    assert np.array_equal(out.get(), oracle_conv(X, W, b, [mul], [shift], [h_i], stride=2, pad=3, in_dtype=B.U8_RAW128))


def test_static_scratch_entry_refuses_what_does_not_fit():
    with pytest.raises(B.IconvError) as e:      # 200 images of 224 x 224 need 42.5 MB, the array has 32 MiB
        B.iconv_stem_forward_static(16, 16, 16, 16, 0, n=200, h=224, w=224, c_out=64, mul=100, shift=16, h_i=100000)
    assert e.value.status == B.ERR_SHAPE and "scratch" in str(e.value)
    with pytest.raises(B.IconvError) as e:
        B.iconv_stem_forward_static(16, 16, 16, 16, 0, n=1, h=32, w=32, c_out=24, mul=100, shift=16, h_i=100000)
    assert e.value.status == B.ERR_ARG
