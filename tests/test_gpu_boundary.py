"""GPU tests of the boundary itself: caller-owned workspaces (two forwards of one plan in flight
at once), the bounded device-side waits seen to run out, and the per-device initialisation."""
import numpy as np
import pytest
import torch

from paper_2006_11735_b200 import binding as B

from gpu_util import Fenced, dev, oracle_conv

pytestmark = pytest.mark.gpu


def _stem_case(seed, n, h, w, c_in, c_out, k):
    rng = np.random.default_rng(seed)
    X = rng.integers(0, 256, size=(n, h, w, c_in), dtype=np.uint8)
    W = np.clip(np.floor(rng.normal(0, 40, size=(c_out, k, k, c_in)) + 0.5), -127, 127).astype(np.int8)
    b = rng.integers(-4096, 4097, size=(c_out,), dtype=np.int32)
    h_i = int(40.0 * 100.0 * np.sqrt(k * k * c_in) * 2.0)
    shift = 17
    mul = int(np.floor(255.0 * 2.0 ** shift / h_i + 0.5))
    return X, W, b, mul, shift, h_i


@pytest.mark.parametrize("shape", [
    dict(n=3, h=70, w=62, c_in=3, c_out=64, k=7, stride=2, pad=3),      # 3-channel 7x7/2 stem
    dict(n=2, h=96, w=80, c_in=1, c_out=64, k=3, stride=1, pad=1),      # single-channel first layer (rows repack)
    dict(n=2, h=64, w=72, c_in=1, c_out=64, k=5, stride=1, pad=2),
])
def test_two_forwards_of_one_plan_on_two_streams_with_two_workspaces(shape):
    """The plan owns no activation-sized memory: its repack scratch is the caller's workspace, so
    the same plan may run twice at once, each forward with its own workspace, input and output."""
    n, h, w, c_in, c_out, k, stride, pad = (shape[x] for x in ("n", "h", "w", "c_in", "c_out", "k", "stride", "pad"))
    Xa, W, b, mul, shift, h_i = _stem_case(31, n, h, w, c_in, c_out, k)
    Xb = np.random.default_rng(32).integers(0, 256, size=Xa.shape, dtype=np.uint8)
    plan = B.iconv_plan(n=n, h=h, w=w, c_in=c_in, c_out=c_out, kh=k, kw=k, stride=stride, pad=pad, in_dtype=B.U8_RAW128,
                        weights=W, bias=b, mul=[mul], shift=[shift], h_i=[h_i])
    try:
        assert B.iconv_plan_kernel(plan) == B.KERNEL_STEM
        size = B.iconv_workspace_bytes(plan)
        assert size >= n * (h // stride) * (w // stride) * 16
        ho, wo = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        xa, xb = dev(Xa), dev(Xb)
        oa, ob = Fenced((n, ho, wo, c_out), np.uint8), Fenced((n, ho, wo, c_out), np.uint8)
        wa, wb = Fenced((size,), np.uint8, 0xC3), Fenced((size,), np.uint8, 0x3C)
        torch.cuda.synchronize()
        for _ in range(3):                                   # several rounds so that the two streams really interleave
            B.iconv_forward(plan, xa.data_ptr(), None, oa.ptr, wa.ptr, s1.cuda_stream)
            B.iconv_forward(plan, xb.data_ptr(), None, ob.ptr, wb.ptr, s2.cuda_stream)
        B.iconv_check(s1.cuda_stream)
        B.iconv_check(s2.cuda_stream)
        wa.get(), wb.get()                                   # nothing was written outside either workspace
        kw = dict(stride=stride, pad=pad, in_dtype=B.U8_RAW128)
        assert np.array_equal(oa.get(), oracle_conv(Xa, W, b, [mul], [shift], [h_i], **kw))
        assert np.array_equal(ob.get(), oracle_conv(Xb, W, b, [mul], [shift], [h_i], **kw))
        # a missing workspace is an argument error, not a fault
        with pytest.raises(B.IconvError) as e:
            B.iconv_forward(plan, xa.data_ptr(), None, oa.ptr, None, s1.cuda_stream)
        assert e.value.status == B.ERR_ARG and "workspace" in str(e.value)
        with pytest.raises(B.IconvError) as e:
            B.iconv_forward(plan, xa.data_ptr(), None, oa.ptr, wa.ptr + 4, s1.cuda_stream)
        assert e.value.status == B.ERR_ALIGN
    finally:
        B.iconv_plan_destroy(plan)


def test_plans_without_a_repack_need_no_workspace():
    rng = np.random.default_rng(5)
    W = rng.integers(-127, 128, size=(32, 3, 3, 64), dtype=np.int8)
    plan = B.iconv_plan(n=1, h=16, w=16, c_in=64, c_out=32, kh=3, kw=3, pad=1, weights=W, bias=np.zeros(32, np.int32),
                        mul=[100], shift=[16], h_i=[100000])
    assert B.iconv_workspace_bytes(plan) == 0
    B.iconv_plan_destroy(plan)
    assert B.iconv_workspace_bytes(None) == 0


@pytest.mark.parametrize("which", [0, 1])
def test_a_bounded_wait_runs_out_and_the_context_stays_usable(which):
    """A barrier that nothing arrives at, waited on with the kernels' own wait routine and a limit
    of about a millisecond: the kernel returns, iconv_check reports the timeout once, and the next
    layer runs as if nothing had happened."""
    st = torch.cuda.current_stream().cuda_stream
    B.iconv_check(st)
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    B.iconv_selftest_wait_timeout(which, 2_000_000, st)       # about 1 ms at 1.9 GHz
    t1.record()
    with pytest.raises(B.IconvError) as e:
        B.iconv_check(st)
    assert e.value.status == B.ERR_TIMEOUT and "code 7" in str(e.value)
    assert 0.3 < t0.elapsed_time(t1) < 200.0                  # it waited for the limit, and not much longer
    B.iconv_check(st)                                         # reported once, then clear
    X, W, b, mul, shift, h_i = _stem_case(3, 1, 12, 12, 16, 16, 3)
    plan = B.iconv_plan(n=1, h=12, w=12, c_in=16, c_out=16, kh=3, kw=3, pad=1, weights=W, bias=b, mul=[mul], shift=[shift],
                        h_i=[h_i], kernel=B.KERNEL_UMMA)
    out = Fenced((1, 12, 12, 16), np.uint8)
    B.iconv_forward(plan, dev(X).data_ptr(), None, out.ptr, None, st)
    B.iconv_check(st)
    B.iconv_plan_destroy(plan)
    assert np.array_equal(out.get(), oracle_conv(X, W, b, [mul], [shift], [h_i], pad=1))
    with pytest.raises(B.IconvError):
        B.iconv_selftest_wait_timeout(2, 2_000_000, st)
    with pytest.raises(B.IconvError):
        B.iconv_selftest_wait_timeout(0, 10 ** 12, st)


def test_initialisation_is_recorded_per_device():
    """The shared-memory opt-in of the kernels and the SM count are kept per device: after a
    tensor-core plan on the current device its slot is filled, a device never used stays empty."""
    cur = torch.cuda.current_device()
    W = np.ones((16, 3, 3, 16), np.int8)
    plan = B.iconv_plan(n=1, h=8, w=8, c_in=16, c_out=16, kh=3, kw=3, pad=1, weights=W, bias=np.zeros(16, np.int32),
                        mul=[100], shift=[16], h_i=[100000], kernel=B.KERNEL_UMMA)
    B.iconv_plan_destroy(plan)
    sms = torch.cuda.get_device_properties(cur).multi_processor_count
    assert B.iconv_device_initialised(cur) == sms
    assert B.iconv_device_initialised(63) == -1 and B.iconv_device_initialised(64) == -1 and B.iconv_device_initialised(-1) == -1
