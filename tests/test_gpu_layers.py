"""GPU parity of single layers: every kernel family against the CPU oracle, bit for bit,
through the C-ABI, on shapes that span several tiles and ragged tails."""
import numpy as np
import pytest
import torch

from oracle import layers as L
from paper_2006_11735_b200 import binding as B

from gpu_util import Fenced, dev, gpu_conv, oracle_conv

pytestmark = pytest.mark.gpu


def _layer(seed, n, h, w, c_in, c_out, k, in_dtype=B.U8, per_channel=False):
    rng = np.random.default_rng(seed)
    if in_dtype == B.S8:
        X = rng.integers(-128, 128, size=(n, h, w, c_in), dtype=np.int8)
    else:
        X = rng.integers(0, 256, size=(n, h, w, c_in), dtype=np.uint8)
    W = np.clip(np.floor(rng.normal(0, 40, size=(c_out, k, k, c_in)) + 0.5), -127, 127).astype(np.int8)
    b = rng.integers(-4096, 4097, size=(c_out,), dtype=np.int32)
    sigma = 40.0 * 100.0 * np.sqrt(c_in * k * k)
    npar = c_out if per_channel else 1
    h_i = np.maximum(1, (sigma * rng.uniform(1.0, 3.0, size=npar))).astype(np.int32)
    shift = rng.integers(16, 20, size=npar).astype(np.int32)
    mul = np.maximum(1, np.floor(255.0 * 2.0 ** shift / h_i + 0.5)).astype(np.int32)
    return X, W, b, mul, shift, h_i


GENERIC_SHAPES = [
    # n, h, w, c_in, c_out, k, stride, pad
    (1, 32, 32, 64, 64, 3, 1, 1),
    (2, 9, 7, 16, 16, 3, 1, 1),
    (1, 13, 11, 3, 8, 7, 2, 3),
    (2, 10, 12, 1, 64, 5, 1, 2),
    (1, 12, 10, 48, 1, 3, 1, 1),
    (2, 8, 8, 64, 16, 5, 1, 2),
    (1, 15, 9, 48, 32, 1, 1, 0),
    (3, 7, 7, 128, 32, 3, 2, 1),
    (1, 6, 6, 5, 3, 3, 1, 0),
    (1, 1, 1, 256, 100, 1, 1, 0),
]


@pytest.mark.parametrize("shape", GENERIC_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("in_dtype", [B.U8, B.U8_RAW128, B.S8])
def test_direct_kernel_matches_oracle(shape, in_dtype):
    n, h, w, c_in, c_out, k, stride, pad = shape
    X, W, b, mul, shift, h_i = _layer(sum(shape), n, h, w, c_in, c_out, k, in_dtype)
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, stride=stride, pad=pad, in_dtype=in_dtype, kernel=B.KERNEL_DIRECT)
    want = oracle_conv(X, W, b, mul, shift, h_i, stride=stride, pad=pad, in_dtype=in_dtype)
    assert fam == B.KERNEL_DIRECT
    assert np.array_equal(got, want)
    zeros = (want == 0).mean()
    assert 0.05 < zeros < 0.95


@pytest.mark.parametrize("kernel", [B.KERNEL_DIRECT, B.KERNEL_AUTO])
def test_raw_int32_output_signed_output_per_channel_and_offsets(kernel):
    X, W, b, mul, shift, h_i = _layer(5, 2, 9, 10, 32, 48, 3, per_channel=True)
    got, _ = gpu_conv(X, W, b, mul, shift, h_i, pad=1, out_dtype=B.I32, brelu=False, kernel=kernel)
    want = oracle_conv(X, W, b, mul, shift, h_i, pad=1, out_dtype=B.I32, brelu=False)
    assert np.array_equal(got, want)
    # per-channel parameters, 8-bit output inside a wider tensor at a channel offset
    got, _ = gpu_conv(X, W, b, mul, shift, h_i, pad=1, out_c_total=80, out_c_offset=16, kernel=kernel)
    want = oracle_conv(X, W, b, mul, shift, h_i, pad=1, out_c_total=80, out_c_offset=16)
    assert np.array_equal(got, want)
    assert (got[..., :16] == 0x5A).all() and (got[..., 64:] == 0x5A).all()
    # signed output without BReLU, zero point and saturation
    got, _ = gpu_conv(X, W, b, [3], [12], [0], pad=1, out_dtype=B.S8, brelu=False, out_lo=-100, out_hi=90,
                      out_zero=-7, kernel=kernel)
    want = oracle_conv(X, W, b, [3], [12], [0], pad=1, out_dtype=B.S8, brelu=False, out_lo=-100, out_hi=90,
                       out_zero=-7)
    assert np.array_equal(got, want)
    assert (want == -100).any() and (want == 90).any() and (want < 0).any()
    # input read as a channel slice of a wider tensor
    Xw = np.random.default_rng(1).integers(0, 256, size=(2, 9, 10, 64), dtype=np.uint8)
    got, _ = gpu_conv(Xw, W, b, mul, shift, h_i, pad=1, in_c_offset=16, c_in=32, kernel=kernel)
    want = oracle_conv(Xw, W, b, mul, shift, h_i, pad=1, in_c_offset=16, c_in=32)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("kernel", [B.KERNEL_DIRECT, B.KERNEL_AUTO])
@pytest.mark.parametrize("skip_dtype", [B.U8, B.I32, B.U8_RAW128, B.S8])
def test_fused_skip_matches_oracle(kernel, skip_dtype):
    X, W, b, mul, shift, h_i = _layer(6, 2, 7, 9, 64, 64, 1)
    rng = np.random.default_rng(7)
    if skip_dtype == B.I32:
        S = rng.integers(-300000, 300000, size=(2, 7, 9, 64)).astype(np.int32)
        sm, ss = 300, 8
    elif skip_dtype == B.S8:
        S = rng.integers(-128, 128, size=(2, 7, 9, 64), dtype=np.int8)
        sm, ss = 25028137, 8
    else:
        S = rng.integers(0, 256, size=(2, 7, 9, 64), dtype=np.uint8)
        sm, ss = 428623, 8
    h_i = h_i * 4
    got, _ = gpu_conv(X, W, b, mul, shift, h_i, skip=S, skip_dtype=skip_dtype, skip_mul=sm, skip_shift=ss, kernel=kernel)
    want = oracle_conv(X, W, b, mul, shift, h_i, skip=S, skip_dtype=skip_dtype, skip_mul=sm, skip_shift=ss)
    assert np.array_equal(got, want)
    assert 0.02 < (want == 0).mean() < 0.98


def test_empty_batch_and_forward_argument_errors():
    X, W, b, mul, shift, h_i = _layer(8, 1, 8, 8, 16, 16, 3)
    plan = B.iconv_plan(n=0, h=8, w=8, c_in=16, c_out=16, kh=3, kw=3, pad=1, weights=W, bias=b, mul=mul,
                        shift=shift, h_i=h_i)
    B.iconv_forward(plan, None, None, None, None, 0)          # nothing to do, no error
    B.iconv_plan_destroy(plan)
    plan = B.iconv_plan(n=1, h=8, w=8, c_in=16, c_out=16, kh=3, kw=3, pad=1, weights=W, bias=b, mul=mul,
                        shift=shift, h_i=h_i)
    with pytest.raises(B.IconvError) as e:
        B.iconv_forward(plan, None, None, None, None, 0)
    assert e.value.status == B.ERR_ARG
    B.iconv_plan_destroy(plan)


@pytest.mark.parametrize("n_elems", [0, 1, 15, 16, 1000, 4096 + 5, 1 << 20])
@pytest.mark.parametrize("a_dtype,b_dtype,out_dtype", [(B.U8, B.U8, B.U8), (B.U8, B.I32, B.U8), (B.I32, B.I32, B.I32),
                                                        (B.S8, B.U8, B.S8)])
def test_iadd_requant_matches_oracle(n_elems, a_dtype, b_dtype, out_dtype):
    rng = np.random.default_rng(n_elems + a_dtype)

    def draw(dt):
        if dt == B.I32:
            return rng.integers(-200000, 200000, size=n_elems).astype(np.int32)
        if dt == B.S8:
            return rng.integers(-128, 128, size=n_elems, dtype=np.int8)
        return rng.integers(0, 256, size=n_elems, dtype=np.uint8)

    A, Bv = draw(a_dtype), draw(b_dtype)
    lo, hi = {B.U8: (0, 255), B.S8: (-128, 127), B.I32: (-2 ** 31, 2 ** 31 - 1)}[out_dtype]
    kw = dict(a_dtype=a_dtype, b_dtype=b_dtype, out_dtype=out_dtype, a_zero=128 if a_dtype == B.U8 else 0, b_zero=0,
              mul_a=811 if a_dtype != B.I32 else 3, sh_a=3, mul_b=1 if b_dtype == B.I32 else 500, sh_b=0,
              brelu=int(out_dtype == B.U8), h_i=150000, mul=150 if out_dtype != B.I32 else 1,
              shift=16 if out_dtype != B.I32 else 0, out_zero=0 if out_dtype != B.S8 else -3, out_lo=lo, out_hi=hi)
    want, _ = L.add_requant(A, Bv, **kw)
    np_out = {B.U8: np.uint8, B.S8: np.int8, B.I32: np.int32}[out_dtype]
    out = Fenced((n_elems,), np_out)
    if n_elems:
        ad, bd = dev(A), dev(Bv)
        B.iadd_requant(ad.data_ptr(), bd.data_ptr(), out.ptr, torch.cuda.current_stream().cuda_stream,
                       n_elems=n_elems, **kw)
    else:
        B.iadd_requant(None, None, None, 0, n_elems=0, **kw)
    torch.cuda.synchronize()
    assert np.array_equal(out.get(), want) if n_elems else True


@pytest.mark.parametrize("trial", range(12))
def test_iadd_requant_8bit_forms_with_random_descriptors(trial):
    """8-bit operands and results take a 32-bit kernel when the descriptor's bounds allow it and the
    64-bit one otherwise; both must give the oracle's bytes for any multipliers, shifts and zeros."""
    rng = np.random.default_rng(500 + trial)
    n_elems = int(rng.integers(1, 70000))
    a_dtype, b_dtype = [B.U8, B.S8][trial % 2], [B.U8, B.S8][(trial // 2) % 2]
    out_dtype = [B.U8, B.S8][(trial // 4) % 2]
    big = trial >= 8                   # multipliers that push the products beyond 32 bits: the general kernel
    A = rng.integers(0, 256, size=n_elems, dtype=np.uint8).view(np.int8 if a_dtype == B.S8 else np.uint8)
    Bv = rng.integers(0, 256, size=n_elems, dtype=np.uint8).view(np.int8 if b_dtype == B.S8 else np.uint8)
    lo, hi = (0, 255) if out_dtype == B.U8 else (-128, 127)
    kw = dict(a_dtype=a_dtype, b_dtype=b_dtype, out_dtype=out_dtype, a_zero=int(rng.integers(-5, 140)), b_zero=int(rng.integers(-5, 140)),
              mul_a=int(rng.integers(1, 2 ** 30 if big else 500000)), sh_a=int(rng.integers(20 if big else 0, 31 if big else 12)),
              mul_b=int(rng.integers(1, 3000)), sh_b=int(rng.integers(0, 12)), brelu=trial % 3 != 0, h_i=int(rng.integers(1, 300000)),
              mul=int(rng.integers(1, 400)), shift=int(rng.integers(0, 22)), out_zero=int(rng.integers(-20, 140)),
              out_lo=lo + int(rng.integers(0, 5)), out_hi=hi - int(rng.integers(0, 5)))
    want, ovf = L.add_requant(A, Bv, **kw)
    if ovf:
        pytest.skip("the drawn descriptor overflows int32 in Y")
    out = Fenced((n_elems,), np.uint8 if out_dtype == B.U8 else np.int8)
    ad, bd = dev(A), dev(Bv)
    B.iadd_requant(ad.data_ptr(), bd.data_ptr(), out.ptr, torch.cuda.current_stream().cuda_stream, n_elems=n_elems, **kw)
    torch.cuda.synchronize()
    got = out.get()
    assert np.array_equal(got, want), "%d mismatches" % (got != want).sum()


def test_pooling_matches_oracle():
    rng = np.random.default_rng(3)
    for (n, h, w, c, k, s, p) in [(2, 16, 14, 64, 3, 2, 1), (1, 9, 9, 16, 3, 2, 1), (3, 7, 8, 32, 2, 2, 0),
                                  (1, 1, 1, 16, 3, 2, 1), (2, 5, 12, 48, 3, 2, 1), (1, 6, 6, 16, 3, 1, 1)]:
        x = rng.integers(0, 256, size=(n, h, w, c), dtype=np.uint8)
        want = L.maxpool(x, k, s, p)
        out = Fenced(want.shape, np.uint8)
        xd = dev(x)
        B.ipool_max(xd.data_ptr(), out.ptr, n, h, w, c, k, s, p, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert np.array_equal(out.get(), want)
    for (n, h, w, c) in [(3, 7, 7, 2048), (2, 2, 2, 40), (1, 5, 3, 7)]:
        x = rng.integers(0, 256, size=(n, h, w, c), dtype=np.uint8)
        mul = (2 ** 16 * 2 + h * w) // (2 * h * w)
        want = L.avgpool_requant(x, mul, 16)
        out = Fenced(want.shape, np.uint8)
        xd = dev(x)
        B.ipool_avg_requant(xd.data_ptr(), out.ptr, n, h, w, c, mul, 16, 255, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert np.array_equal(out.get(), want)


def test_maxpool_with_32_byte_accesses_matches_oracle():
    """3x3/2 pooling over channel counts that are multiples of 32 on 32-byte aligned tensors takes the kernel
    with 32-byte loads and stores; odd sizes, one-pixel images and several images."""
    rng = np.random.default_rng(5)
    for (n, h, w, c) in [(2, 16, 14, 64), (3, 7, 9, 32), (1, 1, 1, 96), (2, 112, 112, 64), (1, 5, 12, 128)]:
        x = rng.integers(0, 256, size=(n, h, w, c), dtype=np.uint8)
        want = L.maxpool(x, 3, 2, 1)
        xd = dev(x)
        out = torch.full(want.shape, 0x5A, dtype=torch.uint8, device="cuda")
        assert xd.data_ptr() % 32 == 0 and out.data_ptr() % 32 == 0
        B.ipool_max(xd.data_ptr(), out.data_ptr(), n, h, w, c, 3, 2, 1, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy(), want)


UMMA_SHAPES = [
    # n, h, w, c_in, c_out, k, stride, pad
    (1, 32, 32, 64, 64, 3, 1, 1),       # configuration 1
    (2, 9, 7, 16, 16, 3, 1, 1),         # one ragged tile
    (3, 13, 11, 32, 32, 3, 1, 1),       # several tiles + tail, 32-byte swizzle
    (2, 12, 12, 64, 16, 5, 1, 2),       # VRCNN 5x5 branch
    (2, 12, 12, 64, 32, 3, 1, 1),
    (2, 11, 13, 48, 16, 3, 1, 1),       # 48 channels: chunk wider than the tensor
    (2, 11, 13, 48, 32, 1, 1, 0),
    (2, 14, 14, 128, 128, 3, 2, 1),     # stride 2, 128-byte swizzle
    (2, 14, 14, 256, 512, 1, 2, 0),     # strided projection, two N tiles
    (1, 9, 9, 256, 64, 1, 1, 0),
    (2, 7, 7, 512, 512, 3, 1, 1),       # long reduction: 36 pipeline iterations
    (5, 1, 1, 2048, 1000, 1, 1, 0),     # fully connected, padded N
    (1, 20, 20, 64, 256, 1, 1, 0),
    (2, 6, 10, 64, 48, 3, 1, 1),        # N = 48
]


PAIR_SHAPES = [
    # long reductions the plan runs on CTA pairs (256-pixel tiles, each CTA loads half of every B tile);
    # n, h, w, c_in, c_out, k, stride, pad
    (2, 14, 14, 256, 256, 3, 1, 1),     # stage-3 3x3: 18 k-iterations, 4 pixel tiles = 2 pairs
    (6, 14, 14, 256, 256, 3, 2, 1),     # stride 2: 294 pixels = 3 pixel tiles, the last pair's second CTA has none
    (3, 14, 14, 1024, 256, 1, 1, 0),    # 5 pixel tiles: the last pair's second CTA has no real pixel at all
    (2, 15, 15, 512, 512, 1, 1, 0),     # two N tiles of 256, 450 pixels
    (40, 14, 14, 1024, 128, 1, 1, 0),   # N = 128 (64 rows of B per CTA), 62 pixel tiles
    (8, 7, 7, 512, 512, 3, 1, 1),       # stage-4 3x3 on 7 x 7 maps, 392 pixels
    (150, 14, 14, 256, 256, 3, 1, 1),   # 230 pixel tiles: more pairs than SM pairs, ragged schedule
]


@pytest.mark.parametrize("shape", PAIR_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("skip", [None, B.U8], ids=["plain", "skip8"])
def test_cta_pair_form_matches_oracle(shape, skip):
    n, h, w, c_in, c_out, k, stride, pad = shape
    if n > 100 and skip is not None:
        pytest.skip("the large case runs once")
    X, W, b, mul, shift, h_i = _layer(sum(shape) + 7, n, h, w, c_in, c_out, k)
    kw = dict(stride=stride, pad=pad)
    if skip is not None:
        ho, wo = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
        S = np.random.default_rng(3).integers(0, 256, size=(n, ho, wo, c_out), dtype=np.uint8)
        kw.update(skip=S, skip_dtype=skip, skip_mul=int(h_i[0]) // 2, skip_shift=8)
    want = oracle_conv(X, W, b, mul, shift, h_i, **kw)
    text = []
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, kernel=B.KERNEL_UMMA, describe=text, **kw)
    assert fam == B.KERNEL_UMMA and "cta pairs" in text[0], text[0]
    bad = np.argwhere(got != want)
    assert bad.shape[0] == 0, "%d mismatches, first at %s" % (bad.shape[0], bad[:1])
    assert 0.02 < (want == 0).mean() < 0.98
    # the single-CTA form of the same layer
    text = []
    got1, _ = gpu_conv(X, W, b, mul, shift, h_i, kernel=B.KERNEL_UMMA_IM2COL, describe=text, **kw)
    assert "cta pairs" not in text[0] and np.array_equal(got1, want)


WINDOW_SHAPES = [
    # stride-1 filters the plan runs in window mode (one patch load per tile); n, h, w, c_in, c_out, k, stride, pad
    (2, 5, 256, 64, 64, 3, 1, 1),       # VDSR rows: two 128-pixel strips per row
    (1, 6, 260, 64, 32, 3, 1, 1),       # ragged third strip
    (1, 9, 250, 64, 16, 5, 1, 2),       # VRCNN 5x5 branch, 16 output channels
    (2, 30, 26, 48, 16, 3, 1, 1),       # 48 channels in a 64-byte row
    (3, 28, 28, 128, 128, 3, 1, 1),     # 128-byte rows, tiles across rows, ragged last tile per image
    (2, 20, 17, 32, 64, 3, 1, 0),       # no padding: the output is narrower than the input
    (1, 40, 33, 16, 256, 3, 1, 1),      # two column halves per tile
    (2, 12, 50, 64, 48, 5, 1, 4),       # padding wider than the filter needs
    (1, 37, 150, 64, 64, 3, 1, 1),      # 8 x 16 pixel blocks, ragged on the right and at the bottom
    (2, 35, 133, 64, 16, 5, 1, 2),      # blocks under a 5x5 filter
    (1, 6, 260, 48, 32, 1, 1, 0),       # a 1x1 layer as strips of one row
    (2, 24, 24, 64, 64, 1, 1, 0),       # a 1x1 layer as blocks
]

# the tiling (of the three window mode has) that the plan's cost model picks for these shapes
WINDOW_TILINGS = {
    (1, 37, 150, 64, 64, 3, 1, 1): "window(blocks)",
    (3, 28, 28, 128, 128, 3, 1, 1): "window(rows)",
    (1, 6, 260, 48, 32, 1, 1, 0): "window(strips)",
}


@pytest.mark.parametrize("shape", UMMA_SHAPES + WINDOW_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("kernel", [B.KERNEL_UMMA, B.KERNEL_UMMA_IM2COL], ids=["plan", "im2col"])
def test_tensor_core_kernel_matches_oracle(shape, kernel):
    n, h, w, c_in, c_out, k, stride, pad = shape
    X, W, b, mul, shift, h_i = _layer(sum(shape) + 1, n, h, w, c_in, c_out, k)
    if c_out % 16:
        got, fam = gpu_conv(X, W, b, mul, shift, h_i, stride=stride, pad=pad, out_dtype=B.I32, brelu=False,
                            kernel=kernel)
        want = oracle_conv(X, W, b, mul, shift, h_i, stride=stride, pad=pad, out_dtype=B.I32, brelu=False)
    else:
        text = []
        got, fam = gpu_conv(X, W, b, mul, shift, h_i, stride=stride, pad=pad, kernel=kernel, describe=text)
        # the shapes listed for window mode must really run in it when the plan is free to choose
        if kernel == B.KERNEL_UMMA_IM2COL:
            assert "im2col" in text[0], text[0]
        elif shape in WINDOW_SHAPES:
            assert "window" in text[0], text[0]
            if shape in WINDOW_TILINGS:      # so that every tiling is known to be covered
                assert WINDOW_TILINGS[shape] in text[0], text[0]
        want = oracle_conv(X, W, b, mul, shift, h_i, stride=stride, pad=pad)
        assert 0.05 < (want == 0).mean() < 0.95
    assert fam == B.KERNEL_UMMA
    bad = np.argwhere(got != want)
    assert bad.shape[0] == 0, "%d mismatches, first at %s: got %s want %s" % (
        bad.shape[0], bad[0], got[tuple(bad[0])], want[tuple(bad[0])])


@pytest.mark.parametrize("kernel", [B.KERNEL_UMMA, B.KERNEL_UMMA_IM2COL], ids=["plan", "im2col"])
def test_tensor_core_kernel_signed_activations_and_large_batch_tail(kernel):
    X, W, b, mul, shift, h_i = _layer(77, 7, 19, 17, 64, 64, 3, in_dtype=B.S8)
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, pad=1, in_dtype=B.S8, kernel=kernel)
    want = oracle_conv(X, W, b, mul, shift, h_i, pad=1, in_dtype=B.S8)
    assert fam == B.KERNEL_UMMA and np.array_equal(got, want)
    # window mode with the explicit-clamp epilogue (a signed output with a zero point) inside a wider tensor
    X, W, b, mul, shift, h_i = _layer(79, 2, 21, 23, 64, 32, 3)
    kw = dict(pad=1, out_dtype=B.S8, out_lo=-100, out_hi=100, out_zero=-90, out_c_total=64, out_c_offset=32)
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, kernel=kernel, **kw)
    want = oracle_conv(X, W, b, mul, shift, h_i, **kw)
    assert fam == B.KERNEL_UMMA and np.array_equal(got, want)


def test_tensor_core_kernel_rejects_what_it_cannot_take():
    X, W, b, mul, shift, h_i = _layer(78, 1, 8, 8, 3, 16, 3)
    with pytest.raises(B.IconvError) as e:
        gpu_conv(X, W, b, mul, shift, h_i, pad=1, kernel=B.KERNEL_UMMA)
    assert e.value.status == B.ERR_UNSUPPORTED


@pytest.mark.parametrize("shape", [(2, 30, 26, 64), (1, 33, 31, 16), (3, 16, 16, 32)], ids=str)
@pytest.mark.parametrize("in_dtype", [B.U8_RAW128, B.U8, B.S8])
def test_stem_path_matches_oracle(shape, in_dtype):
    n, h, w, c_out = shape
    X, W, b, mul, shift, h_i = _layer(h * w + c_out, n, h, w, 3, c_out, 7, in_dtype)
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, stride=2, pad=3, in_dtype=in_dtype, kernel=B.KERNEL_STEM)
    want = oracle_conv(X, W, b, mul, shift, h_i, stride=2, pad=3, in_dtype=in_dtype)
    assert fam == B.KERNEL_STEM
    assert np.array_equal(got, want)
    assert 0.05 < (want == 0).mean() < 0.95
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, stride=2, pad=3, in_dtype=in_dtype)
    assert fam == B.KERNEL_STEM and np.array_equal(got, want)      # AUTO picks it too


ROWS_SHAPES = [
    # single-channel images repacked for the tensor cores: n, h, w, c_out, kh, kw, pad
    (2, 40, 48, 64, 3, 3, 1),           # VDSR first layer
    (2, 21, 37, 64, 5, 5, 2),           # VRCNN first layer, ragged sizes
    (1, 37, 150, 32, 3, 5, 2),          # a filter that is not square, padding beyond what it needs vertically
    (3, 19, 9, 48, 7, 2, 0),            # no padding, output narrower than the image
    (1, 18, 140, 64, 1, 16, 3),         # the widest filter row the repack holds
]


@pytest.mark.parametrize("shape", ROWS_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("in_dtype", [B.U8_RAW128, B.U8, B.S8])
def test_single_channel_repack_path_matches_oracle(shape, in_dtype):
    n, h, w, c_out, kh, kw, pad = shape
    rng = np.random.default_rng(sum(shape) + in_dtype)
    X = rng.integers(0, 256, size=(n, h, w, 1), dtype=np.uint8)
    if in_dtype == B.S8:
        X = X.view(np.int8)
    W = np.clip(np.floor(rng.normal(0, 40, size=(c_out, kh, kw, 1)) + 0.5), -127, 127).astype(np.int8)
    b = rng.integers(-2048, 2049, size=(c_out,), dtype=np.int32)
    h_i = np.array([int(40 * 74 * np.sqrt(kh * kw) * 2)], dtype=np.int32)
    mul = np.array([int(np.floor(255.0 * 2.0 ** 16 / h_i[0] + 0.5))], dtype=np.int32)
    shift = np.array([16], dtype=np.int32)
    want = oracle_conv(X, W, b, mul, shift, h_i, pad=pad, in_dtype=in_dtype)
    assert 0.05 < (want == 0).mean() < 0.95
    for kernel in (B.KERNEL_STEM, B.KERNEL_AUTO):
        got, fam = gpu_conv(X, W, b, mul, shift, h_i, pad=pad, in_dtype=in_dtype, kernel=kernel)
        assert fam == B.KERNEL_STEM
        bad = np.argwhere(got != want)
        assert bad.shape[0] == 0, "%d mismatches, first at %s: got %s want %s" % (
            bad.shape[0], bad[0], got[tuple(bad[0])], want[tuple(bad[0])])


NARROW_SHAPES = [
    # 8-bit outputs too narrow or too oddly placed for 16-byte stores: n, h, w, c_in, c_out, k, pad, out_c_total, out_c_offset
    (2, 40, 48, 64, 1, 3, 1, 1, 0),         # VDSR last layer
    (1, 37, 150, 48, 1, 3, 1, 1, 0),        # VRCNN last layer, block tiling with ragged edges
    (2, 21, 19, 32, 3, 5, 2, 3, 0),         # three channels (a colour picture)
    (1, 30, 26, 64, 24, 3, 1, 40, 9),       # 24 channels at an odd offset of a wider tensor
    (2, 16, 16, 16, 7, 1, 0, 7, 0),         # a 1x1 layer
]


@pytest.mark.parametrize("shape", NARROW_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("skip_dtype", [-1, B.U8_RAW128, B.S8], ids=["noskip", "skipraw", "skips8"])
def test_narrow_outputs_on_the_tensor_cores_match_oracle(shape, skip_dtype):
    n, h, w, c_in, c_out, k, pad, out_c_total, out_c_offset = shape
    X, W, b, mul, shift, h_i = _layer(sum(shape) + 5, n, h, w, c_in, c_out, k, per_channel=(c_out == 24))
    ho, wo = h + 2 * pad - k + 1, w + 2 * pad - k + 1
    kw = dict(pad=pad, out_c_total=out_c_total, out_c_offset=out_c_offset)
    if skip_dtype >= 0:
        S = np.random.default_rng(7).integers(0, 256, size=(n, ho, wo, c_out + 2), dtype=np.uint8)
        if skip_dtype == B.S8:
            S = S.view(np.int8)
        kw.update(skip=S, skip_dtype=skip_dtype, skip_c_offset=1, skip_mul=int(h_i[0]) // 300, skip_shift=1)
    want = oracle_conv(X, W, b, mul, shift, h_i, **kw)
    text = []
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, kernel=B.KERNEL_UMMA, describe=text, **kw)
    assert fam == B.KERNEL_UMMA and "window" in text[0], text
    bad = np.argwhere(got != want)
    assert bad.shape[0] == 0, "%d mismatches, first at %s: got %s want %s" % (
        bad.shape[0], bad[0], got[tuple(bad[0])], want[tuple(bad[0])])
    assert np.unique(want[..., out_c_offset:out_c_offset + c_out]).size > 8


def test_mma_issue_rate_probe_reports_a_plausible_peak():
    import bench
    tops, cycles = bench.probe_mma_rate(256, 20000)
    assert 100.0 <= cycles <= 400.0          # 128 cycles per M128 N256 K32 instruction at the nominal rate
    assert 1000.0 < tops < 10000.0
    with pytest.raises(RuntimeError):
        bench.probe_mma_rate(100, 10)
    # 64-byte rows with the block tiling's group stride, 64 columns: half the work per instruction at
    # about the same duration
    tops64, cycles64 = bench.probe_mma_rate_rows(64, 64, 640, 20000)
    assert 30.0 <= cycles64 <= 200.0 and tops64 < tops
    with pytest.raises(RuntimeError):
        bench.probe_mma_rate_rows(64, 48, 512, 10)


THIN_SHAPES = [
    # n, h, w, c_in, c_out, k, stride, pad
    (2, 40, 48, 1, 64, 3, 1, 1),        # VDSR first layer
    (2, 21, 37, 1, 64, 5, 1, 2),        # VRCNN first layer, ragged sizes
    (1, 9, 11, 1, 16, 3, 2, 1),         # one channel group, stride 2
    (3, 8, 8, 1, 128, 1, 1, 0),
    (2, 40, 48, 64, 1, 3, 1, 1),        # VDSR last layer
    (2, 19, 23, 48, 1, 3, 1, 1),        # VRCNN last layer: three lanes per pixel
    (1, 7, 9, 16, 1, 5, 1, 2),
    (2, 6, 6, 512, 1, 1, 1, 0),         # a whole warp per pixel
]


@pytest.mark.parametrize("shape", THIN_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("in_dtype", [B.U8, B.U8_RAW128, B.S8])
def test_thin_kernels_match_oracle(shape, in_dtype):
    n, h, w, c_in, c_out, k, stride, pad = shape
    if c_out == 1 and in_dtype == B.U8_RAW128:
        pytest.skip("raw-128 input is a first-layer format")
    X, W, b, mul, shift, h_i = _layer(sum(shape) + 3, n, h, w, c_in, c_out, k, in_dtype)
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, stride=stride, pad=pad, in_dtype=in_dtype, kernel=B.KERNEL_THIN)
    want = oracle_conv(X, W, b, mul, shift, h_i, stride=stride, pad=pad, in_dtype=in_dtype)
    assert fam == B.KERNEL_THIN
    assert np.array_equal(got, want)
    if c_out == 1:          # one channel, one bias: the zero share of a small sample is arbitrary
        assert (want == 0).mean() < 0.95 and np.unique(want).size > 8
    else:
        assert 0.05 < (want == 0).mean() < 0.95
    # AUTO picks it too, except where a single-channel layer can be repacked for the tensor cores
    # or a single-channel output comes out of the tensor-core window mode byte by byte
    repack = c_in == 1 and stride == 1 and k > 1 and c_out >= 32
    narrow = c_out == 1 and c_in <= 128 and h * w >= 256
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, stride=stride, pad=pad, in_dtype=in_dtype)
    assert fam == (B.KERNEL_STEM if repack else B.KERNEL_UMMA if narrow else B.KERNEL_THIN) and np.array_equal(got, want)


def test_thin_kernels_variants():
    # c_in = 1 into a channel offset of a wider tensor, per-channel parameters, wide (64-bit) Eq. 4
    X, W, b, mul, shift, h_i = _layer(91, 2, 17, 13, 1, 32, 3, B.U8_RAW128, per_channel=True)
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, pad=1, in_dtype=B.U8_RAW128, out_c_total=64, out_c_offset=16,
                        kernel=B.KERNEL_THIN)
    want = oracle_conv(X, W, b, mul, shift, h_i, pad=1, in_dtype=B.U8_RAW128, out_c_total=64, out_c_offset=16)
    assert fam == B.KERNEL_THIN and np.array_equal(got, want)
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, pad=1, in_dtype=B.U8_RAW128, out_c_total=64, out_c_offset=16)
    assert fam == B.KERNEL_STEM and np.array_equal(got, want)      # repacked: per-channel parameters on the tensor-core path
    # h_i * mul >= 2^32: no 32-bit epilogue, so no window mode, so AUTO leaves the layer to the thin kernel
    got, fam = gpu_conv(X, W, b, mul * 4096, shift + 12, h_i, pad=1, in_dtype=B.U8_RAW128)
    want = oracle_conv(X, W, b, mul * 4096, shift + 12, h_i, pad=1, in_dtype=B.U8_RAW128)
    assert fam == B.KERNEL_THIN and np.array_equal(got, want)
    # c_out = 1 with the global residual: raw image skip, no BReLU, zero point 128 (the regression output)
    X, W, b, mul, shift, h_i = _layer(92, 2, 18, 22, 64, 1, 3)
    S = np.random.default_rng(5).integers(0, 256, size=(2, 18, 22, 1), dtype=np.uint8)
    kw = dict(pad=1, brelu=False, out_zero=128, skip=S, skip_dtype=B.U8_RAW128, skip_mul=3000, skip_shift=2)
    got, fam = gpu_conv(X, W, b, [20], [14], [0], kernel=B.KERNEL_THIN, **kw)
    want = oracle_conv(X, W, b, [20], [14], [0], **kw)
    assert fam == B.KERNEL_THIN and np.array_equal(got, want)
    assert (want == 0).any() and (want == 255).any() and ((want > 0) & (want < 255)).mean() > 0.3
    text = []
    got, fam = gpu_conv(X, W, b, [20], [14], [0], describe=text, **kw)       # AUTO: the tensor cores, byte stores
    assert fam == B.KERNEL_UMMA and "window" in text[0] and np.array_equal(got, want)
    # c_out = 1, raw int32 output
    got, fam = gpu_conv(X, W, b, [1], [0], [0], pad=1, out_dtype=B.I32, brelu=False)
    want = oracle_conv(X, W, b, [1], [0], [0], pad=1, out_dtype=B.I32, brelu=False)
    assert fam == B.KERNEL_THIN and np.array_equal(got, want)


@pytest.mark.parametrize("case", [
    # n, h, w, c_prev, width, c_out, stride
    (2, 12, 12, 64, 64, 256, 1),        # stage 1: both reductions 64 wide, two 128-column tiles
    (2, 12, 10, 256, 128, 512, 2),      # strided projection over the block input
    (1, 8, 8, 32, 16, 48, 1),           # narrow: four accumulator buffers, padded columns
], ids=str)
@pytest.mark.parametrize("skip_mul,skip_shift", [(766, 8), (20011, 14)], ids=["rescale32", "rescale64"])
def test_fused_projection_equals_projection_layer_plus_int32_skip(case, skip_mul, skip_shift):
    n, h, w, c_prev, width, c_out, stride = case
    ho, wo = (h - 1) // stride + 1, (w - 1) // stride + 1
    rng = np.random.default_rng(sum(case))
    X0 = rng.integers(0, 256, size=(n, h, w, c_prev), dtype=np.uint8)            # block input: the projection's operand
    Xb = rng.integers(0, 256, size=(n, ho, wo, width), dtype=np.uint8)           # output of the block's 3x3
    _, Wp, bp, _, _, _ = _layer(3, 1, 1, 1, c_prev, c_out, 1)
    _, W, b, mul, shift, h_i = _layer(4, 1, 1, 1, width, c_out, 1)
    h_i = h_i * 6
    # oracle: the projection as a layer of its own (int32 Y), then the closing layer with that int32 skip
    S = oracle_conv(X0, Wp, bp, [1], [0], [0], stride=stride, out_dtype=B.I32, brelu=False)
    want = oracle_conv(Xb, W, b, mul, shift, h_i, skip=S, skip_dtype=B.I32, skip_mul=skip_mul, skip_shift=skip_shift)
    plan = B.iconv_plan(n=n, h=ho, w=wo, c_in=width, c_out=c_out, kh=1, kw=1, weights=W, bias=b, mul=mul, shift=shift, h_i=h_i,
                        skip_dtype=B.U8, skip_mul=skip_mul, skip_shift=skip_shift,
                        proj=dict(weights=Wp, bias=bp, h=h, w=w, stride=stride, pad=0))
    try:
        assert B.iconv_plan_kernel(plan) == B.KERNEL_UMMA
        out = Fenced(want.shape, np.uint8)
        xd, sd = dev(Xb), dev(X0)
        st = torch.cuda.current_stream().cuda_stream
        B.iconv_forward(plan, xd.data_ptr(), sd.data_ptr(), out.ptr, None, st)
        B.iconv_check(st)
        got = out.get()
    finally:
        B.iconv_plan_destroy(plan)
    bad = np.argwhere(got != want)
    assert bad.shape[0] == 0, "%d mismatches, first at %s" % (bad.shape[0], bad[0])
    assert 0.02 < (want == 0).mean() < 0.98 and (want == 255).mean() < 0.9


@pytest.mark.parametrize("max_int", [127, 63, 31, 15], ids=lambda m: "max_int%d" % m)
@pytest.mark.parametrize("kernel", [B.KERNEL_UMMA, B.KERNEL_UMMA_IM2COL, B.KERNEL_DIRECT], ids=["plan", "im2col", "direct"])
def test_activation_bit_depth_sweep_matches_oracle(max_int, kernel):
    """Activations of 7, 6, 5 and 4 bits (the bit-depth sweep of Table 5): the stored values stay in
    [0, max_int], the BReLU bound and Eq. 4's (mul, shift) come from Section 3.3 for that max_int,
    and the output saturates at max_int instead of 255."""
    from oracle import planner as OP
    rng = np.random.default_rng(1000 + max_int)
    n, h, w, c_in, c_out = 2, 22, 26, 64, 64
    X = rng.integers(0, max_int + 1, size=(n, h, w, c_in), dtype=np.uint8)
    W = np.clip(np.floor(rng.normal(0, 40, size=(c_out, 3, 3, c_in)) + 0.5), -127, 127).astype(np.int8)
    b = rng.integers(-2048, 2049, size=(c_out,), dtype=np.int32)
    h_ri = int(40.0 * (max_int / 2.5) * np.sqrt(c_in * 9) * 2)
    q = OP.brelu_params_from_h_ri(h_ri, 1.0, max_int)
    mul, shift, h_i = [q["mul"]], [q["shift"]], [q["h_i"]]
    S = rng.integers(0, max_int + 1, size=(n, h, w, c_out), dtype=np.uint8)
    for kw in (dict(pad=1, out_hi=max_int),
               dict(pad=1, out_hi=max_int, skip=S, skip_dtype=B.U8, skip_mul=int(h_ri / max_int * 64), skip_shift=8)):
        want = oracle_conv(X, W, b, mul, shift, h_i, **kw)
        got, fam = gpu_conv(X, W, b, mul, shift, h_i, kernel=kernel, **kw)
        assert np.array_equal(got, want)
        assert want.max() == max_int and (want == 0).mean() > 0.02 and ((want > 0) & (want < max_int)).mean() > 0.2


WINDOW_SKIP_SHAPES = [
    # stride-1 layers with an 8-bit identity skip (the closing 3x3 of a basic block): n, h, w, c, k, pad
    (2, 28, 28, 64, 3, 1),              # block tiling, 64-byte rows
    (1, 37, 150, 64, 3, 1),             # ragged blocks
    (3, 14, 14, 128, 3, 1),             # 128-byte rows, tiles across rows
    (2, 20, 24, 64, 1, 0),              # a 1x1 with a skip
    (1, 6, 260, 32, 5, 2),              # strips, another filter size (the generic issue path)
]


@pytest.mark.parametrize("shape", WINDOW_SKIP_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("skip_dtype", [B.U8, B.U8_RAW128, B.S8], ids=["u8", "raw128", "s8"])
@pytest.mark.parametrize("variant", ["fast", "safe"])
def test_window_mode_with_identity_skip_matches_oracle(shape, skip_dtype, variant):
    n, h, w, c, k, pad = shape
    X, W, b, mul, shift, h_i = _layer(sum(shape) + 11, n, h, w, c, c, k)
    ho, wo = h + 2 * pad - k + 1, w + 2 * pad - k + 1
    rng = np.random.default_rng(sum(shape))
    S = rng.integers(0, 256, size=(n, ho, wo, c + 16), dtype=np.uint8)
    if skip_dtype == B.S8:
        S = S.view(np.int8)
    kw = dict(pad=pad, skip=S, skip_dtype=skip_dtype, skip_c_offset=16, skip_mul=int(h_i[0]) // 200, skip_shift=2)
    if variant == "safe":               # a zero point and a narrower range: the explicit-clamp epilogue
        kw.update(out_zero=3, out_lo=3, out_hi=200)
    h_i = h_i * 2
    want = oracle_conv(X, W, b, mul, shift, h_i, **kw)
    assert 0.02 < (want == want.min()).mean() < 0.98 and np.unique(want).size > 16
    for kernel in (B.KERNEL_UMMA, B.KERNEL_UMMA_IM2COL):
        text = []
        got, fam = gpu_conv(X, W, b, mul, shift, h_i, kernel=kernel, describe=text, **kw)
        assert fam == B.KERNEL_UMMA and ("window" in text[0]) == (kernel == B.KERNEL_UMMA), text
        bad = np.argwhere(got != want)
        assert bad.shape[0] == 0, "%s: %d mismatches, first at %s: got %s want %s" % (
            text[0], bad.shape[0], bad[0], got[tuple(bad[0])], want[tuple(bad[0])])


MANY_TILE_SHAPES = [
    # enough tiles that every MMA-issuing warp of a CTA takes several and the stage and accumulator rings wrap
    # many times: n, h, w, c_in, c_out, text the plan must show
    (96, 28, 28, 128, 128, "stages=2"),         # tiles across image rows, two stages (a large filter bank): two issuers
    (6, 256, 256, 64, 64, "stages=6"),          # six stages, eight accumulator buffers: three issuers
    (40, 56, 56, 64, 64, "window(blocks)"),     # ragged blocks at the bottom of every image
]


@pytest.mark.parametrize("shape", MANY_TILE_SHAPES, ids=lambda s: "x".join(map(str, s[:5])))
def test_window_mode_with_many_tiles_per_cta_matches_oracle(shape):
    """The issuing warps take a CTA's tiles in turn and wait by phase parity; every stage's fills must stay with
    one of them.  Several hundred to several thousand tiles on the GPU's CTAs, against the oracle."""
    n, h, w, c_in, c_out, expect = shape
    X, W, b, mul, shift, h_i = _layer(sum(shape[:5]) + 37, n, h, w, c_in, c_out, 3)
    want = oracle_conv(X, W, b, mul, shift, h_i, pad=1)
    text = []
    got, fam = gpu_conv(X, W, b, mul, shift, h_i, pad=1, kernel=B.KERNEL_UMMA, describe=text)
    assert fam == B.KERNEL_UMMA and "window" in text[0] and expect in text[0], text
    fields = dict(f.split("=") for f in text[0].split() if "=" in f)
    stages, issuers, nbuf = int(fields["stages"]), int(fields["issuers"]), int(fields["nbuf"])
    assert stages % issuers == 0 and (issuers == 2 or stages <= nbuf), text      # a stage's fills stay with one issuer
    assert np.array_equal(got, want)
