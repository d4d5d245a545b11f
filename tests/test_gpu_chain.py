"""Two consecutive 1x1 layers as one kernel (`iconv_plan_chain` / `iconv_forward_chain`) against the
oracle, which runs the two layers one after the other: both output tensors bit for bit."""
import numpy as np
import pytest
import torch

from paper_2006_11735_b200 import binding as B

from gpu_util import Fenced, dev, oracle_conv

pytestmark = pytest.mark.gpu


def _pair(seed, n, h, w, c_in, c1, c2, skip_dtype=B.U8):
    rng = np.random.default_rng(seed)
    X = rng.integers(0, 256, size=(n, h, w, c_in), dtype=np.uint8)
    S = rng.integers(0, 256, size=(n, h, w, c1), dtype=np.uint8)
    W1 = np.clip(np.floor(rng.normal(0, 30, size=(c1, 1, 1, c_in)) + 0.5), -127, 127).astype(np.int8)
    W2 = np.clip(np.floor(rng.normal(0, 30, size=(c2, 1, 1, c1)) + 0.5), -127, 127).astype(np.int8)
    b1 = rng.integers(-4096, 4097, size=(c1,), dtype=np.int32)
    b2 = rng.integers(-4096, 4097, size=(c2,), dtype=np.int32)
    h1 = int(30 * 150 * np.sqrt(c_in) * 1.7)
    h2 = int(30 * 100 * np.sqrt(c1) * 1.9)
    q1 = dict(mul=[int(np.floor(255 * 65536 / h1 + 0.5))], shift=[16], h_i=[h1])
    q2 = dict(mul=[int(np.floor(255 * 65536 / h2 + 0.5))], shift=[16], h_i=[h2])
    return X, S, W1, b1, q1, W2, b2, q2, dict(skip_dtype=skip_dtype, skip_mul=h1 // 2, skip_shift=8)


def _run(X, S, W1, b1, q1, W2, b2, q2, sk, out_c_total=None, out_c_offset=0, out2_c_total=None, out2_c_offset=0, skip_c_offset=0):
    n, h, w, c_in = X.shape
    c1, c2 = W1.shape[0], W2.shape[0]
    t1, t2 = out_c_total or c1, out2_c_total or c2
    first = dict(n=n, h=h, w=w, c_in=c_in, c_out=c1, kh=1, kw=1, weights=W1, bias=b1, out_c_total=t1, out_c_offset=out_c_offset,
                 skip_c_total=S.shape[3], skip_c_offset=skip_c_offset, **q1, **sk)
    second = dict(n=n, h=h, w=w, c_in=c1, c_out=c2, kh=1, kw=1, in_c_total=t1, in_c_offset=out_c_offset, weights=W2, bias=b2,
                  out_c_total=t2, out_c_offset=out2_c_offset, **q2)
    chain = B.iconv_plan_chain(first, second)
    try:
        o1, o2 = Fenced((n, h, w, t1), np.uint8), Fenced((n, h, w, t2), np.uint8, 0x6B)
        st = torch.cuda.current_stream().cuda_stream
        xd, sd = dev(X), dev(S)
        for _ in range(2):                  # twice: the second launch starts under the first one's tail
            B.iconv_forward_chain(chain, xd.data_ptr(), sd.data_ptr(), o1.ptr, o2.ptr, st)
        B.iconv_check(st)
        return o1.get(), o2.get()
    finally:
        B.iconv_chain_destroy(chain)


def _oracle(X, S, W1, b1, q1, W2, b2, q2, sk, out_c_total=None, out_c_offset=0, out2_c_total=None, out2_c_offset=0, skip_c_offset=0):
    c1 = W1.shape[0]
    Ssig = S.view(np.int8) if sk["skip_dtype"] == B.S8 else S
    v1 = oracle_conv(X, W1, b1, q1["mul"], q1["shift"], q1["h_i"], skip=Ssig, skip_c_offset=skip_c_offset, out_c_total=out_c_total,
                     out_c_offset=out_c_offset, **sk)
    v2 = oracle_conv(v1, W2, b2, q2["mul"], q2["shift"], q2["h_i"], in_c_offset=out_c_offset, c_in=c1, out_c_total=out2_c_total,
                     out_c_offset=out2_c_offset, fill=0x6B)
    return v1, v2


@pytest.mark.parametrize("n,h,w,c_in,c1,c2", [
    (1, 9, 11, 64, 256, 64),          # less than one pixel tile
    (3, 28, 28, 64, 256, 64),         # stage-1 shape: 18.4 pixel tiles, two N tiles
    (2, 28, 28, 64, 256, 128),        # the stage transition (256 -> 128)
    (2, 14, 14, 128, 512, 128),       # stage-2 shape: four N tiles, 64 KB + 64 KB of weights resident
    (1, 20, 20, 128, 128, 64),        # one N tile
    (1, 195, 197, 64, 256, 64),       # 300 pixel tiles: two or three per CTA, ragged last tile
])
def test_chained_pair_matches_the_two_layers_of_the_oracle(n, h, w, c_in, c1, c2):
    case = _pair(n * 1000 + h, n, h, w, c_in, c1, c2)
    got1, got2 = _run(*case)
    want1, want2 = _oracle(*case)
    bad = np.argwhere(got1 != want1)
    assert bad.shape[0] == 0, "first layer: %d mismatches, first at %s" % (bad.shape[0], bad[:1])
    bad = np.argwhere(got2 != want2)
    assert bad.shape[0] == 0, "second layer: %d mismatches, first at %s" % (bad.shape[0], bad[:1])
    assert 0.02 < (want1 == 0).mean() < 0.98 and 0.02 < (want2 == 0).mean() < 0.98
    assert np.unique(want2).size > 16


def test_chained_pair_with_channel_slices_and_signed_skip():
    """Outputs written into wider tensors at channel offsets, the skip read from a slice, int8 skip bytes."""
    X, S, W1, b1, q1, W2, b2, q2, sk = _pair(77, 2, 12, 13, 64, 256, 64, skip_dtype=B.S8)
    S = np.random.default_rng(5).integers(0, 256, size=(2, 12, 13, 288), dtype=np.uint8)
    kw = dict(out_c_total=320, out_c_offset=32, out2_c_total=96, out2_c_offset=16, skip_c_offset=16)
    got1, got2 = _run(X, S, W1, b1, q1, W2, b2, q2, sk, **kw)
    want1, want2 = _oracle(X, S, W1, b1, q1, W2, b2, q2, sk, **kw)
    assert np.array_equal(got1, want1) and np.array_equal(got2, want2)
    assert (got1[..., :32] == 0x5A).all() and (got2[..., :16] == 0x6B).all() and (got2[..., 80:] == 0x6B).all()


@pytest.mark.parametrize("change,why", [
    (dict(first=dict(kh=3, kw=3, pad=1)), "1x1"),
    (dict(second=dict(c_out=32)), "64 or 128"),
    (dict(first=dict(skip_shift=7)), "clamp-free"),
    (dict(second=dict(in_c_offset=16, in_c_total=272)), "exactly"),
])
def test_pairs_that_do_not_qualify_are_refused_with_a_reason(change, why):
    X, S, W1, b1, q1, W2, b2, q2, sk = _pair(3, 1, 8, 8, 64, 256, 64)
    first = dict(n=1, h=8, w=8, c_in=64, c_out=256, kh=1, kw=1, weights=W1, bias=b1, skip_c_total=256, **q1, **sk)
    second = dict(n=1, h=8, w=8, c_in=256, c_out=64, kh=1, kw=1, weights=W2, bias=b2, **q2)
    first.update(change.get("first", {}))
    second.update(change.get("second", {}))
    if first["kh"] == 3:
        first["weights"] = np.ones((256, 3, 3, 64), np.int8)
    if second["c_out"] == 32:
        second["weights"], second["bias"] = W2[:32], b2[:32]
    with pytest.raises(B.IconvError) as e:
        B.iconv_plan_chain(first, second)
    assert e.value.status == B.ERR_UNSUPPORTED and why in str(e.value)
