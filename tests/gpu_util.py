"""Helpers of the GPU parity tests: run one layer through the C-ABI on device buffers that
are fenced by canary bytes, and the oracle call with the same arguments."""
import numpy as np
import torch

from oracle import layers as L
from paper_2006_11735_b200 import binding as B

CANARY = 0xA5
FENCE = 256
_NP = {B.U8: np.uint8, B.S8: np.int8, B.I32: np.int32, B.U8_RAW128: np.uint8}


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


class Fenced:
    """A device buffer with FENCE canary bytes on both sides, prefilled with ``fill``."""

    def __init__(self, shape, np_dtype, fill=0x5A):
        self.shape, self.np_dtype = shape, np_dtype
        self.nbytes = int(np.prod(shape)) * np.dtype(np_dtype).itemsize
        self.raw = torch.full((self.nbytes + 2 * FENCE,), CANARY, dtype=torch.uint8, device="cuda")
        self.raw[FENCE:FENCE + self.nbytes] = fill
        self.ptr = self.raw.data_ptr() + FENCE
        assert self.ptr % 16 == 0

    def get(self) -> np.ndarray:
        h = self.raw.cpu().numpy()
        assert (h[:FENCE] == CANARY).all() and (h[FENCE + self.nbytes:] == CANARY).all(), "canary overwritten"
        return h[FENCE:FENCE + self.nbytes].view(self.np_dtype).reshape(self.shape).copy()


def workspace_for(plan):
    """A canary-fenced device buffer of exactly ``iconv_workspace_bytes(plan)`` bytes, or None."""
    size = B.iconv_workspace_bytes(plan)
    return Fenced((size,), np.uint8, 0xC3) if size else None


def gpu_conv(X, W, b, mul, shift, h_i, *, stride=1, pad=0, in_dtype=B.U8, in_c_offset=0, c_in=None,
             out_dtype=B.U8, out_c_total=None, out_c_offset=0, brelu=True, out_lo=0, out_hi=255, out_zero=0,
             skip=None, skip_dtype=-1, skip_c_offset=0, skip_mul=1, skip_shift=0, kernel=B.KERNEL_AUTO,
             fill=0x5A, describe=None):
    n, h, w, in_c_total = X.shape
    c_out, kh, kw, wc = W.shape
    c_in = wc if c_in is None else c_in
    ho, wo = L.out_hw(h, w, kh, kw, stride, pad)
    out_c_total = c_out if out_c_total is None else out_c_total
    plan = B.iconv_plan(n=n, h=h, w=w, c_in=c_in, c_out=c_out, kh=kh, kw=kw, stride=stride, pad=pad,
                        in_dtype=in_dtype, in_c_total=in_c_total, in_c_offset=in_c_offset, out_dtype=out_dtype,
                        out_c_total=out_c_total, out_c_offset=out_c_offset, brelu=int(brelu), out_lo=out_lo,
                        out_hi=out_hi, out_zero=out_zero, skip_dtype=skip_dtype,
                        skip_c_total=0 if skip is None else skip.shape[3], skip_c_offset=skip_c_offset,
                        skip_mul=skip_mul, skip_shift=skip_shift, kernel=kernel,
                        weights=W, bias=b, mul=mul, shift=shift, h_i=h_i)
    try:
        if describe is not None:
            describe.append(B.iconv_plan_describe(plan))
        xd = dev(X)
        sd = dev(skip) if skip is not None else None
        out = Fenced((n, ho, wo, out_c_total), _NP[out_dtype], fill)
        ws = workspace_for(plan)
        B.iconv_forward(plan, xd.data_ptr(), sd.data_ptr() if sd is not None else None, out.ptr,
                        ws.ptr if ws is not None else None, torch.cuda.current_stream().cuda_stream)
        if ws is not None:
            ws.get()            # the canaries around the workspace must be intact
        B.iconv_check(torch.cuda.current_stream().cuda_stream)
        return out.get(), B.iconv_plan_kernel(plan)
    finally:
        B.iconv_plan_destroy(plan)


def oracle_conv(X, W, b, mul, shift, h_i, *, out_c_total=None, fill=0x5A, out_dtype=B.U8, kernel=None, **kw):
    """Same call on the oracle; the untouched channels of a wider output keep ``fill``."""
    n, h, w, _ = X.shape
    c_out, kh, kwid, _ = W.shape
    ho, wo = L.out_hw(h, w, kh, kwid, kw.get("stride", 1), kw.get("pad", 0))
    out_c_total = c_out if out_c_total is None else out_c_total
    out = np.full((n, ho, wo, out_c_total), fill, dtype=np.uint8).view(np.int8 if out_dtype == B.S8 else np.uint8)
    if out_dtype == B.I32:
        out = np.frombuffer(np.full(n * ho * wo * out_c_total * 4, fill, dtype=np.uint8).tobytes(),
                            dtype=np.int32).reshape(n, ho, wo, out_c_total).copy()
    res, ovf = L.conv(X, W, b, mul, shift, h_i, out=out, out_dtype=out_dtype, **kw)
    assert not ovf
    return res
