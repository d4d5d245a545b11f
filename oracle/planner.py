"""TEST INFRASTRUCTURE -- the paper's closed-form parameter arithmetic, written out plainly.

Covers weight quantisation (Eq. 1-2), the ratio bookkeeping (Eq. 3), the quantised
BReLU parameters (Section 3.3, Eq. 7-13), ``mul_shift`` (named by Eq. 9, never defined
in the paper), ratio synchronisation of a residual addition (Section 4.1) and of a
concatenation (Algorithm 2).  Exact rationals (``fractions.Fraction``) are used where a
rounding decides an integer; ratios that are only metadata are doubles.

Readings taken where the paper is silent:
  * "[.]" rounds to nearest with ties toward +infinity.
  * ``mul_shift(r)``: the smallest ``shift >= shift_min`` for which
    ``mul = [r * 2^shift]`` reaches ``mul_min`` (2^6, which keeps the single-layer
    configuration at its stated shift of 16); ``shift <= 40``; ``1 <= mul < 2^31``.
    ratio_V is then *defined* by mul / 2^shift (Eq. 11), so a coarse mul costs nothing.
  * Eq. 13's ``h_i = [h_f * ratio_Y]`` with ``h_f = max_int / ratio_V`` (Eq. 12) and
    ``ratio_V = ratio_Y * mul / 2^shift`` (Eq. 11) is ``[max_int * 2^shift / mul]``: ratio_Y
    cancels, so it is evaluated in exact integers.
"""
from fractions import Fraction
import math

import numpy as np

SHIFT_MAX = 40
MUL_MIN = 1 << 6


def round_half_up(x) -> int:
    """[x]: nearest integer, ties toward +infinity.  x is a Fraction, int or float."""
    return math.floor(Fraction(x) + Fraction(1, 2))


def weight_delta(W_f) -> float:
    """Eq. 2: the quantisation step that maps max|W_f| to 127."""
    return float(np.max(np.abs(np.asarray(W_f, dtype=np.float64)))) / 127.0


def quantize_weights(W_f, delta: float):
    """Eq. 1: W_i = [W_f / delta], kept inside [-127, 127] (an adjusted delta may push
    the largest weight past 127; the paper is silent, the value is clipped)."""
    q = np.floor(np.asarray(W_f, dtype=np.float64) / float(delta) + 0.5)
    return np.clip(q, -127, 127).astype(np.int8)


def mul_shift(r, shift_min: int = 16, mul_min: int = MUL_MIN):
    """Integers (mul, shift) with mul / 2^shift ~ r  (the ``mul_shift`` of Eq. 9)."""
    r = Fraction(r)
    if r <= 0:
        raise ValueError("mul_shift needs a positive ratio")
    for shift in range(shift_min, SHIFT_MAX + 1):
        mul = round_half_up(r * (1 << shift))
        if mul >= mul_min:
            break
    if mul < 1 or mul >= (1 << 31):
        raise ValueError("mul_shift: ratio %r not representable" % float(r))
    return int(mul), int(shift)


def brelu_params(h_rf: float, ratio_Y: float, max_int: int, shift_min: int = 16):
    """Section 3.3.  Returns dict(h_ri, mul, shift, ratio_V, h_f, h_i)."""
    # Eq. 8: the bracket is taken of the exact product of the two given numbers (the doubles as
    # they are, multiplied as rationals), not of a product already rounded to a double
    h_ri = max(1, round_half_up(Fraction(float(h_rf)) * Fraction(float(ratio_Y))))
    return brelu_params_from_h_ri(h_ri, ratio_Y, max_int, shift_min)


def brelu_params_from_h_ri(h_ri: int, ratio_Y: float, max_int: int, shift_min: int = 16):
    mul, shift = mul_shift(Fraction(max_int, h_ri), shift_min)                # Eq. 9
    ratio_V = ratio_Y * mul / float(1 << shift)                               # Eq. 11
    h_f = max_int / ratio_V                                                   # Eq. 12
    h_i = round_half_up(Fraction(max_int * (1 << shift), mul))                # Eq. 13
    return dict(h_ri=int(h_ri), mul=mul, shift=shift, ratio_V=ratio_V, h_f=h_f, h_i=int(h_i))


def bn_fold(W_f, b_f, gamma, beta, mean, var, eps: float):
    """Section 3.4.3: a batch-normalisation layer merged into the convolution before it, one
    quantisation step per output channel.  With g = gamma / sqrt(var + eps) (per channel):
    W'[co] = W[co] * g[co], b'[co] = (b[co] - mean[co]) * g[co] + beta[co], delta[co] = max|W'[co]| / 127
    (Eq. 2 channel by channel; 0 for a channel whose weights all vanish, which can be pruned).
    Returns (W', b', delta) in float64; W_f is [c_out][...]."""
    W = np.asarray(W_f, dtype=np.float64)
    c_out = W.shape[0]
    b = np.zeros(c_out) if b_f is None else np.asarray(b_f, dtype=np.float64)
    g = np.asarray(gamma, dtype=np.float64) / np.sqrt(np.asarray(var, dtype=np.float64) + float(eps))
    Wp = W * g.reshape((c_out,) + (1,) * (W.ndim - 1))
    bp = (b - np.asarray(mean, dtype=np.float64)) * g + np.asarray(beta, dtype=np.float64)
    delta = np.max(np.abs(Wp.reshape(c_out, -1)), axis=1) / 127.0
    return Wp, bp, delta


def sigma_bound(Y, fraction: float = 0.0015) -> int:
    """Section 3.2.2, the n-sigma rule: the minimal value among the largest ``fraction`` of the
    feature map Y (0.15 % for three sigma), never below 1 (a BReLU bound is positive)."""
    flat = np.sort(np.asarray(Y).reshape(-1))
    if flat.size == 0:
        return 1
    k = max(1, int(np.ceil(flat.size * fraction)))
    return max(1, int(flat[flat.size - k]))


def requant_exact(Y: int, mul: int, shift: int) -> int:
    """Eq. 4 in exact rational arithmetic (used by tests as the definition of the bracket)."""
    return round_half_up(Fraction(Y * mul, 1 << shift))


def skip_sync(ratio_Y: float, ratio_S: float, shift_min: int = 8):
    """Ratio synchronisation of a residual addition (Section 4.1): rescale the skip
    operand (ratio_S) by mul / 2^shift to come close to ratio_Y, then move the
    convolution's quantisation step so that the two ratios agree exactly.

    Returns dict(skip_mul, skip_shift, ratio_Y_new, delta_scale) with
    ratio_Y_new = ratio_S * skip_mul / 2^skip_shift and delta_new = delta * delta_scale.
    """
    skip_mul, skip_shift = mul_shift(ratio_Y / ratio_S, shift_min)
    ratio_Y_new = ratio_S * skip_mul / float(1 << skip_shift)
    return dict(skip_mul=skip_mul, skip_shift=skip_shift, ratio_Y_new=ratio_Y_new,
                delta_scale=ratio_Y / ratio_Y_new)


def concat_sync(ratio_Y, ratio_V, shift_min: int = 16):
    """Algorithm 2.  ratio_Y, ratio_V: one entry per branch.

    Returns dict(ratio_V_min, mul[], shift[], delta_scale[], ratio_Y_new[]).  The value the
    algorithm assigns to Delta_i is a pure number; it is read as the factor applied to
    the branch's old quantisation step (it equals ratio_Y_old / ratio_Y_new).
    """
    ratio_min = min(ratio_V)
    mul, shift, scale, ry_new = [], [], [], []
    for ry in ratio_Y:
        m, s = mul_shift(ratio_min / ry, shift_min)
        mul.append(m)
        shift.append(s)
        scale.append((ry * m) / (float(1 << s) * ratio_min))
        ry_new.append((ratio_min * float(1 << s)) / m)
    return dict(ratio_V_min=ratio_min, mul=mul, shift=shift, delta_scale=scale, ratio_Y_new=ry_new)


def avgpool_mul_shift(count: int, shift: int = 16):
    """Multiplier of the integer average over ``count`` values: [2^shift / count]."""
    return round_half_up(Fraction(1 << shift, count)), shift
