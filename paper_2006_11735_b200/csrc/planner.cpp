// Host-side parameter arithmetic of the integer network: weight quantisation (Eq. 1-2),
// mul_shift (named by Eq. 9), the quantised BReLU parameters (Section 3.3, Eq. 7-13),
// residual ratio synchronisation (Section 4.1) and Algorithm 2 for concatenations.
// Integers are decided in exact integer arithmetic or on exactly representable doubles.
#include <cmath>
#include <cstdint>

#include "iconv.h"

namespace iconv {
void set_error(const char *fmt, ...);
}
using iconv::set_error;

namespace {

const int kShiftMax = 40;
const int64_t kMulMin = 1 << 6;

// nearest integer, ties toward +infinity, of a finite double (exact: no x + 0.5 rounding)
double round_half_up(double x)
{
    const double f = std::floor(x);
    return (x - f >= 0.5) ? f + 1.0 : f;
}

// nearest integer, ties toward +infinity, of num / den (den > 0, num >= 0)
int64_t div_round_half_up(int64_t num, int64_t den) { return (2 * num + den) / (2 * den); }

}  // namespace

extern "C" int iq_weight_delta(const float *w_f, int64_t count, double *delta)
{
    if (!w_f || !delta || count < 1) { set_error("iq_weight_delta: bad argument"); return ICONV_ERR_ARG; }
    double m = 0.0;
    for (int64_t i = 0; i < count; ++i) {
        const double a = std::fabs((double)w_f[i]);
        if (a > m) m = a;
    }
    *delta = m / 127.0;
    return ICONV_OK;
}

extern "C" int iq_bn_fold(const float *w_f, const float *b_f, const float *gamma, const float *beta, const float *mean,
                          const float *var, double eps, int32_t c_out, int64_t k, double *w_out, double *b_out, double *delta)
{
    if (!w_f || !gamma || !beta || !mean || !var || !w_out || !b_out || !delta || c_out < 1 || k < 1 || !(eps >= 0.0)) {
        set_error("iq_bn_fold: bad argument");
        return ICONV_ERR_ARG;
    }
    for (int32_t co = 0; co < c_out; ++co) {
        const double s = (double)var[co] + eps;
        if (!(s > 0.0)) { set_error("iq_bn_fold: var + eps must be positive (channel %d)", (int)co); return ICONV_ERR_ARG; }
        const double g = (double)gamma[co] / std::sqrt(s);
        double m = 0.0;
        for (int64_t i = 0; i < k; ++i) {
            const double w = (double)w_f[(int64_t)co * k + i] * g;
            w_out[(int64_t)co * k + i] = w;
            const double a = std::fabs(w);
            if (a > m) m = a;
        }
        b_out[co] = ((b_f ? (double)b_f[co] : 0.0) - (double)mean[co]) * g + (double)beta[co];
        delta[co] = m / 127.0;
    }
    return ICONV_OK;
}

extern "C" int iq_quantize_weights(const float *w_f, int64_t count, double delta, int8_t *w_i)
{
    if (!w_f || !w_i || count < 0 || !(delta > 0.0)) { set_error("iq_quantize_weights: bad argument"); return ICONV_ERR_ARG; }
    for (int64_t i = 0; i < count; ++i) {
        double q = std::floor((double)w_f[i] / delta + 0.5);
        if (q < -127.0) q = -127.0;
        if (q > 127.0) q = 127.0;
        w_i[i] = (int8_t)q;
    }
    return ICONV_OK;
}

extern "C" int iq_mul_shift(double r, int32_t shift_min, int32_t *mul, int32_t *shift)
{
    if (!mul || !shift || !(r > 0.0) || !std::isfinite(r) || shift_min < 0 || shift_min > kShiftMax) {
        set_error("iq_mul_shift: needs a positive finite ratio and 0 <= shift_min <= %d", kShiftMax);
        return ICONV_ERR_ARG;
    }
    double m = 0.0;
    int s = shift_min;
    for (;; ++s) {
        m = round_half_up(std::ldexp(r, s));
        if (m >= (double)kMulMin || s == kShiftMax) break;
    }
    if (m < 1.0 || m >= 2147483648.0) {
        set_error("iq_mul_shift: ratio %g not representable as mul / 2^shift with 1 <= mul < 2^31", r);
        return ICONV_ERR_ARG;
    }
    *mul = (int32_t)m;
    *shift = s;
    return ICONV_OK;
}

// mul_shift for the exact rational max_int / h_ri
static int mul_shift_ratio(int64_t num, int64_t den, int shift_min, int64_t *mul, int *shift)
{
    int64_t m = 0;
    int s = shift_min;
    for (;; ++s) {
        m = div_round_half_up(num << s, den);
        if (m >= kMulMin || s == kShiftMax) break;
    }
    if (m < 1 || m >= (1ll << 31)) return ICONV_ERR_ARG;
    *mul = m;
    *shift = s;
    return ICONV_OK;
}

extern "C" int iq_brelu_params(double h_rf, double ratio_y, int32_t max_int, int32_t shift_min, int32_t *h_ri,
                               int32_t *mul, int32_t *shift, int32_t *h_i, double *h_f, double *ratio_v)
{
    if (!h_ri || !mul || !shift || !h_i || !(h_rf > 0.0) || !(ratio_y > 0.0) || max_int < 1 || max_int > 65535 ||
        shift_min < 0 || shift_min > kShiftMax) {
        set_error("iq_brelu_params: bad argument");
        return ICONV_ERR_ARG;
    }
    // Eq. 8: [h_rf * ratio_Y] of the EXACT product.  p is the product rounded to a double and
    // e = h_rf * ratio_Y - p exactly (one fused multiply-add), so the product is p + e with
    // |e| <= ulp(p) / 2: only when p sits exactly on a tie (fraction 0.5) can e move the bracket,
    // and then its sign decides (ties go up, so e >= 0 rounds up and e < 0 rounds down).
    const double prod = h_rf * ratio_y;
    if (!(prod < 2147483648.0)) { set_error("iq_brelu_params: h_ri does not fit int32"); return ICONV_ERR_OVERFLOW; }
    const double err = std::fma(h_rf, ratio_y, -prod);
    const double fl = std::floor(prod), frac = prod - fl;
    double hr = (frac > 0.5 || (frac == 0.5 && err >= 0.0)) ? fl + 1.0 : fl;
    if (hr < 1.0) hr = 1.0;
    if (hr >= 2147483648.0) { set_error("iq_brelu_params: h_ri does not fit int32"); return ICONV_ERR_OVERFLOW; }
    const int64_t hri = (int64_t)hr;
    int64_t m;
    int s;
    if (mul_shift_ratio(max_int, hri, shift_min, &m, &s) != ICONV_OK) {   // Eq. 9
        set_error("iq_brelu_params: max_int / h_ri not representable");
        return ICONV_ERR_ARG;
    }
    const int64_t hi = div_round_half_up((int64_t)max_int << s, m);  // Eq. 11-13: ratio_Y cancels
    if (hi >= (1ll << 31)) { set_error("iq_brelu_params: h_i does not fit int32"); return ICONV_ERR_OVERFLOW; }
    *h_ri = (int32_t)hri;
    *mul = (int32_t)m;
    *shift = s;
    *h_i = (int32_t)hi;
    const double rv = ratio_y * (double)m / std::ldexp(1.0, s);      // Eq. 11
    if (ratio_v) *ratio_v = rv;
    if (h_f) *h_f = (double)max_int / rv;                            // Eq. 12
    return ICONV_OK;
}

extern "C" int iq_skip_sync(double ratio_y, double ratio_s, int32_t shift_min, int32_t *skip_mul,
                            int32_t *skip_shift, double *ratio_y_new, double *delta_scale)
{
    if (!skip_mul || !skip_shift || !(ratio_y > 0.0) || !(ratio_s > 0.0)) {
        set_error("iq_skip_sync: bad argument");
        return ICONV_ERR_ARG;
    }
    const int rc = iq_mul_shift(ratio_y / ratio_s, shift_min, skip_mul, skip_shift);
    if (rc != ICONV_OK) return rc;
    const double ry = ratio_s * (double)*skip_mul / std::ldexp(1.0, *skip_shift);
    if (ratio_y_new) *ratio_y_new = ry;
    if (delta_scale) *delta_scale = ratio_y / ry;
    return ICONV_OK;
}

extern "C" int iconcat_plan(int32_t n_branches, const double *ratio_y, const double *ratio_v, int32_t shift_min,
                            int32_t *mul, int32_t *shift, double *delta_scale, double *ratio_y_new,
                            double *ratio_v_min)
{
    if (n_branches < 1 || !ratio_y || !ratio_v || !mul || !shift) {
        set_error("iconcat_plan: bad argument");
        return ICONV_ERR_ARG;
    }
    double rmin = ratio_v[0];
    for (int i = 0; i < n_branches; ++i) {
        if (!(ratio_v[i] > 0.0) || !(ratio_y[i] > 0.0)) { set_error("iconcat_plan: ratios must be positive"); return ICONV_ERR_ARG; }
        if (ratio_v[i] < rmin) rmin = ratio_v[i];
    }
    for (int i = 0; i < n_branches; ++i) {
        const int rc = iq_mul_shift(rmin / ratio_y[i], shift_min, &mul[i], &shift[i]);
        if (rc != ICONV_OK) return rc;
        const double p2 = std::ldexp(1.0, shift[i]);
        if (delta_scale) delta_scale[i] = (ratio_y[i] * (double)mul[i]) / (p2 * rmin);
        if (ratio_y_new) ratio_y_new[i] = (rmin * p2) / (double)mul[i];
    }
    if (ratio_v_min) *ratio_v_min = rmin;
    return ICONV_OK;
}
