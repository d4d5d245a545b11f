/*
 * TEST INFRASTRUCTURE -- not part of the product.
 *
 * Plain CPU oracle for the integer-arithmetic-only convolution layer of
 * "Efficient Integer-Arithmetic-Only Convolutional Neural Networks" (Zhao, Liu, Li).
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 * It shares no code, header, table or helper with the CUDA path.
 *
 * Everything is computed in int64_t with a direct loop nest that follows the
 * paper's layer statement (Section 3.1, Figure 1 caption) in its own order:
 *
 *     U_i = X_i (*) W_i          integer convolution (cross-correlation, zero padding)
 *     Y_i = U_i + b_i            int32 bias
 *     Y_i += rescaled skip       ratio synchronisation of a residual (Sections 3.4.2, 4.1)
 *     Y_i = BReLU(Y_i)           Eq. 5 with l = 0 and h = h_i
 *     V_i = [Y_i * mul / 2^shift]   Eq. 4
 *
 * "[.]" is read as round-to-nearest with ties toward +infinity (add half, floor).
 * No blocking, no im2col, no intrinsics; OpenMP spreads (image, output row) pairs
 * over the host cores and nothing else.
 *
 * Layouts: activations NHWC with a pixel stride of c_total channels and a channel
 * offset (so a layer can read or write a slice of a concatenated tensor, Section
 * 4.2.2); weights [c_out][kh][kw][c_in].
 */
#include <stdint.h>
#include <stddef.h>

enum { ORC_U8 = 0, ORC_S8 = 1, ORC_I32 = 2, ORC_U8_RAW128 = 3 };

typedef struct {
    int64_t n, h, w, c_in;          /* input tensor extent (the slice that is convolved) */
    int64_t c_out, kh, kw, stride, pad;
    int64_t in_dtype, in_c_total, in_c_offset;
    int64_t out_dtype, out_c_total, out_c_offset;
    int64_t brelu;                   /* 1: clamp Y to [0, h_i] before Eq. 4 */
    int64_t per_channel;             /* 0: mul/shift/h_i hold one entry; 1: c_out entries */
    int64_t out_lo, out_hi, out_zero;
    int64_t skip_dtype;              /* -1: no skip */
    int64_t skip_c_total, skip_c_offset, skip_mul, skip_shift;
    int64_t check_partial;           /* 1: also bound every partial sum (sum of |x*w|) */
} orc_conv_desc;

/* floor(a / b) for b > 0, written out so that no shift of a negative value is relied on */
static int64_t floor_div(int64_t a, int64_t b)
{
    int64_t q = a / b;
    int64_t r = a % b;
    if (r != 0 && r < 0) q -= 1;
    return q;
}

/* [v / 2^s] with ties toward +infinity (Eq. 4's bracket) */
int64_t orc_round_shift(int64_t v, int64_t s)
{
    if (s == 0) return v;
    int64_t half = (int64_t)1 << (s - 1);
    int64_t den = (int64_t)1 << s;
    return floor_div(v + half, den);
}

/* value of element idx of a tensor of the given storage type, in the integer domain
 * the arithmetic uses (raw uint8 images are re-normalised by subtracting 128, Section 3.4.1) */
static int64_t load_value(const void *p, int64_t idx, int64_t dtype)
{
    switch (dtype) {
    case ORC_U8:        return (int64_t)((const uint8_t *)p)[idx];
    case ORC_S8:        return (int64_t)((const int8_t *)p)[idx];
    case ORC_I32:       return (int64_t)((const int32_t *)p)[idx];
    case ORC_U8_RAW128: return (int64_t)((const uint8_t *)p)[idx] - 128;
    default:            return 0;
    }
}

static void store_value(void *p, int64_t idx, int64_t dtype, int64_t v)
{
    switch (dtype) {
    case ORC_U8:  ((uint8_t *)p)[idx] = (uint8_t)v; break;
    case ORC_S8:  ((int8_t *)p)[idx] = (int8_t)v; break;
    case ORC_I32: ((int32_t *)p)[idx] = (int32_t)v; break;
    default: break;
    }
}

static int64_t iabs64(int64_t v) { return v < 0 ? -v : v; }

/* BReLU (Eq. 5, l = 0), Eq. 4, output zero point and the final saturation */
static int64_t requant_tail(int64_t Y, int64_t brelu, int64_t h_i, int64_t mul, int64_t shift,
                            int64_t out_zero, int64_t out_lo, int64_t out_hi)
{
    if (brelu) {
        if (Y < 0) Y = 0;
        if (Y > h_i) Y = h_i;
    }
    int64_t V = orc_round_shift(Y * mul, shift) + out_zero;
    if (V < out_lo) V = out_lo;
    if (V > out_hi) V = out_hi;
    return V;
}

/*
 * One integer convolution layer.  Returns 0, or 1 when some Y (or U, or -- with
 * check_partial -- some bound on the partial sums) does not fit int32, or 2 on a bad
 * descriptor.  The output is still written in full in case 1.
 */
int orc_conv(const orc_conv_desc *d, const void *X, const int8_t *W, const int32_t *b,
             const int32_t *mul, const int32_t *shift, const int32_t *h_i,
             const void *S, void *out)
{
    if (d->stride < 1 || d->kh < 1 || d->kw < 1 || d->pad < 0) return 2;
    const int64_t h_out = (d->h + 2 * d->pad - d->kh) / d->stride + 1;
    const int64_t w_out = (d->w + 2 * d->pad - d->kw) / d->stride + 1;
    if (h_out < 1 || w_out < 1) return 2;
    const int64_t lim = (int64_t)1 << 31;
    int overflow = 0;

#pragma omp parallel for collapse(2) schedule(static) reduction(| : overflow)
    for (int64_t n = 0; n < d->n; ++n) {
        for (int64_t oh = 0; oh < h_out; ++oh) {
            for (int64_t ow = 0; ow < w_out; ++ow) {
                for (int64_t co = 0; co < d->c_out; ++co) {
                    int64_t U = 0, U_abs = 0;
                    for (int64_t r = 0; r < d->kh; ++r) {
                        const int64_t ih = oh * d->stride - d->pad + r;
                        if (ih < 0 || ih >= d->h) continue;       /* zero padding */
                        for (int64_t s = 0; s < d->kw; ++s) {
                            const int64_t iw = ow * d->stride - d->pad + s;
                            if (iw < 0 || iw >= d->w) continue;   /* zero padding */
                            const int64_t xb = ((n * d->h + ih) * d->w + iw) * d->in_c_total + d->in_c_offset;
                            const int64_t wb = ((co * d->kh + r) * d->kw + s) * d->c_in;
                            for (int64_t ci = 0; ci < d->c_in; ++ci) {
                                const int64_t p = load_value(X, xb + ci, d->in_dtype) * (int64_t)W[wb + ci];
                                U += p;
                                if (d->check_partial) U_abs += iabs64(p);
                            }
                        }
                    }
                    int64_t Y = U + (int64_t)b[co];
                    int64_t bound = U_abs + iabs64((int64_t)b[co]);
                    const int64_t pix = (n * h_out + oh) * w_out + ow;
                    if (d->skip_dtype >= 0) {
                        const int64_t sv = load_value(S, pix * d->skip_c_total + d->skip_c_offset + co, d->skip_dtype);
                        const int64_t add = orc_round_shift(sv * d->skip_mul, d->skip_shift);
                        Y += add;
                        bound += iabs64(add);
                    }
                    if (iabs64(U) >= lim || iabs64(Y) >= lim) overflow |= 1;
                    if (d->check_partial && bound >= lim) overflow |= 1;
                    const int64_t oi = pix * d->out_c_total + d->out_c_offset + co;
                    if (d->out_dtype == ORC_I32) {
                        store_value(out, oi, ORC_I32, Y);
                    } else {
                        const int64_t q = d->per_channel ? co : 0;
                        const int64_t V = requant_tail(Y, d->brelu, h_i[q], mul[q], shift[q],
                                                       d->out_zero, d->out_lo, d->out_hi);
                        store_value(out, oi, d->out_dtype, V);
                    }
                }
            }
        }
    }
    return overflow;
}

typedef struct {
    int64_t n_elems;
    int64_t a_dtype, b_dtype, out_dtype, a_zero, b_zero;
    int64_t mul_a, sh_a, mul_b, sh_b;
    int64_t brelu, h_i, mul, shift, out_zero, out_lo, out_hi;
} orc_add_desc;

/*
 * Stand-alone feature-map addition with ratio synchronisation (Sections 3.4.2 and 4.1):
 * each operand is brought to the common ratio by multiplication and right shift, the
 * sum takes the same BReLU / Eq. 4 tail as a convolution output.
 */
int orc_add_requant(const orc_add_desc *d, const void *A, const void *B, void *out)
{
    const int64_t lim = (int64_t)1 << 31;
    int overflow = 0;
#pragma omp parallel for schedule(static) reduction(| : overflow)
    for (int64_t i = 0; i < d->n_elems; ++i) {
        const int64_t a = load_value(A, i, d->a_dtype) - d->a_zero;
        const int64_t bb = load_value(B, i, d->b_dtype) - d->b_zero;
        const int64_t Y = orc_round_shift(a * d->mul_a, d->sh_a) + orc_round_shift(bb * d->mul_b, d->sh_b);
        if (iabs64(Y) >= lim) overflow |= 1;
        const int64_t V = requant_tail(Y, d->brelu, d->h_i, d->mul, d->shift, d->out_zero, d->out_lo, d->out_hi);
        store_value(out, i, d->out_dtype, V);
    }
    return overflow;
}

/* k x k / stride max-pool over the taps that fall inside the image (uint8, NHWC).
 * The paper only says that its ResNets contain pooling layers (Section 4.1); a maximum
 * of integers needs no rescaling, so the ratio of the tensor is unchanged. */
int orc_maxpool(const uint8_t *X, int64_t n, int64_t h, int64_t w, int64_t c,
                int64_t k, int64_t stride, int64_t pad, uint8_t *out)
{
    const int64_t h_out = (h + 2 * pad - k) / stride + 1;
    const int64_t w_out = (w + 2 * pad - k) / stride + 1;
    if (h_out < 1 || w_out < 1) return 2;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t in = 0; in < n; ++in)
        for (int64_t oh = 0; oh < h_out; ++oh)
            for (int64_t ow = 0; ow < w_out; ++ow)
                for (int64_t ch = 0; ch < c; ++ch) {
                    int64_t best = -1;
                    for (int64_t r = 0; r < k; ++r)
                        for (int64_t s = 0; s < k; ++s) {
                            const int64_t ih = oh * stride - pad + r, iw = ow * stride - pad + s;
                            if (ih < 0 || ih >= h || iw < 0 || iw >= w) continue;
                            const int64_t v = X[((in * h + ih) * w + iw) * c + ch];
                            if (v > best) best = v;
                        }
                    out[((in * h_out + oh) * w_out + ow) * c + ch] = (uint8_t)(best < 0 ? 0 : best);
                }
    return 0;
}

/* Global average over h x w as an integer sum followed by Eq. 4's multiply / shift /
 * round with mul ~ 2^shift / (h*w); result clamped to [0, max_int]. */
int orc_avgpool_requant(const uint8_t *X, int64_t n, int64_t h, int64_t w, int64_t c,
                        int64_t mul, int64_t shift, int64_t max_int, uint8_t *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t in = 0; in < n; ++in)
        for (int64_t ch = 0; ch < c; ++ch) {
            int64_t sum = 0;
            for (int64_t i = 0; i < h * w; ++i) sum += X[(in * h * w + i) * c + ch];
            int64_t V = orc_round_shift(sum * mul, shift);
            if (V < 0) V = 0;
            if (V > max_int) V = max_int;
            out[in * c + ch] = (uint8_t)V;
        }
    return 0;
}
