/*
 * iconv.h -- C ABI of the B200 (sm_100a) integer-arithmetic-only convolution layer.
 *
 * The operations are those of "Efficient Integer-Arithmetic-Only Convolutional Neural
 * Networks" (Zhao, Liu, Li).  One layer (Section 3.1, Figure 1, integer branch):
 *
 *     U_i = X_i (*) W_i            int8 weights x 8-bit activations, int32 accumulation
 *     Y_i = U_i + b_i              int32 bias
 *     Y_i += [S * skip_mul / 2^skip_shift]      residual ratio synchronisation (Section 4.1)
 *     Y_i = min(max(Y_i, 0), h_i)  Bounded ReLU with l = 0 (Eq. 5, Section 3.3)
 *     V_i = [Y_i * mul / 2^shift]  requantisation (Eq. 4)
 *     out = clamp(V_i + out_zero, out_lo, out_hi), stored at a channel offset
 *                                  (concatenation without a copy, Section 4.2.2)
 *
 * "[.]" is round-to-nearest with ties toward +infinity: [v / 2^s] = floor((v + 2^(s-1)) / 2^s).
 *
 * Conventions for every entry point
 *   - Plain C, no exceptions cross the boundary.  Every function returns an iconv_status
 *     (0 = success, negative = error); iconv_last_error() gives the text of the calling
 *     thread's last error.  Nothing falls back to the CPU or to a vendor library.
 *   - "host" / "device" on a pointer says where the memory lives.  Device pointers must be
 *     16-byte aligned unless stated otherwise.
 *   - Activations are NHWC.  A tensor may be a channel slice of a wider tensor: the pixel
 *     stride is *_c_total channels and the slice starts at *_c_offset.
 *   - Weights are [c_out][kh][kw][c_in] int8.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Forward calls only enqueue work on it and return; they never synchronise.
 *   - Devices: a plan belongs to the device that was current when iconv_plan ran (its weights and
 *     constants live there); forwards run on the current device.  The library keeps a small
 *     table per device (shared-memory opt-in of its kernels, SM count, address of the status
 *     word), filled by the first call on each device, so one process may drive several GPUs;
 *     device indices up to 63 are supported.
 */
#ifndef ICONV_H_
#define ICONV_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ICONV_API __attribute__((visibility("default")))
#else
#define ICONV_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ICONV_OK = 0,
    ICONV_ERR_ARG = -1,          /* null pointer, bad enum, negative size */
    ICONV_ERR_SHAPE = -2,        /* empty output, slice outside its tensor */
    ICONV_ERR_ALIGN = -3,        /* pointer or channel offset not aligned as required */
    ICONV_ERR_OVERFLOW = -4,     /* worst-case |Y| could exceed int32 */
    ICONV_ERR_UNSUPPORTED = -5,  /* valid request that no kernel implements */
    ICONV_ERR_CUDA = -6,         /* a CUDA call failed; text in iconv_last_error() */
    ICONV_ERR_TIMEOUT = -7       /* a bounded device-side wait ran out (reported by iconv_check; nothing else maps to it) */
} iconv_status;

typedef enum {
    ICONV_U8 = 0,        /* unsigned 8-bit activation */
    ICONV_S8 = 1,        /* signed 8-bit activation */
    ICONV_I32 = 2,       /* raw int32 Y (projection skips, logits) */
    ICONV_U8_RAW128 = 3  /* raw uint8 image; 128 is subtracted on load (Section 3.4.1).
                            Padding is zero AFTER the subtraction. */
} iconv_dtype;

/* Kernel families; ICONV_KERNEL_AUTO lets the plan choose. */
typedef enum {
    ICONV_KERNEL_AUTO = 0,
    ICONV_KERNEL_DIRECT = 1,   /* CUDA-core direct convolution, any shape */
    ICONV_KERNEL_UMMA = 2,     /* tcgen05.mma kind::i8 implicit GEMM, TMA im2col staging */
    ICONV_KERNEL_THIN = 3,     /* bandwidth-bound layers: c_in <= 4 or c_out == 1 */
    ICONV_KERNEL_STEM = 4,     /* first layers the tensor cores cannot read directly (7x7/2 over a 3-channel
                                  image; stride-1 filters over a single-channel image): a repack of the
                                  image into the caller's workspace (iconv_workspace_bytes), then the
                                  tensor-core kernel on the repacked tensor */
    ICONV_KERNEL_UMMA_IM2COL = 5  /* the tensor-core kernel in its plainest form: im2col staging even where the
                                  plan would load one input patch per tile (stride-1 filters), and single
                                  CTAs even where it would run CTA pairs (long reductions); reported as
                                  ICONV_KERNEL_UMMA by iconv_plan_kernel */
} iconv_kernel;

/*
 * Layer descriptor.  All pointers are HOST pointers; iconv_plan copies what they point
 * to, so the caller may free them after the call.
 */
typedef struct {
    int32_t n, h, w, c_in;             /* input extent (c_in = width of the slice convolved) */
    int32_t c_out, kh, kw, stride, pad;
    int32_t in_dtype, in_c_total, in_c_offset;      /* ICONV_U8 | ICONV_S8 | ICONV_U8_RAW128 */
    int32_t out_dtype, out_c_total, out_c_offset;   /* ICONV_U8 | ICONV_S8 | ICONV_I32 (raw Y) */
    int32_t brelu;                     /* 1: clamp Y to [0, h_i] before Eq. 4 */
    int32_t per_channel;               /* 0: mul/shift/h_i hold 1 entry; 1: c_out entries */
    int32_t out_lo, out_hi, out_zero;  /* final saturation and zero point of the stored value */
    int32_t skip_dtype;                /* -1: none, else an iconv_dtype */
    int32_t skip_c_total, skip_c_offset;
    int32_t skip_mul, skip_shift;      /* Y += [ (S - 128 if RAW128) * skip_mul / 2^skip_shift ] */
    int32_t kernel;                    /* iconv_kernel; AUTO unless a test forces a family */
    /* Fused projection skip (Section 4.1, the skip that is itself a convolution of the block's
     * quantised input): used when proj_weights != NULL.  Then the `skip` tensor of iconv_forward is
     * the projection's INPUT, [n][proj_h][proj_w][proj_c_total] of skip_dtype (U8 or S8), and
     *     S = sum x_p * W_p + proj_bias          (int32, never stored)
     *     Y += [S * skip_mul / 2^skip_shift]
     * exactly as if S had been written as an ICONV_I32 tensor by a separate layer and read back.
     * The projection's output grid must equal this layer's (n, h_out, w_out).  skip_c_total and
     * skip_c_offset are ignored.  Tensor-core kernel only; needs brelu = 1 and an 8-bit output. */
    int32_t proj_h, proj_w, proj_c_in, proj_c_total, proj_c_offset, proj_k, proj_stride, proj_pad;
    const int8_t *weights;             /* host [c_out][kh][kw][c_in] */
    const int32_t *bias;               /* host [c_out] */
    const int32_t *mul;                /* host [1 or c_out], 1 <= mul < 2^31 (ignored for I32 out) */
    const int32_t *shift;              /* host [1 or c_out], 0 <= shift <= 40 */
    const int32_t *h_i;                /* host [1 or c_out], 0 <= h_i (ignored unless brelu) */
    const int8_t *proj_weights;        /* host [c_out][proj_k][proj_k][proj_c_in], or NULL */
    const int32_t *proj_bias;          /* host [c_out] (with proj_weights) */
} iconv_desc;

typedef struct iconv_plan_s iconv_plan_t;

/*
 * iconv_plan -- validate a layer, choose its kernel, upload its parameters (Section 3.1's
 * W_i, b_i; Eq. 4's mul, shift; Section 3.3's h_i) and build its TMA descriptors.
 * Allocates device memory with cudaMalloc on the current device for those parameters only (a plan
 * owns no activation-sized memory); call it outside any stream capture.  Rejects layers whose worst-case |Y| (c_in*kh*kw * 255 * 127 + |b| +
 * skip bound) reaches 2^31 with ICONV_ERR_OVERFLOW.  *plan_out is owned by the caller
 * and released with iconv_plan_destroy.
 */
ICONV_API int iconv_plan(const iconv_desc *desc, iconv_plan_t **plan_out);
ICONV_API int iconv_plan_destroy(iconv_plan_t *plan);

/* Which kernel family the plan selected (an iconv_kernel), or a negative status. */
ICONV_API int iconv_plan_kernel(const iconv_plan_t *plan);

/* One line of text on what the plan decided (kernel family, tile and pipeline geometry, epilogue
 * variant), for logs and tests: at most `size` bytes including the terminating zero are written
 * to the HOST buffer `text`. */
ICONV_API int iconv_plan_describe(const iconv_plan_t *plan, char *text, size_t size);

/*
 * iconv_workspace_bytes -- bytes of caller-owned device scratch one forward of this plan needs
 * (Section 3.1's layer takes X_i, W_i, b_i; the scratch only holds a rearranged copy of X_i for the
 * first layers of kernel family ICONV_KERNEL_STEM: 16 bytes per repacked position).  0 for every
 * other plan and for a NULL plan.  The size depends on the plan alone, so one buffer of the
 * largest size over a network's plans serves all of them in turn.
 */
ICONV_API size_t iconv_workspace_bytes(const iconv_plan_t *plan);

/*
 * iconv_forward -- one layer forward (Section 3.1 / Eq. 4 / Eq. 5 as listed at the top).
 * x, skip, out: DEVICE pointers owned by the caller.  x holds n*h*w*in_c_total elements
 * of in_dtype; out holds n*h_out*w_out*out_c_total elements of out_dtype, of which only
 * the slice [out_c_offset, out_c_offset + c_out) of each pixel is written; skip (NULL when
 * skip_dtype < 0) holds n*h_out*w_out*skip_c_total elements (or, with a fused projection, the
 * projection's input: n*proj_h*proj_w*proj_c_total elements).  workspace: DEVICE, 16-byte aligned,
 * at least iconv_workspace_bytes(plan) bytes, owned by the caller, contents undefined before and
 * after the call (NULL when that size is 0; ICONV_ERR_ARG when it is missing).  Asynchronous on
 * cuda_stream.  The plan is not modified and holds no per-call state: concurrent forwards of one
 * plan on different streams are allowed as long as each has its own workspace (and output).
 */
ICONV_API int iconv_forward(const iconv_plan_t *plan, const void *x, const void *skip, void *out,
                  void *workspace, void *cuda_stream);

/*
 * Two consecutive layers in one kernel (Section 3.1: the output V_i of a layer is the input of the
 * next; Section 4.1 for the first layer's skip): `first` is a block-closing 1x1 convolution with an
 * 8-bit skip, `second` the 1x1 convolution that reads exactly first's output slice.  The first
 * layer's output tile is staged in shared memory on its way to HBM and serves from there as the
 * second layer's operand, so the wide tensor is written once and the second layer never reads it
 * back.  Both outputs are bit-identical to iconv_forward of the two layers one after the other.
 * Taken: both 1x1, stride 1, unpadded, the same pixel grid; 8-bit unsigned activations; first.c_in
 * 64 or 128, first.c_out a multiple of 128 up to 512, second.c_out 64 or 128; per-layer mul / shift
 * / h_i whose clamp-free 32-bit epilogue forms the plan can prove (BReLU on, u8 saturation,
 * skip_shift = 8); both filter banks resident in shared memory.  Anything else returns
 * ICONV_ERR_UNSUPPORTED with the reason in iconv_last_error(): run the layers apart.
 * iconv_plan_chain copies what the descriptors point to (host pointers, as iconv_plan) and
 * allocates the two layers' parameters with cudaMalloc.  iconv_forward_chain: x, skip, out as in
 * iconv_forward of `first`; out2 DEVICE, the second layer's output tensor (n*h*w*second.out_c_total
 * bytes, slice [out_c_offset, +c_out) written); all 16-byte aligned; asynchronous on cuda_stream;
 * no workspace.
 */
typedef struct iconv_chain_s iconv_chain_t;
ICONV_API int iconv_plan_chain(const iconv_desc *first, const iconv_desc *second, iconv_chain_t **chain_out);
ICONV_API int iconv_chain_destroy(iconv_chain_t *chain);
ICONV_API int iconv_forward_chain(const iconv_chain_t *chain, const void *x, const void *skip, void *out, void *out2,
                        void *cuda_stream);

/*
 * Device-side waits (mbarrier phases) are bounded.  A kernel whose wait runs out records
 * a code (1-7) in a per-device status word and returns early.  iconv_check synchronises the
 * stream, reads and clears the word of the current device and returns ICONV_ERR_TIMEOUT if a
 * kernel recorded such a code since the last call, ICONV_ERR_ARG for code 8 (a bias that
 * iconv_stem_forward_static found out of range on the device), ICONV_ERR_CUDA on a CUDA error,
 * ICONV_OK otherwise.
 */
ICONV_API int iconv_check(void *cuda_stream);

/*
 * Test hooks (the paper has no counterpart).
 * iconv_selftest_wait_timeout enqueues one tiny kernel (one CTA) that waits, with the very wait
 * routine of the convolution kernels, on a barrier that nothing ever arrives at, with a limit of
 * `limit_cycles` SM cycles (1e3 .. 2e8) instead of the kernels' two seconds; which = 0 the wait of
 * a single-thread role, 1 the wait of an epilogue warp.  The wait gives up, records code 7 and the
 * kernel returns, so the next iconv_check reports ICONV_ERR_TIMEOUT once and the context stays
 * usable.  iconv_device_initialised returns the SM count recorded for `device` once a
 * tensor-core plan or launch initialised that device's table, else -1.
 */
ICONV_API int iconv_selftest_wait_timeout(int32_t which, int64_t limit_cycles, void *cuda_stream);
ICONV_API int iconv_device_initialised(int32_t device);

/* Feature-map addition with ratio synchronisation as a stand-alone step (Sections 3.4.2,
 * 4.1):  Y = [(A - a_zero) * mul_a / 2^sh_a] + [(B - b_zero) * mul_b / 2^sh_b], then the
 * same BReLU / Eq. 4 / zero point / saturation tail as a convolution output. */
typedef struct {
    int64_t n_elems;
    int32_t a_dtype, b_dtype, out_dtype;     /* ICONV_U8 | ICONV_S8 | ICONV_I32 */
    int32_t a_zero, b_zero;
    int32_t mul_a, sh_a, mul_b, sh_b;        /* (1, 0) for an operand already at the target ratio */
    int32_t brelu, h_i, mul, shift, out_zero, out_lo, out_hi;
} iadd_desc;

/* a, b, out: DEVICE pointers to n_elems contiguous elements.  Asynchronous. */
ICONV_API int iadd_requant(const iadd_desc *desc, const void *a, const void *b, void *out, void *cuda_stream);

/* ResNet glue (Section 4.1 only says that pooling layers exist; a maximum needs no
 * rescaling, the average is an integer sum followed by Eq. 4 with mul ~ 2^shift / (h*w)).
 * x, out: DEVICE, uint8 NHWC, contiguous.  c must be a multiple of 16 for ipool_max. */
ICONV_API int ipool_max(const void *x, void *out, int32_t n, int32_t h, int32_t w, int32_t c,
              int32_t k, int32_t stride, int32_t pad, void *cuda_stream);
ICONV_API int ipool_avg_requant(const void *x, void *out, int32_t n, int32_t h, int32_t w, int32_t c,
                      int32_t mul, int32_t shift, int32_t max_int, void *cuda_stream);

/*
 * iconv_stem_forward_static -- the 7x7 stride-2 pad-3 first layer over a 3-channel image, for
 * callers that may not allocate device memory.  (The paper has no counterpart; this exists for
 * the way the library is embedded.)  Code that runs under a framework's memory pool, inside a
 * latency-critical serving loop or in a process whose device memory is fully budgeted up front
 * cannot call cudaMalloc, yet iconv_plan does (weights, constants and, for this layer, a
 * repacked copy of the image).  This entry point needs no plan and calls no cudaMalloc, cudaFree
 * or allocating library routine: its working memory -- the repacked image, the rearranged
 * weights and the epilogue constants -- is a fixed array of ICONV_STEM_STATIC_BYTES inside the
 * library's device image, which every GPU that loads the library holds until the process exits.
 *
 *   x        DEVICE uint8 (or int8) [n][h][w][3], 16-byte aligned
 *   weights  DEVICE int8 [c_out][7][7][3]
 *   bias     DEVICE int32 [c_out], |b| <= 2^30 (a larger one is replaced by 0 and recorded in the
 *            device status word as code 8, which the next iconv_check reports as ICONV_ERR_ARG)
 *   out      DEVICE uint8 [n][h_out][w_out][out_c_total], 16-byte aligned; only the slice
 *            [out_c_offset, out_c_offset + c_out) of each pixel is written
 *
 * The arithmetic is iconv_forward's with brelu = 1 and per-layer mul / shift / h_i; results are
 * bit-identical to a planned forward of the same layer.  Returns ICONV_ERR_SHAPE with the sizes in
 * iconv_last_error() when n * (h_out + 3) * (w_out + 3) * 16 + 196608 exceeds ICONV_STEM_STATIC_BYTES
 * (157 images of 224 x 224 fit), ICONV_ERR_ARG unless c_out is a multiple of 16 in [16, 256],
 * 1 <= shift <= 31 and h_i * mul + 2^(shift-1) < 2^32, ICONV_ERR_UNSUPPORTED (before anything is
 * enqueued) when a TMA descriptor of the repacked layer cannot be encoded.  Asynchronous on cuda_stream.
 *
 * The first call on each device looks up the array's device address (the GPU with that array
 * must be current); make that first call outside any stream capture.  All calls on a device share
 * the one array, which keeps whatever the last call left in it; each call rewrites every byte it
 * later reads, so nothing has to be cleared, but two calls that overlap on the GPU (different
 * streams, or different host threads) race on it: serialise them.
 */
#define ICONV_STEM_STATIC_BYTES (32u * 1024u * 1024u)
typedef struct {
    int32_t n, h, w, c_out;
    int32_t in_dtype;                  /* ICONV_U8 | ICONV_S8 | ICONV_U8_RAW128 */
    int32_t out_c_total, out_c_offset;
    int32_t mul, shift, h_i;           /* Eq. 4 and the BReLU bound, one value for the layer */
    int32_t out_lo, out_hi, out_zero;
} istem_desc;
ICONV_API int iconv_stem_forward_static(const istem_desc *desc, const void *x, const int8_t *weights, const int32_t *bias,
                              void *out, void *cuda_stream);

/* ---- host-side parameter arithmetic (no GPU involved) ------------------------------- */

/* Eq. 2: delta = max|W_f| / 127. */
ICONV_API int iq_weight_delta(const float *w_f, int64_t count, double *delta);
/* Section 3.4.3: a batch-normalisation layer merged into the convolution before it, with one
 * quantisation step per output channel.  g = gamma / sqrt(var + eps); w_out[co][i] = w_f[co][i] * g[co];
 * b_out[co] = (b_f[co] - mean[co]) * g[co] + beta[co] (b_f may be NULL: no bias);
 * delta[co] = max_i |w_out[co][i]| / 127 (Eq. 2 per channel; 0 when the channel's weights all
 * vanish: such a channel can be pruned).  Everything in double.  All pointers HOST; w_f is
 * [c_out][k], the per-channel arrays have c_out entries; w_out [c_out][k], b_out and delta [c_out]
 * are written.  The per-channel steps give per-channel ratios, which `iconcat_plan` (Algorithm 2,
 * one branch per channel) brings to a common output ratio: its mul / shift arrays are the
 * per-channel parameters `iconv_plan` accepts.  Errors: ICONV_ERR_ARG (null pointer, c_out < 1,
 * k < 1, var + eps <= 0). */
ICONV_API int iq_bn_fold(const float *w_f, const float *b_f, const float *gamma, const float *beta, const float *mean,
               const float *var, double eps, int32_t c_out, int64_t k, double *w_out, double *b_out, double *delta);
/* Eq. 1: w_i = clamp([w_f / delta], -127, 127), computed in double. */
ICONV_API int iq_quantize_weights(const float *w_f, int64_t count, double delta, int8_t *w_i);
/* The mul_shift() named by Eq. 9: the smallest shift in [shift_min, 40] whose
 * mul = [r * 2^shift] reaches 2^6; fails with ICONV_ERR_ARG unless 1 <= mul < 2^31. */
ICONV_API int iq_mul_shift(double r, int32_t shift_min, int32_t *mul, int32_t *shift);
/* Section 3.3, Eq. 7-13: from h_rf and ratio_Y to mul, shift, h_i (and h_f, ratio_V). */
ICONV_API int iq_brelu_params(double h_rf, double ratio_y, int32_t max_int, int32_t shift_min,
                    int32_t *h_ri, int32_t *mul, int32_t *shift, int32_t *h_i,
                    double *h_f, double *ratio_v);
/* Section 4.1: rescale of a skip operand of ratio_s toward ratio_y, and the factor by
 * which the convolution's quantisation step moves so that both ratios agree exactly. */
ICONV_API int iq_skip_sync(double ratio_y, double ratio_s, int32_t shift_min,
                 int32_t *skip_mul, int32_t *skip_shift, double *ratio_y_new, double *delta_scale);
/* Algorithm 2: ratio synchronisation of n_branches concatenated feature maps.  Outputs are
 * host arrays of n_branches entries; *ratio_v_min receives the common ratio. */
ICONV_API int iconcat_plan(int32_t n_branches, const double *ratio_y, const double *ratio_v,
                 int32_t shift_min, int32_t *mul, int32_t *shift,
                 double *delta_scale, double *ratio_y_new, double *ratio_v_min);

/* Section 3.2.2, the n-sigma rule on the GPU: the smallest value among the largest `fraction`
 * of an int32 feature map Y (its k-th largest element, k = max(1, ceil(count * fraction)); 0.0015
 * for 3 sigma), never below 1.  This is the h_ri that Eq. 9-13 (`iq_brelu_params`' arithmetic)
 * turn into mul, shift and h_i; the paper averages it over batches, which is the caller's job.
 * y: DEVICE pointer to `count` int32 values, 4-byte aligned, read only; bound: HOST.  Exact
 * (a four-pass radix select, no sorting, no approximation).  Enqueues on `cuda_stream` and
 * waits for the result; keeps a 2 KB scratch per device, allocated at the first call.
 * Errors: ICONV_ERR_ARG (null pointer, fraction outside (0, 1]), ICONV_ERR_ALIGN, ICONV_ERR_CUDA.
 * count = 0 returns 1. */
ICONV_API int iq_sigma_bound(const int32_t *y, int64_t count, double fraction, int32_t *bound, void *cuda_stream);

/* Text of the calling thread's last error (never NULL; valid until its next failing call). */
ICONV_API const char *iconv_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ICONV_H_ */
