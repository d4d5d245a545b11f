// C-ABI entry points: validation, plans, dispatch.  No arithmetic of the layer lives here.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "plan.h"

namespace iconv {

static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

int cuda_fail(cudaError_t e, const char *what)
{
    set_error("CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
    return ICONV_ERR_CUDA;
}

// status word written by kernels whose bounded waits run out
__device__ int g_device_status = 0;

// Index of the current device in the library's per-device tables, or -1.
int current_device_slot()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return -1;
    return dev;
}

// Device address of the status word on the current device (looked up once per device: the
// symbol has one instance per GPU that loaded the library).
int *device_status_ptr()
{
    static std::atomic<int *> cache[MAX_DEVICES];
    const int dev = current_device_slot();
    if (dev < 0) return nullptr;
    int *p = cache[dev].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress((void **)&p, g_device_status) != cudaSuccess) return nullptr;
        cache[dev].store(p, std::memory_order_release);
    }
    return p;
}

static bool dtype_is_8bit(int d) { return d == ICONV_U8 || d == ICONV_S8 || d == ICONV_U8_RAW128; }

static int validate(const iconv_desc &d, int &h_out, int &w_out)
{
    if (d.n < 0 || d.h < 1 || d.w < 1 || d.c_in < 1 || d.c_out < 1 || d.kh < 1 || d.kw < 1 || d.stride < 1 ||
        d.pad < 0) {
        set_error("iconv_plan: sizes must be positive (n may be 0)");
        return ICONV_ERR_ARG;
    }
    if (!(d.in_dtype == ICONV_U8 || d.in_dtype == ICONV_S8 || d.in_dtype == ICONV_U8_RAW128)) {
        set_error("iconv_plan: in_dtype must be U8, S8 or U8_RAW128");
        return ICONV_ERR_ARG;
    }
    if (!(d.out_dtype == ICONV_U8 || d.out_dtype == ICONV_S8 || d.out_dtype == ICONV_I32)) {
        set_error("iconv_plan: out_dtype must be U8, S8 or I32");
        return ICONV_ERR_ARG;
    }
    if (d.skip_dtype < -1 || d.skip_dtype > ICONV_U8_RAW128) {
        set_error("iconv_plan: bad skip_dtype");
        return ICONV_ERR_ARG;
    }
    if (d.kernel < ICONV_KERNEL_AUTO || d.kernel > ICONV_KERNEL_UMMA_IM2COL) {
        set_error("iconv_plan: bad kernel selector");
        return ICONV_ERR_ARG;
    }
    if (!d.weights || !d.bias) {
        set_error("iconv_plan: w and bias must be given");
        return ICONV_ERR_ARG;
    }
    h_out = (d.h + 2 * d.pad - d.kh) / d.stride + 1;
    w_out = (d.w + 2 * d.pad - d.kw) / d.stride + 1;
    if (d.h + 2 * d.pad < d.kh || d.w + 2 * d.pad < d.kw || h_out < 1 || w_out < 1) {
        set_error("iconv_plan: kernel larger than the padded input");
        return ICONV_ERR_SHAPE;
    }
    if (d.in_c_offset < 0 || d.in_c_offset + d.c_in > d.in_c_total || d.out_c_offset < 0 ||
        d.out_c_offset + d.c_out > d.out_c_total) {
        set_error("iconv_plan: channel slice outside its tensor");
        return ICONV_ERR_SHAPE;
    }
    const bool proj = d.proj_weights != nullptr;
    if (proj) {
        if (!d.proj_bias || !(d.skip_dtype == ICONV_U8 || d.skip_dtype == ICONV_S8) || d.proj_h < 1 || d.proj_w < 1 ||
            d.proj_c_in < 1 || d.proj_k < 1 || d.proj_stride < 1 || d.proj_pad < 0) {
            set_error("iconv_plan: a fused projection needs proj_bias, skip_dtype U8 or S8 and positive sizes");
            return ICONV_ERR_ARG;
        }
        if (d.proj_c_offset < 0 || d.proj_c_offset + d.proj_c_in > d.proj_c_total) {
            set_error("iconv_plan: projection input slice outside its tensor");
            return ICONV_ERR_SHAPE;
        }
        if (d.proj_h + 2 * d.proj_pad < d.proj_k || d.proj_w + 2 * d.proj_pad < d.proj_k ||
            (d.proj_h + 2 * d.proj_pad - d.proj_k) / d.proj_stride + 1 != h_out ||
            (d.proj_w + 2 * d.proj_pad - d.proj_k) / d.proj_stride + 1 != w_out) {
            set_error("iconv_plan: the projection's output grid differs from the layer's");
            return ICONV_ERR_SHAPE;
        }
        if (!d.brelu || d.out_dtype == ICONV_I32) {
            set_error("iconv_plan: a fused projection needs brelu = 1 and an 8-bit output");
            return ICONV_ERR_UNSUPPORTED;
        }
    }
    if (!proj && d.skip_dtype >= 0 && (d.skip_c_offset < 0 || d.skip_c_offset + d.c_out > d.skip_c_total)) {
        set_error("iconv_plan: skip slice outside its tensor");
        return ICONV_ERR_SHAPE;
    }
    if (d.skip_dtype >= 0 && (d.skip_mul < 1 || d.skip_shift < 0 || d.skip_shift > 40)) {
        set_error("iconv_plan: skip_mul must be >= 1 and 0 <= skip_shift <= 40");
        return ICONV_ERR_ARG;
    }
    if ((long long)d.n * d.h * d.w * d.in_c_total >= (1ll << 40) ||
        (long long)d.n * h_out * w_out * d.out_c_total >= (1ll << 40)) {
        set_error("iconv_plan: tensor too large");
        return ICONV_ERR_SHAPE;
    }
    if (d.out_dtype != ICONV_I32) {
        if (!d.mul || !d.shift || !d.h_i) {
            set_error("iconv_plan: mul, shift and h_i must be given for an 8-bit output");
            return ICONV_ERR_ARG;
        }
        const int np = d.per_channel ? d.c_out : 1;
        for (int i = 0; i < np; ++i) {
            if (d.mul[i] < 1 || d.shift[i] < 0 || d.shift[i] > 40 || d.h_i[i] < 0) {
                set_error("iconv_plan: need mul >= 1, 0 <= shift <= 40, h_i >= 0 (entry %d)", i);
                return ICONV_ERR_ARG;
            }
        }
        const int lo = d.out_dtype == ICONV_U8 ? 0 : -128, hi = d.out_dtype == ICONV_U8 ? 255 : 127;
        if (d.out_lo > d.out_hi || d.out_lo < lo || d.out_hi > hi) {
            set_error("iconv_plan: [out_lo, out_hi] must lie inside the output type's range");
            return ICONV_ERR_ARG;
        }
    }
    // worst-case |Y| per output channel from the actual weights: every partial sum, in any
    // order, stays inside int32 when this bound does.
    const long long xmax = d.in_dtype == ICONV_U8 ? 255 : 128;
    long long skip_bound = 0;
    if (!proj && d.skip_dtype >= 0 && dtype_is_8bit(d.skip_dtype)) {
        const long long smax = d.skip_dtype == ICONV_U8 ? 255 : 128;
        skip_bound = ((smax * d.skip_mul) >> d.skip_shift) + 1;
    }
    if (proj) {
        // worst-case |S| over the channels from the projection's actual weights
        const long long pmax = d.skip_dtype == ICONV_U8 ? 255 : 128;
        const long long KP = (long long)d.proj_k * d.proj_k * d.proj_c_in;
        long long worst = 0;
        for (int co = 0; co < d.c_out; ++co) {
            long long sw = 0;
            const int8_t *wr = d.proj_weights + (long long)co * KP;
            for (long long k = 0; k < KP; ++k) sw += wr[k] < 0 ? -(long long)wr[k] : wr[k];
            long long b = d.proj_bias[co];
            if (b < 0) b = -b;
            if (sw * pmax + b >= (1ll << 31)) {
                set_error("iconv_plan: worst-case |S| of projection channel %d does not fit int32", co);
                return ICONV_ERR_OVERFLOW;
            }
            if (sw * pmax + b > worst) worst = sw * pmax + b;
        }
        if (worst > ((1ll << 62) / d.skip_mul)) { set_error("iconv_plan: rescaled projection skip overflows"); return ICONV_ERR_OVERFLOW; }
        skip_bound = ((worst * d.skip_mul) >> d.skip_shift) + 1;
    }
    const long long K = (long long)d.kh * d.kw * d.c_in;
    for (int co = 0; co < d.c_out; ++co) {
        long long sw = 0;
        const int8_t *wr = d.weights + (long long)co * K;
        for (long long k = 0; k < K; ++k) sw += wr[k] < 0 ? -(long long)wr[k] : wr[k];
        long long b = d.bias[co];
        if (b < 0) b = -b;
        if (sw * xmax + b + skip_bound >= (1ll << 31)) {
            set_error("iconv_plan: worst-case |Y| of output channel %d does not fit int32", co);
            return ICONV_ERR_OVERFLOW;
        }
    }
    return ICONV_OK;
}

template <typename T>
static int upload(T **dev, const T *host, size_t count)
{
    *dev = nullptr;
    if (count == 0) return ICONV_OK;
    ICONV_CUDA_TRY(cudaMalloc((void **)dev, count * sizeof(T)));
    ICONV_CUDA_TRY(cudaMemcpy(*dev, host, count * sizeof(T), cudaMemcpyHostToDevice));
    return ICONV_OK;
}

}  // namespace iconv

using namespace iconv;

extern "C" const char *iconv_last_error(void) { return g_err; }

extern "C" int iconv_plan_destroy(iconv_plan_t *p)
{
    if (!p) return ICONV_OK;
    cudaFree(p->w_dev);
    cudaFree(p->bias_dev);
    cudaFree(p->mul_dev);
    cudaFree(p->shift_dev);
    cudaFree(p->h_i_dev);
    cudaFree(p->w_packed);
    cudaFree(p->params_packed);
    if (p->inner) iconv_plan_destroy(p->inner);
    delete p;
    return ICONV_OK;
}

extern "C" int iconv_plan(const iconv_desc *desc, iconv_plan_t **plan_out) { return iconv::plan_create(desc, 0, plan_out); }

int iconv::plan_create(const iconv_desc *desc, int pair16, iconv_plan_t **plan_out)
{
    if (!desc || !plan_out) {
        set_error("iconv_plan: null argument");
        return ICONV_ERR_ARG;
    }
    *plan_out = nullptr;
    int h_out = 0, w_out = 0;
    int rc = validate(*desc, h_out, w_out);
    if (rc != ICONV_OK) return rc;

    iconv_plan_t *p = new (std::nothrow) iconv_plan_t();
    if (!p) {
        set_error("iconv_plan: out of host memory");
        return ICONV_ERR_ARG;
    }
    p->d = *desc;
    p->h_out = h_out;
    p->w_out = w_out;
    p->pair16 = pair16;
    const iconv_desc &d = *desc;
    const size_t K = (size_t)d.kh * d.kw * d.c_in;
    const int np = d.per_channel ? d.c_out : 1;
    const int32_t one = 1, zero = 0;
    rc = upload(&p->w_dev, d.weights, K * d.c_out);
    if (rc == ICONV_OK) rc = upload(&p->bias_dev, d.bias, (size_t)d.c_out);
    if (rc == ICONV_OK) rc = d.out_dtype != ICONV_I32 ? upload(&p->mul_dev, d.mul, (size_t)np) : upload(&p->mul_dev, &one, 1);
    if (rc == ICONV_OK) rc = d.out_dtype != ICONV_I32 ? upload(&p->shift_dev, d.shift, (size_t)np) : upload(&p->shift_dev, &zero, 1);
    if (rc == ICONV_OK) rc = d.out_dtype != ICONV_I32 ? upload(&p->h_i_dev, d.h_i, (size_t)np) : upload(&p->h_i_dev, &zero, 1);
    if (rc == ICONV_OK) rc = choose_kernel(p);
    // the plan keeps no host pointers
    p->d.weights = nullptr;
    p->d.bias = nullptr;
    p->d.mul = p->d.shift = p->d.h_i = nullptr;
    p->d.proj_weights = nullptr;
    p->d.proj_bias = nullptr;
    if (rc != ICONV_OK) {
        iconv_plan_destroy(p);
        return rc;
    }
    *plan_out = p;
    return ICONV_OK;
}

extern "C" int iconv_plan_kernel(const iconv_plan_t *plan)
{
    if (!plan) {
        set_error("iconv_plan_kernel: null plan");
        return ICONV_ERR_ARG;
    }
    return plan->kernel;
}

extern "C" int iconv_plan_describe(const iconv_plan_t *p, char *text, size_t size)
{
    if (!p || !text || size == 0) {
        set_error("iconv_plan_describe: null argument");
        return ICONV_ERR_ARG;
    }
    static const char *fam[] = {"auto", "direct", "umma", "thin", "stem", "umma"};
    if (p->kernel == ICONV_KERNEL_UMMA)
        snprintf(text, size, "umma %s block_n=%d kc=%d stages=%d kg=%d resident_b=%d epi_warps=%d cs=%d bi=%d nbuf=%d epi=%d proj_iters=%d issuers=%d",
                 p->window ? (p->win_blocks ? "window(blocks)" : p->win_full_width ? "window(rows)" : "window(strips)") : p->pair ? "im2col(cta pairs)" : "im2col", p->block_n, p->kc,
                 p->window ? p->win_stages : p->stages, p->kg, p->window ? 1 : p->resident_b, p->epi_warps, p->cs, p->bi, p->window ? p->win_nbuf : p->nbuf, p->epi,
                 p->proj_iters, p->window ? p->win_issuers : 1);
    else if (p->kernel == ICONV_KERNEL_STEM && p->inner)
        snprintf(text, size, "stem -> umma block_n=%d kc=%d stages=%d kg=%d issuers=%d", p->inner->block_n, p->inner->kc,
                 p->inner->window ? p->inner->win_stages : p->inner->stages, p->inner->kg, p->inner->window ? p->inner->win_issuers : 1);
    else
        snprintf(text, size, "%s", fam[p->kernel >= 0 && p->kernel <= 5 ? p->kernel : 0]);
    return ICONV_OK;
}

extern "C" size_t iconv_workspace_bytes(const iconv_plan_t *p) { return p ? p->workspace_bytes : 0; }

extern "C" int iconv_forward(const iconv_plan_t *p, const void *x, const void *skip, void *out, void *workspace, void *cuda_stream)
{
    if (!p) {
        set_error("iconv_forward: null plan");
        return ICONV_ERR_ARG;
    }
    const iconv_desc &d = p->d;
    if (d.n == 0) return ICONV_OK;
    if (!x || !out || (d.skip_dtype >= 0 && !skip)) {
        set_error("iconv_forward: null tensor pointer");
        return ICONV_ERR_ARG;
    }
    if (p->workspace_bytes && !workspace) {
        set_error("iconv_forward: this plan needs a workspace of %zu bytes (iconv_workspace_bytes)", p->workspace_bytes);
        return ICONV_ERR_ARG;
    }
    if (p->workspace_bytes && ((uintptr_t)workspace % 16)) {
        set_error("iconv_forward: the workspace must be 16-byte aligned");
        return ICONV_ERR_ALIGN;
    }
    ConvArgs a;
    a.x = x; a.skip = d.skip_dtype >= 0 ? skip : nullptr; a.out = out;
    a.w = p->w_dev; a.bias = p->bias_dev; a.mul = p->mul_dev; a.shift = p->shift_dev; a.h_i = p->h_i_dev;
    a.n = d.n; a.h = d.h; a.w_ = d.w; a.c_in = d.c_in; a.c_out = d.c_out; a.kh = d.kh; a.kw = d.kw;
    a.stride = d.stride; a.pad = d.pad; a.h_out = p->h_out; a.w_out = p->w_out;
    a.in_dtype = d.in_dtype; a.in_c_total = d.in_c_total; a.in_c_offset = d.in_c_offset;
    a.out_dtype = d.out_dtype; a.out_c_total = d.out_c_total; a.out_c_offset = d.out_c_offset;
    a.brelu = d.brelu; a.per_channel = d.per_channel; a.out_lo = d.out_lo; a.out_hi = d.out_hi; a.out_zero = d.out_zero;
    a.skip_dtype = d.skip_dtype; a.skip_c_total = d.skip_c_total; a.skip_c_offset = d.skip_c_offset;
    a.skip_mul = d.skip_mul; a.skip_shift = d.skip_shift;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    switch (p->kernel) {
    case ICONV_KERNEL_UMMA: return launch_umma(p, a, st);
    case ICONV_KERNEL_THIN: return launch_thin(p, a, st);
    case ICONV_KERNEL_STEM: return launch_stem(p, a, workspace, st);
    default: return launch_direct(a, st);
    }
}

extern "C" int iconv_check(void *cuda_stream)
{
    ICONV_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)cuda_stream));
    int st = 0;
    ICONV_CUDA_TRY(cudaMemcpyFromSymbol(&st, g_device_status, sizeof(int)));
    if (st != 0) {
        const int z = 0;
        ICONV_CUDA_TRY(cudaMemcpyToSymbol(g_device_status, &z, sizeof(int)));
        if (st == 8) {
            set_error("a kernel recorded device status code 8: a bias beyond 2^30 in magnitude was given to "
                      "iconv_stem_forward_static and replaced by 0");
            return ICONV_ERR_ARG;
        }
        set_error("a kernel recorded device status code %d: a bounded device-side wait ran out", st);
        return ICONV_ERR_TIMEOUT;
    }
    return ICONV_OK;
}

extern "C" int iconv_selftest_wait_timeout(int32_t which, int64_t limit_cycles, void *cuda_stream)
{
    if (which < 0 || which > 1 || limit_cycles < 1000 || limit_cycles > 200000000ll) {
        set_error("iconv_selftest_wait_timeout: which must be 0 or 1 and 1e3 <= limit_cycles <= 2e8");
        return ICONV_ERR_ARG;
    }
    return launch_wait_selftest(which, limit_cycles, (cudaStream_t)cuda_stream);
}

extern "C" int iconv_device_initialised(int32_t device) { return umma_device_ready(device); }

extern "C" int iadd_requant(const iadd_desc *d, const void *a, const void *b, void *out, void *cuda_stream)
{
    if (!d || d->n_elems < 0) {
        set_error("iadd_requant: bad descriptor");
        return ICONV_ERR_ARG;
    }
    if (d->n_elems == 0) return ICONV_OK;
    if (!a || !b || !out) {
        set_error("iadd_requant: null tensor pointer");
        return ICONV_ERR_ARG;
    }
    const int dts[3] = {d->a_dtype, d->b_dtype, d->out_dtype};
    for (int i = 0; i < 3; ++i)
        if (!(dts[i] == ICONV_U8 || dts[i] == ICONV_S8 || dts[i] == ICONV_I32)) {
            set_error("iadd_requant: dtypes must be U8, S8 or I32");
            return ICONV_ERR_ARG;
        }
    if (d->mul_a < 1 || d->mul_b < 1 || d->mul < 1 || d->sh_a < 0 || d->sh_a > 40 || d->sh_b < 0 || d->sh_b > 40 ||
        d->shift < 0 || d->shift > 40 || d->h_i < 0 || d->out_lo > d->out_hi) {
        set_error("iadd_requant: need multipliers >= 1, shifts in [0, 40], h_i >= 0, out_lo <= out_hi");
        return ICONV_ERR_ARG;
    }
    if (d->out_dtype == ICONV_U8 && (d->out_lo < 0 || d->out_hi > 255)) { set_error("iadd_requant: range outside uint8"); return ICONV_ERR_ARG; }
    if (d->out_dtype == ICONV_S8 && (d->out_lo < -128 || d->out_hi > 127)) { set_error("iadd_requant: range outside int8"); return ICONV_ERR_ARG; }
    return launch_add_requant(*d, a, b, out, (cudaStream_t)cuda_stream);
}

extern "C" int ipool_max(const void *x, void *out, int32_t n, int32_t h, int32_t w, int32_t c, int32_t k,
                         int32_t stride, int32_t pad, void *cuda_stream)
{
    if (n < 0 || h < 1 || w < 1 || c < 1 || k < 1 || stride < 1 || pad < 0 || pad >= k) {
        set_error("ipool_max: bad size");
        return ICONV_ERR_ARG;
    }
    if (c % 16 != 0 || (uintptr_t)x % 16 != 0 || (uintptr_t)out % 16 != 0) {
        set_error("ipool_max: c must be a multiple of 16 and pointers 16-byte aligned");
        return ICONV_ERR_ALIGN;
    }
    if (h + 2 * pad < k || w + 2 * pad < k) {
        set_error("ipool_max: window larger than the padded input");
        return ICONV_ERR_SHAPE;
    }
    if (n == 0) return ICONV_OK;
    if (!x || !out) { set_error("ipool_max: null tensor pointer"); return ICONV_ERR_ARG; }
    return launch_maxpool(x, out, n, h, w, c, k, stride, pad, (cudaStream_t)cuda_stream);
}

extern "C" int ipool_avg_requant(const void *x, void *out, int32_t n, int32_t h, int32_t w, int32_t c, int32_t mul,
                                 int32_t shift, int32_t max_int, void *cuda_stream)
{
    if (n < 0 || h < 1 || w < 1 || c < 1 || mul < 1 || shift < 0 || shift > 40 || max_int < 1 || max_int > 255) {
        set_error("ipool_avg_requant: bad argument");
        return ICONV_ERR_ARG;
    }
    if (n == 0) return ICONV_OK;
    if (!x || !out) { set_error("ipool_avg_requant: null tensor pointer"); return ICONV_ERR_ARG; }
    return launch_avgpool(x, out, n, h, w, c, mul, shift, max_int, (cudaStream_t)cuda_stream);
}
