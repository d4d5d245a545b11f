// Host side of the tensor-core convolution: plan geometry, epilogue selection, TMA descriptors,
// per-device initialisation and launch dispatch.  The device code is in umma_device.cuh; the
// kernel instances live in umma_inst_*.cu.
#include <cuda.h>

#include <atomic>
#include <mutex>
#include <vector>

#include "umma_device.cuh"
#include "umma_inst.h"

namespace iconv {

// Self-test of the bounded waits: one CTA initialises an mbarrier that nothing ever arrives at
// and waits on it with the kernels' own wait routines and a short limit.  The wait must give up,
// record its code in the device status word and let the kernel return normally.
__global__ void __launch_bounds__(64, 1) wait_timeout_selftest_kernel(int which, long long limit, int *status)
{
    __shared__ unsigned long long bar;
    __shared__ volatile int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (which == 0 && threadIdx.x == 0) {              // the wait of a single-thread role (TMA producer, MMA issuer)
        if (!mbar_wait(smem_u32(&bar), 0, &abort_flag, limit)) atomicCAS(status, 0, 7);
    } else if (which == 1 && warp == 1) {             // the wait of an epilogue warp
        if (!mbar_wait_warp(smem_u32(&bar), 0, &abort_flag, lane, limit) && lane == 0) atomicCAS(status, 0, 7);
    }
}

// ---------------------------------------------------------------- host side
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const int *, const int *, cuuint32_t, cuuint32_t,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;

int load_driver_entry_points()
{
    if (g_encode_tiled && g_encode_im2col) return ICONV_OK;
    cudaDriverEntryPointQueryResult q;
    void *f = nullptr;
    ICONV_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q));
    if (q != cudaDriverEntryPointSuccess || !f) { set_error("cuTensorMapEncodeTiled not available"); return ICONV_ERR_CUDA; }
    g_encode_tiled = (EncodeTiledFn)f;
    ICONV_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f, cudaEnableDefault, &q));
    if (q != cudaDriverEntryPointSuccess || !f) { set_error("cuTensorMapEncodeIm2col not available"); return ICONV_ERR_CUDA; }
    g_encode_im2col = (EncodeIm2colFn)f;
    return ICONV_OK;
}

// Multiplier and shift with umulhi(x, mul) >> shr == x / d for every 0 <= x < 2^31
// (mul == 0 stands for d == 1): mul = ceil(2^(31 + ceil(log2 d)) / d) fits 32 bits.
void find_divisor(unsigned d, unsigned &mul, unsigned &shr)
{
    if (d <= 1) { mul = 0; shr = 0; return; }
    unsigned lg = 0;
    while ((1ull << lg) < d) ++lg;
    const unsigned long long pw = 1ull << (31 + lg);
    mul = (unsigned)((pw + d - 1) / d);
    shr = lg - 1;
}

CUtensorMapSwizzle swizzle_of(int kc)
{
    return kc == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (kc == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

// im2col-mode map over the activation slice: dims {c_in, w, h, n}; the box is KC channels
// of 128 consecutive output pixels; base-pixel coordinates run over [-pad, dim + pad - k].
int encode_im2col_map(const iconv_plan_t *p, const void *x, int c_in, int c_total, int c_offset, int h, int w, int kh, int kw,
                      int stride, int pad, CUtensorMap *map)
{
    const iconv_desc &d = p->d;
    const cuuint64_t dims[4] = {(cuuint64_t)c_in, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)d.n};
    const cuuint64_t strides[3] = {(cuuint64_t)c_total, (cuuint64_t)c_total * w, (cuuint64_t)c_total * w * h};
    const int lower[2] = {-pad, -pad};
    const int upper[2] = {pad - (kw - 1), pad - (kh - 1)};
    const cuuint32_t estr[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
    const CUresult r = g_encode_im2col(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, (void *)((const uint8_t *)x + c_offset),
                                       dims, strides, lower, upper, (cuuint32_t)p->kc, (cuuint32_t)BLOCK_M, estr,
                                       CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(p->kc),
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeIm2col failed with %d", (int)r);
        return ICONV_ERR_UNSUPPORTED;
    }
    return ICONV_OK;
}

int encode_activation_map(const iconv_plan_t *p, const void *x, CUtensorMap *map)
{
    const iconv_desc &d = p->d;
    return encode_im2col_map(p, x, d.c_in, d.in_c_total, d.in_c_offset, d.h, d.w, d.kh, d.kw, d.stride, d.pad, map);
}

// Tiled 4-D map over the activation slice for window mode: dims {c_in, w, h, n}, box
// {KC, win_bw, win_bh, 1}; coordinates outside the image read as zero.
int encode_patch_map(const iconv_plan_t *p, const void *x, CUtensorMap *map)
{
    const iconv_desc &d = p->d;
    // (paired taps: every position is read together with its right-hand neighbour, as 32
    // channels at a 16-byte pitch; the caller keeps 16 readable bytes behind the tensor)
    const cuuint64_t dims[4] = {(cuuint64_t)(p->pair16 ? 32 : d.c_in), (cuuint64_t)d.w, (cuuint64_t)d.h, (cuuint64_t)d.n};
    const cuuint64_t strides[3] = {(cuuint64_t)d.in_c_total, (cuuint64_t)d.in_c_total * d.w, (cuuint64_t)d.in_c_total * d.w * d.h};
    const cuuint32_t box[4] = {(cuuint32_t)p->kc, (cuuint32_t)p->win_bw, (cuuint32_t)p->win_bh, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, (void *)((const uint8_t *)x + d.in_c_offset), dims, strides, box,
                                      estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(p->kc), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled (patch map) failed with %d", (int)r);
        return ICONV_ERR_UNSUPPORTED;
    }
    return ICONV_OK;
}

int encode_projection_map(const iconv_plan_t *p, const void *x, CUtensorMap *map)
{
    const iconv_desc &d = p->d;
    return encode_im2col_map(p, x, d.proj_c_in, d.proj_c_total, d.proj_c_offset, d.proj_h, d.proj_w, d.proj_k, d.proj_k,
                             d.proj_stride, d.proj_pad, map);
}

long long labs64(long long v) { return v < 0 ? -v : v; }

// Epilogue of a layer with a fused projection: explicit BReLU clamp and 32-bit Eq. 4 (as EPI_SAFE);
// the skip rescale in 32 bits when |S|max * skip_mul + |C| < 2^31 for every channel, else in 64.
// Fills c_a (C, or the layer's bias) and c_b (the projection's bias).  Returns < 0 when Eq. 4
// itself does not fit 32 bits (the caller then plans the two convolutions apart).
int choose_projection_epilogue(const iconv_desc &d, int c_out_pad, std::vector<int32_t> &c_a, std::vector<int32_t> &c_b, int &tail,
                               int &proj32)
{
    c_a.assign((size_t)c_out_pad, 0);
    c_b.assign((size_t)c_out_pad, 0);
    const int np = d.per_channel ? d.c_out : 1;
    bool tail_free = d.out_zero == 0 && d.out_lo <= 0;
    for (int i = 0; i < np; ++i) {
        if (d.shift[i] < 1 || d.shift[i] > 31) return -1;
        const unsigned long long top = (unsigned long long)d.h_i[i] * (unsigned long long)d.mul[i] + (1ull << (d.shift[i] - 1));
        if (top >= (1ull << 32)) return -1;
        if ((long long)(top >> d.shift[i]) > d.out_hi) tail_free = false;
    }
    tail = tail_free ? 0 : 1;
    const long long pmax = d.skip_dtype == ICONV_U8 ? 255 : 128;
    const long long KP = (long long)d.proj_k * d.proj_k * d.proj_c_in;
    const long long half = d.skip_shift ? (1ll << (d.skip_shift - 1)) : 0;
    proj32 = d.skip_shift <= 30 ? 1 : 0;
    for (int co = 0; co < d.c_out; ++co) {
        long long sw = 0;
        const int8_t *wr = d.proj_weights + (long long)co * KP;
        for (long long k = 0; k < KP; ++k) sw += wr[k] < 0 ? -(long long)wr[k] : wr[k];
        const long long C = (long long)d.proj_bias[co] * d.skip_mul + half + ((long long)d.bias[co] << d.skip_shift);
        if (sw * pmax * d.skip_mul + labs64(C) >= (1ll << 31)) proj32 = 0;
    }
    // The fast form (no explicit BReLU clamp, as EPI_FAST): per-layer parameters, a plain u8 output
    // whose bound h_i already maps to 255, and |Y| * mul + half < 2^31 for the worst case of both
    // reductions with the layer's actual weights.
    if (proj32 && !d.per_channel && tail_free && d.out_dtype == ICONV_U8 && d.out_hi == 255 && d.brelu && d.skip_shift == FAST_SKIP_SHIFT) {
        const long long mul = d.mul[0], qhalf = 1ll << (d.shift[0] - 1);
        bool fast = (long long)(((unsigned long long)d.h_i[0] * (unsigned long long)mul + (unsigned long long)qhalf) >> d.shift[0]) >= 255;
        const long long xmax = d.in_dtype == ICONV_U8 ? 255 : 128;
        const long long K = (long long)d.kh * d.kw * d.c_in;
        for (int co = 0; co < d.c_out && fast; ++co) {
            long long sw = 0, swp = 0;
            const int8_t *wr = d.weights + (long long)co * K, *wp = d.proj_weights + (long long)co * KP;
            for (long long k = 0; k < K; ++k) sw += wr[k] < 0 ? -(long long)wr[k] : wr[k];
            for (long long k = 0; k < KP; ++k) swp += wp[k] < 0 ? -(long long)wp[k] : wp[k];
            const long long C = (long long)d.proj_bias[co] * d.skip_mul + half + ((long long)d.bias[co] << d.skip_shift);
            const long long ymax = sw * xmax + ((swp * pmax * d.skip_mul + labs64(C)) >> d.skip_shift) + 1;
            if (ymax * mul + qhalf >= (1ll << 31)) fast = false;
        }
        if (fast) proj32 = 2;
    }
    for (int co = 0; co < d.c_out; ++co) {
        c_b[co] = d.proj_bias[co];
        c_a[co] = proj32 ? (int32_t)((long long)d.proj_bias[co] * d.skip_mul + half + ((long long)d.bias[co] << d.skip_shift))
                         : d.bias[co];
    }
    return EPI_PROJ;
}

// Per-channel parameters equal within every group of 16 channels?
bool group_uniform(const iconv_desc &d)
{
    if (!d.per_channel) return false;
    for (int co = 0; co < d.c_out; ++co) {
        const int g = co / 16 * 16;
        if (d.mul[co] != d.mul[g] || d.shift[co] != d.shift[g] || d.h_i[co] != d.h_i[g]) return false;
    }
    return true;
}

// Picks the cheapest epilogue whose 32-bit arithmetic is provably exact for this layer and
// fills the per-channel additive constant of that variant (c_a, c_out_pad entries).
// group_fast: the fast forms may also take per-channel parameters that are uniform per group of
// 16 channels (window mode fetches a group's scalars; the im2col kernel does not).
//   worst[co] = sum |w| * max|x|: no accumulator of channel co can exceed it in magnitude.
int choose_epilogue(const iconv_desc &d, int c_out_pad, std::vector<int32_t> &c_a, int &tail, bool group_fast)
{
    const long long K = (long long)d.kh * d.kw * d.c_in;
    const long long xmax = d.in_dtype == ICONV_U8 ? 255 : 128;
    c_a.assign((size_t)c_out_pad, 0);
    for (int co = 0; co < d.c_out; ++co) c_a[co] = d.bias[co];
    tail = 1;
    if (d.out_dtype == ICONV_I32) return d.skip_dtype < 0 ? EPI_RAW : EPI_WIDE;
    if (!d.brelu) return EPI_WIDE;
    const int np = d.per_channel ? d.c_out : 1;
    bool tail_free = d.out_zero == 0 && d.out_lo <= 0;
    for (int i = 0; i < np; ++i) {
        if (d.shift[i] < 1 || d.shift[i] > 31) return EPI_WIDE;
        const unsigned long long top = (unsigned long long)d.h_i[i] * (unsigned long long)d.mul[i] + (1ull << (d.shift[i] - 1));
        if (top >= (1ull << 32)) return EPI_WIDE;
        if ((long long)(top >> d.shift[i]) > d.out_hi) tail_free = false;
    }
    tail = tail_free ? 0 : 1;

    const bool skip8 = d.skip_dtype >= 0 && d.skip_dtype != ICONV_I32;
    long long skip_bound = 0;      // bound of |rescaled skip|
    if (skip8) {
        // t = s * skip_mul + C, C = (b << skip_shift) + half - z * skip_mul, must fit int32 for every byte s
        if (d.skip_shift > 30) return EPI_WIDE;
        const long long z = d.skip_dtype == ICONV_U8 ? 0 : 128;
        const long long half = d.skip_shift ? (1ll << (d.skip_shift - 1)) : 0;
        for (int co = 0; co < d.c_out; ++co) {
            const long long C = ((long long)d.bias[co] << d.skip_shift) + half - z * d.skip_mul;
            if (labs64(C) + 255ll * d.skip_mul >= (1ll << 31)) return EPI_WIDE;
            c_a[co] = (int32_t)C;
        }
        skip_bound = ((255ll * d.skip_mul) >> d.skip_shift) + 1;
    }
    // the fast form: no clamp before the multiplication, the u8 saturation does both clamps
    bool fast = (!d.per_channel || (group_fast && group_uniform(d))) && d.out_dtype == ICONV_U8 && d.out_zero == 0 && d.out_lo == 0 && d.out_hi == 255 &&
                d.skip_dtype != ICONV_I32;
    if (fast) {
        for (int co = 0; co < d.c_out && fast; ++co) {
            const int q = d.per_channel ? co : 0;
            const long long mul = d.mul[q], half = 1ll << (d.shift[q] - 1);
            // BReLU's upper clamp may only be dropped when h_i already maps to the saturation bound
            if ((long long)(((unsigned long long)d.h_i[q] * (unsigned long long)mul + (unsigned long long)half) >> d.shift[q]) < 255) fast = false;
            long long sw = 0;
            const int8_t *wr = d.weights + (long long)co * K;
            for (long long k = 0; k < K; ++k) sw += wr[k] < 0 ? -(long long)wr[k] : wr[k];
            const long long ymax = sw * xmax + labs64(d.bias[co]) + skip_bound;
            if (ymax * mul + half >= (1ll << 31)) fast = false;
        }
        if (fast) {
            if (!skip8)
                for (int co = 0; co < d.c_out; ++co) {
                    const int q = d.per_channel ? co : 0;
                    c_a[co] = (int32_t)((long long)d.bias[co] * d.mul[q] + (1ll << (d.shift[q] - 1)));
                }
            if (!skip8) return EPI_FAST;
            if (d.skip_shift == FAST_SKIP_SHIFT) return EPI_FAST_SKIP8;     // the clamp-free skip form is compiled for this shift only
        }
    }
    if (d.skip_dtype < 0) return EPI_SAFE;
    return skip8 ? EPI_SAFE_SKIP8 : EPI_SAFE_SKIP32;
}

// Tiled 2-D map over a channel slice of an NHWC tensor seen as [pixels][channels]; the box
// is one staged piece: 32 pixels x piece_bytes.
int encode_rows_map(const void *base, int elem_bytes, int c_slice, int c_total, long long pixels,
                    int piece_bytes, CUtensorMap *map)
{
    const cuuint64_t dims[2] = {(cuuint64_t)c_slice, (cuuint64_t)pixels};
    const cuuint64_t strides[1] = {(cuuint64_t)c_total * elem_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)(piece_bytes / elem_bytes), 32};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapSwizzle sw = piece_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : piece_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                  : piece_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
    const CUresult r = g_encode_tiled(map, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_INT32 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
                                      (void *)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                                      CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled (rows map) failed with %d", (int)r);
        return ICONV_ERR_UNSUPPORTED;
    }
    return ICONV_OK;
}

}  // namespace

// A layer whose 8-bit output (or skip) is too narrow or too oddly placed for 16-byte stores:
// window mode writes it byte by byte (EPI_NARROW) where its other conditions hold.
bool umma_narrow(const iconv_desc &d)
{
    if (d.out_dtype == ICONV_I32) return false;
    const bool odd_out = d.c_out % 16 || d.out_c_total % 16 || d.out_c_offset % 16;
    const bool odd_skip = d.skip_dtype >= 0 && d.skip_dtype != ICONV_I32 && (d.skip_c_total % 16 || d.skip_c_offset % 16);
    return (odd_out || odd_skip) && d.stride == 1 && d.c_in <= 128 && d.c_out <= 64 && !d.proj_weights &&
           d.kernel != ICONV_KERNEL_UMMA_IM2COL;
}

int umma_supported(const iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    const char *why = nullptr;
    const bool narrow = umma_narrow(d);
    if (d.in_dtype == ICONV_U8_RAW128) why = "raw-128 inputs are not GEMM operands";
    else if (d.c_in % 16 || d.in_c_total % 16 || d.in_c_offset % 16) why = "input channels must be multiples of 16";
    else if (d.c_out < 16 && !narrow) why = "c_out below 16";
    else if (d.out_dtype == ICONV_I32 && (d.c_out % 4 || d.out_c_total % 4 || d.out_c_offset % 4)) why = "int32 output channels must be multiples of 4";
    else if (!narrow && d.out_dtype != ICONV_I32 && (d.c_out % 16 || d.out_c_total % 16 || d.out_c_offset % 16)) why = "8-bit output channels must be multiples of 16";
    else if (d.skip_dtype == ICONV_I32 && (d.skip_c_total % 4 || d.skip_c_offset % 4)) why = "int32 skip channels must be multiples of 4";
    else if (!narrow && d.skip_dtype >= 0 && d.skip_dtype != ICONV_I32 && (d.skip_c_total % 16 || d.skip_c_offset % 16)) why = "8-bit skip channels must be multiples of 16";
    else if (d.kh > 16 || d.kw > 16 || d.pad > 16 || d.stride > 8) why = "filter, padding or stride beyond the im2col descriptor's range";
    else if ((long long)d.kh * d.kw * ((d.c_in + 127) / 128 * 128) >= (1ll << 24)) why = "reduction too long";
    else if ((long long)d.n * p->h_out * p->w_out >= (1ll << 31) - 256) why = "more than 2^31 output pixels";
    else if (d.proj_weights && (d.proj_c_in % 16 || d.proj_c_total % 16 || d.proj_c_offset % 16)) why = "projection input channels must be multiples of 16";
    else if (d.proj_weights && (d.proj_k > 16 || d.proj_pad > 16 || d.proj_stride > 8)) why = "projection filter, padding or stride beyond the im2col descriptor's range";
    else if (d.proj_weights && d.out_dtype == ICONV_I32) why = "a fused projection needs an 8-bit output";
    if (why) {
        set_error("tensor-core path: %s", why);
        return ICONV_ERR_UNSUPPORTED;
    }
    return ICONV_OK;
}

// Once per device: driver entry points (once per process) and the kernels' shared-memory opt-in,
// which is an attribute of the function ON THE CURRENT DEVICE, so every GPU a process uses gets
// its own pass.  Allocates nothing.
namespace {

struct DeviceInit {
    std::atomic<int> ready{0};      // 1 once the opt-ins ran on this device
    int sms = 0;
};
DeviceInit g_device_init[MAX_DEVICES];
std::mutex g_device_init_mutex;

}  // namespace

// The slot of the per-device table the first call on a device fills; tests read it to see that
// initialisation is keyed by device (-1: not initialised yet).
int umma_device_ready(int device)
{
    if (device < 0 || device >= MAX_DEVICES) return -1;
    return g_device_init[device].ready.load(std::memory_order_acquire) ? g_device_init[device].sms : -1;
}

cudaError_t umma_conv_launch(int epi, int issue, const UmmaLaunch &l)
{
    switch (epi) {
    case EPI_RAW: return umma_conv_launch_1(issue, l);
    case EPI_FAST: return umma_conv_launch_2(issue, l);
    case EPI_FAST_SKIP8: return umma_conv_launch_3(issue, l);
    case EPI_SAFE: return umma_conv_launch_4(issue, l);
    case EPI_SAFE_SKIP8: return umma_conv_launch_5(issue, l);
    case EPI_SAFE_SKIP32: return umma_conv_launch_6(issue, l);
    case EPI_PROJ: return umma_conv_launch_7(issue, l);
    default: return umma_conv_launch_0(issue, l);
    }
}

cudaError_t umma_conv_opt_in(int epi)
{
    switch (epi) {
    case EPI_RAW: return umma_conv_opt_in_1();
    case EPI_FAST: return umma_conv_opt_in_2();
    case EPI_FAST_SKIP8: return umma_conv_opt_in_3();
    case EPI_SAFE: return umma_conv_opt_in_4();
    case EPI_SAFE_SKIP8: return umma_conv_opt_in_5();
    case EPI_SAFE_SKIP32: return umma_conv_opt_in_6();
    case EPI_PROJ: return umma_conv_opt_in_7();
    default: return umma_conv_opt_in_0();
    }
}

cudaError_t umma_window_launch(int epi, int kh, int kw, int kj, int pair16, const UmmaLaunch &l)
{
    switch (epi) {
    case EPI_FAST: return umma_window_launch_2(kh, kw, kj, pair16, l);
    case EPI_FAST_SKIP8: return umma_window_launch_3(kh, kw, kj, pair16, l);
    case EPI_SAFE_SKIP8: return umma_window_launch_5(kh, kw, kj, pair16, l);
    case EPI_NARROW: return umma_window_launch_8(kh, kw, kj, pair16, l);
    default: return umma_window_launch_4(kh, kw, kj, pair16, l);
    }
}

cudaError_t umma_window_opt_in(int epi)
{
    switch (epi) {
    case EPI_FAST: return umma_window_opt_in_2();
    case EPI_FAST_SKIP8: return umma_window_opt_in_3();
    case EPI_SAFE_SKIP8: return umma_window_opt_in_5();
    case EPI_NARROW: return umma_window_opt_in_8();
    default: return umma_window_opt_in_4();
    }
}

int umma_init_once()
{
    const int rc = load_driver_entry_points();
    if (rc != ICONV_OK) return rc;
    const int dev = current_device_slot();
    if (dev < 0) { set_error("tensor-core path: no current device, or its index is beyond %d", MAX_DEVICES - 1); return ICONV_ERR_UNSUPPORTED; }
    DeviceInit &di = g_device_init[dev];
    if (di.ready.load(std::memory_order_acquire)) return ICONV_OK;
    std::lock_guard<std::mutex> lock(g_device_init_mutex);
    if (di.ready.load(std::memory_order_acquire)) return ICONV_OK;
    for (int epi = EPI_WIDE; epi <= EPI_PROJ; ++epi) ICONV_CUDA_TRY(umma_conv_opt_in(epi));
    for (int epi : {EPI_FAST, EPI_FAST_SKIP8, EPI_SAFE, EPI_SAFE_SKIP8, EPI_NARROW}) ICONV_CUDA_TRY(umma_window_opt_in(epi));
    ICONV_CUDA_TRY(cudaDeviceGetAttribute(&di.sms, cudaDevAttrMultiProcessorCount, dev));
    di.ready.store(1, std::memory_order_release);
    return ICONV_OK;
}

// Reduction steps along the filter: kh * kw taps, or half of that when two horizontally
// adjacent 16-channel taps share one 32-byte K step (paired taps).
int plan_taps(const iconv_plan_t *p) { return p->pair16 ? p->d.kh * (p->d.kw / 2) : p->d.kh * p->d.kw; }

// Tile, pipeline and epilogue geometry of a layer, from its descriptor alone (host only).
int umma_geometry(iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    // channel chunk per pipeline stage: the padded reduction should be as short as possible,
    // ties go to the wider chunk (fewer, larger TMA transactions)
    const bool proj = d.proj_weights != nullptr;
    int best_kc = 0, best_pad = 0;
    for (int kc = 128; kc >= 32; kc /= 2) {
        const int padded = (d.c_in + kc - 1) / kc * kc + (proj ? (d.proj_c_in + kc - 1) / kc * kc : 0);
        if (best_kc == 0 || padded < best_pad) { best_kc = kc; best_pad = padded; }
    }
    p->kc = best_kc;
    p->c_in_pad = (d.c_in + best_kc - 1) / best_kc * best_kc;
    p->proj_c_in_pad = proj ? (d.proj_c_in + best_kc - 1) / best_kc * best_kc : 0;
    p->swizzle_bytes = best_kc;
    // a fused projection keeps two accumulator tiles per buffer: at most 128 columns each
    const int n_max = proj ? 128 : 256;
    const int n_tiles = (d.c_out + n_max - 1) / n_max;
    p->block_n = ((d.c_out + n_tiles - 1) / n_tiles + 15) / 16 * 16;
    p->c_out_pad = p->block_n * n_tiles;
    const int taps = plan_taps(p);
    p->proj_iters = proj ? d.proj_k * d.proj_k * (p->proj_c_in_pad / p->kc) : 0;
    const int k_iters = p->proj_iters + taps * (p->c_in_pad / p->kc);
    const int esz = d.out_dtype == ICONV_I32 ? 4 : 1;

    // accumulator buffers: four when a buffer has at most 128 columns, else two
    p->nbuf = p->block_n * (proj ? 2 : 1) <= 128 ? 4 : 2;

    // shared-memory budget: pipeline stages (+ the resident filter bank) against the
    // epilogue warps' staging.  Sixteen epilogue warps unless that leaves the pipeline short.
    const int stage_a = BLOCK_M * p->kc;
    const int b_tile = (p->block_n * p->kc + 1023) / 1024 * 1024;
    const long long bank = (long long)b_tile * k_iters * n_tiles;
    const int fixed = (int)sizeof(Shared) + 2048;
    // Epilogue-heavy layers (many output columns per k-iteration, more with a skip to rescale) get
    // sixteen epilogue warps, the others eight and a deeper pipeline.  A stage groups kg
    // k-iterations (at most 48 KB) as long as three stages still fit (two for a tile that is a
    // single stage): the MMA issuer's wait + commit round costs about 400 cycles whatever the
    // stage holds.
    p->resident_b = 0;
    p->epi_warps = 0;
    p->kg = 1;
    const int weight = p->block_n * (proj ? 7 : (d.skip_dtype >= 0 ? 5 : 2)) / (2 * k_iters);
    // staging per epilogue warp: 8-bit pieces are 2 KB each, and only an 8-bit skip (not a fused
    // projection's operand) is staged behind them
    const bool stage_skip = d.skip_dtype >= 0 && d.skip_dtype != ICONV_I32 && !proj;
    // Candidates in order of preference: sixteen warps with the full skip ring, sixteen with a ring of
    // two pieces (the load of a piece then leads its use by one piece instead of two), eight warps.
    const int first_ew = weight >= 100 ? 16 : 8;
    int cand[3][2], n_cand = 0;
    cand[n_cand][0] = first_ew; cand[n_cand++][1] = SKIP_RING;
    if (stage_skip) { cand[n_cand][0] = first_ew; cand[n_cand++][1] = 2; }
    if (first_ew != 8) { cand[n_cand][0] = 8; cand[n_cand++][1] = SKIP_RING; }
    for (int ci = 0; ci < n_cand && !p->epi_warps; ++ci) {
        const int ew = cand[ci][0], ring = cand[ci][1];
        const int warp_bytes = stage_skip ? 4096 + ring * 2048 : (d.out_dtype == ICONV_I32 ? EPI_WARP_SMEM : EPI_WARP_SMEM_SMALL);
        const int avail = MAX_SMEM - fixed - ew * warp_bytes;
        const int want = 2;
        const bool last = ci == n_cand - 1;
        int room = 0, slot = 0;
        if (bank <= RESIDENT_B_MAX && avail - (int)bank >= want * stage_a) {
            p->resident_b = 1;
            room = avail - (int)bank;
            slot = stage_a;
        } else if (avail >= want * (stage_a + b_tile) || last) {
            room = avail;
            slot = stage_a + b_tile;
        }
        if (slot) {
            p->epi_warps = ew;
            p->skip_ring = ring;
            p->epi_warp_bytes = warp_bytes;
            p->pipe_room = room;
            for (int kg = k_iters < 8 ? k_iters : 8; kg >= 1; --kg)
                if (kg * slot <= 48 * 1024 && room / (kg * slot) >= 3) { p->kg = kg; break; }
            p->stages = room / (p->kg * slot);
        }
    }
    if (p->stages > MAX_STAGES) p->stages = MAX_STAGES;
    if (p->stages < 2) { set_error("tensor-core path: tile does not fit shared memory"); return ICONV_ERR_UNSUPPORTED; }

    // epilogue geometry: slots per TMEM lane quadrant, split between a tile's columns (cs)
    // and tiles in flight (bi)
    // Twice as many accumulator buffers as tiles in flight: a group of warps that finishes a tile
    // finds the next one computed already, and the MMAs of the tile after that (into the buffer just
    // released) run under its epilogue.  With as many tiles in flight as buffers every group waited
    // for its own buffer's next MMA round after every tile (a quarter to half of its time on the
    // block-closing layers).
    const int slots = p->epi_warps / 4;
    p->bi = p->nbuf / 2 < slots ? p->nbuf / 2 : slots;
    if (p->bi < 1) p->bi = 1;
    p->cs = slots / p->bi;
    while (p->cs > 1 && p->block_n < 32 * p->cs) p->cs /= 2;     // at least 32 columns per warp
    if (p->block_n > 128 && p->cs < 2) p->cs = 2;
    p->epi_warps = 4 * p->cs * p->bi;
    p->half_n = p->cs > 1 ? (p->block_n / p->cs + 15) / 16 * 16 : p->block_n;
    {
        // staged piece: the widest power of two dividing every warp's row width, at most 64
        // bytes of 8-bit outputs or 128 bytes of int32 (two pieces fit half the warp's staging)
        int last = p->block_n - (p->cs - 1) * p->half_n;
        while (last <= 0) { --p->cs; p->epi_warps = 4 * p->cs * p->bi; p->half_n = p->cs > 1 ? (p->block_n / p->cs + 15) / 16 * 16 : p->block_n; last = p->block_n - (p->cs - 1) * p->half_n; }
        const int w0 = p->half_n * esz, w1 = last * esz;
        int pb = esz == 4 ? 128 : 64;
        while (pb > 16 && (w0 % pb || w1 % pb)) pb /= 2;
        p->piece_bytes = pb;
    }

    return ICONV_OK;
}

int umma_epilogue_safe() { return EPI_SAFE; }

// Window mode for this layer?  Fills the plan's win_* fields when it applies: stride 1, a filter
// wider than one tap, one channel chunk, one N tile, no skip, an 8-bit output whose epilogue is
// one of the 32-bit forms, the filter bank and at least two patches in shared memory, and
// tiles that are mostly real pixels.
void window_plan(iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    p->window = 0;
    if (d.kernel == ICONV_KERNEL_UMMA_IM2COL) return;
    const bool skip8_epi = p->epi == EPI_FAST_SKIP8 || p->epi == EPI_SAFE_SKIP8;      // the epilogue reads the skip rows itself
    if (d.stride != 1 || d.proj_weights || (d.skip_dtype >= 0 && p->epi != EPI_NARROW && !skip8_epi) || d.out_dtype == ICONV_I32) return;
    if (p->c_in_pad != p->kc || p->c_out_pad != p->block_n) return;
    if (p->epi != EPI_FAST && p->epi != EPI_SAFE && p->epi != EPI_NARROW && !skip8_epi) return;
    // Window mode stores 16 bytes per pixel and group straight from registers; the im2col kernel
    // stages whole rows and stores them by TMA, which wins once a pixel's output is wide: a 1x1
    // layer (no halo to save) stays there beyond 64 columns, a layer with a skip beyond 128
    // (measured: 64 -> 256 1x1 with skip 0.134 ms by im2col, 0.217 ms in window mode).
    if (d.kh * d.kw == 1 && p->block_n > 64 && p->epi != EPI_NARROW) return;
    if (skip8_epi && p->block_n > 128) return;
    const int taps = plan_taps(p);
    const int b_tile = (p->block_n * p->kc + 1023) / 1024 * 1024;
    const long long bank = (long long)b_tile * taps;
    const int wp = p->w_out + d.kw - 1;
    const long long room = MAX_SMEM - 1024 - (long long)sizeof(Shared) - bank;
    // Three tilings of an image into 128 output pixels per tile; the cheapest by a simple
    // model wins (per tile the patch comes in at about 20 bytes per clock, an MMA takes 64 or
    // 128 clocks, and the two overlap only in part):
    //   rows    the padded width, tiles run on across rows        (narrow images)
    //   strips  128 pixels of one row                              (wide images)
    //   blocks  8 x 16 pixels: the smallest halo, 8-row operand groups one patch line apart
    const int n_mma = taps * (p->kc / 32);
    const double mma_clk = (double)n_mma * (p->block_n > 128 ? 128 : 64);
    double best = -1;
    int vw = 0, bw = 0, bh = 0, full_width = 0, blocks = 0;
    long long tpi = 0, patch = 0;
    for (int mode = 0; mode < 3; ++mode) {
        int m_vw, m_bw, m_bh;
        long long m_tpi;
        if (mode == 0) {
            if (p->w_out >= 128) continue;
            m_vw = wp; m_bw = wp; m_bh = (wp - 1 + 127) / wp + d.kh;
            m_tpi = ((long long)p->h_out * m_vw + BLOCK_M - 1) / BLOCK_M;
        } else if (mode == 1) {
            if (p->w_out < 128) continue;
            m_vw = (p->w_out + 127) / 128 * 128; m_bw = 128 + d.kw - 1; m_bh = d.kh;
            m_tpi = ((long long)p->h_out * m_vw + BLOCK_M - 1) / BLOCK_M;
        } else {
            m_vw = (p->w_out + 7) / 8; m_bw = 8 + d.kw - 1; m_bh = 16 + d.kh - 1;
            m_tpi = (long long)m_vw * ((p->h_out + 15) / 16);
            if ((long long)m_bw * p->kc >= (1 << 18)) continue;     // the group stride field holds 14 bits of 16-byte units
        }
        if (m_bw > 256 || m_bh > 256) continue;
        const long long m_patch = ((long long)(m_bh * m_bw + d.kw) * p->kc + 1023) / 1024 * 1024;
        if (m_patch > 64 * 1024 || room < 2 * m_patch) continue;
        if ((long long)p->h_out * p->w_out * 10 < m_tpi * BLOCK_M * 6) continue;      // under 60 % real pixels
        if (m_tpi * d.n >= (1ll << 31) / BLOCK_M) continue;
        const double tma_clk = (double)m_patch / 20.0;
        const double cost = (double)m_tpi * ((mma_clk > tma_clk ? mma_clk : tma_clk) + 0.25 * (mma_clk > tma_clk ? tma_clk : mma_clk));
        if (best < 0 || cost < best) {
            best = cost; vw = m_vw; bw = m_bw; bh = m_bh; full_width = mode == 0; blocks = mode == 2; tpi = m_tpi; patch = m_patch;
        }
    }
    if (best < 0) return;
    p->window = 1;
    p->win_vw = vw; p->win_bw = bw; p->win_bh = bh; p->win_full_width = full_width; p->win_blocks = blocks; p->win_tpi = (int)tpi;
    p->win_patch_bytes = (int)patch;
    p->win_stages = (int)(room / patch < 6 ? room / patch : 6);
    // Sixteen epilogue warps (no staging memory is needed here), and twice as many accumulator buffers
    // as tiles in flight wherever the 512 TMEM columns allow it: a buffer belongs to one group of warps,
    // so with as many tiles in flight as buffers the MMAs of a group's next tile could only start once
    // its epilogue had ended, and the two never overlapped.
    const int slots = 4;
    p->win_nbuf = p->block_n <= 64 ? 8 : p->nbuf;
    // MMA-issuing warps: three with six stages and eight accumulator buffers, else two with an even number of
    // stages.  The issuers take the tiles in turn and wait on barriers by phase parity, which tells a phase only
    // from its neighbours: a stage's fills must all pass through one issuer (issuers divide stages), and an
    // issuer must never be a whole round of accumulator buffers ahead of the others (stages <= buffers, or
    // issuers divide buffers).
    if (p->win_stages >= 6 && p->win_nbuf >= 8) {
        p->win_stages = 6;
        p->win_issuers = 3;
    } else {
        p->win_stages = p->win_stages / 2 * 2;
        p->win_issuers = 2;
    }
    p->bi = p->win_nbuf / 2 < slots ? p->win_nbuf / 2 : slots;
    if (p->bi < 1) p->bi = 1;
    p->cs = slots / p->bi;
    while (p->cs > 1 && p->block_n < 32 * p->cs) p->cs /= 2;
    p->half_n = p->cs > 1 ? (p->block_n / p->cs + 15) / 16 * 16 : p->block_n;
    while (p->cs > 1 && p->block_n - (p->cs - 1) * p->half_n <= 0) { --p->cs; p->half_n = p->cs > 1 ? (p->block_n / p->cs + 15) / 16 * 16 : p->block_n; }
    p->epi_warps = 4 * p->cs * p->bi;
}

// 2-D tiled map over the packed weights p->w_packed, [c_out_pad][taps * c_in_pad].
int umma_encode_weight_map(iconv_plan_t *p)
{
    const size_t k_pad = (size_t)plan_taps(p) * p->c_in_pad + (size_t)p->proj_iters * p->kc;
    const cuuint64_t dims[2] = {(cuuint64_t)k_pad, (cuuint64_t)p->c_out_pad};
    const cuuint64_t strides[1] = {(cuuint64_t)k_pad};
    const cuuint32_t box[2] = {(cuuint32_t)p->kc, (cuuint32_t)(p->pair ? p->block_n / 2 : p->block_n)};    // pairs: each CTA loads half of a B tile
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode_tiled(&p->tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, p->w_packed, dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(p->kc), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed with %d", (int)r);
        return ICONV_ERR_UNSUPPORTED;
    }
    return ICONV_OK;
}

int umma_setup(iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    int rc = umma_init_once();
    if (rc != ICONV_OK) return rc;
    rc = umma_geometry(p);
    if (rc != ICONV_OK) return rc;

    // repack weights [c_out][tap][c_in] -> [c_out_pad][tap][c_in_pad], zero filled; a fused
    // projection's weights come first in every row
    const int taps = plan_taps(p), ptaps = d.proj_weights ? d.proj_k * d.proj_k : 0;
    const size_t kp_pad = (size_t)ptaps * p->proj_c_in_pad;
    const size_t k_pad = kp_pad + (size_t)taps * p->c_in_pad;
    std::vector<int8_t> packed((size_t)p->c_out_pad * k_pad, 0);
    for (int co = 0; co < d.c_out; ++co) {
        for (int t = 0; t < ptaps; ++t)
            memcpy(&packed[(size_t)co * k_pad + (size_t)t * p->proj_c_in_pad], d.proj_weights + ((size_t)co * ptaps + t) * d.proj_c_in,
                   (size_t)d.proj_c_in);
        if (p->pair16) {    // [R][S][16] read as [R][S / 2][32]: the row as it stands
            memcpy(&packed[(size_t)co * k_pad], d.weights + (size_t)co * k_pad, k_pad);
            continue;
        }
        for (int t = 0; t < taps; ++t)
            memcpy(&packed[(size_t)co * k_pad + kp_pad + (size_t)t * p->c_in_pad], d.weights + ((size_t)co * taps + t) * d.c_in, (size_t)d.c_in);
    }
    ICONV_CUDA_TRY(cudaMalloc((void **)&p->w_packed, packed.size()));
    ICONV_CUDA_TRY(cudaMemcpy(p->w_packed, packed.data(), packed.size(), cudaMemcpyHostToDevice));

    rc = umma_encode_weight_map(p);
    if (rc != ICONV_OK) return rc;
    // make sure the activation descriptor can be encoded for this geometry (the address is
    // only stored, never read, so the packed weights stand in for it)
    CUtensorMap probe;
    rc = encode_activation_map(p, (const uint8_t *)p->w_packed - d.in_c_offset, &probe);
    if (rc != ICONV_OK) return rc;
    if (d.proj_weights) {
        rc = encode_projection_map(p, (const uint8_t *)p->w_packed - d.proj_c_offset, &probe);
        if (rc != ICONV_OK) return rc;
    }

    // epilogue variant and its per-channel constants: {c_a, mul, shift, h_i, c_b} x c_out_pad
    std::vector<int32_t> c_a, c_b;
    p->proj32 = 0;
    if (d.proj_weights) {
        p->epi = choose_projection_epilogue(d, p->c_out_pad, c_a, c_b, p->tail, p->proj32);
        if (p->epi < 0) { set_error("tensor-core path: Eq. 4 of a layer with a fused projection must fit 32 bits"); return ICONV_ERR_UNSUPPORTED; }
    } else {
        p->epi = choose_epilogue(d, p->c_out_pad, c_a, p->tail, true);
        c_b.assign((size_t)p->c_out_pad, 0);
        if (umma_narrow(d)) {
            p->epi = EPI_NARROW;
            p->tail = 1;
            for (int co = 0; co < d.c_out; ++co) c_a[co] = d.bias[co];
        }
    }
    p->group_uniform = d.out_dtype != ICONV_I32 && group_uniform(d) ? 1 : 0;
    window_plan(p);
    if (p->window) {
        CUtensorMap probe2;     // the tiled patch map must be encodable as well
        if (encode_patch_map(p, p->w_packed, &probe2) != ICONV_OK) p->window = 0;
    }
    // Long reductions (one 128-byte k-iteration per stage, the B tile riding in the stage) run on CTA
    // pairs: per k-iteration a CTA then pulls its 128 pixel rows and HALF of the B tile through its own
    // L2 port (32 KB instead of 48 for 256 output channels), which is what bounds these layers, and the
    // stages are deeper.  Not with a forced single-CTA form, a fused projection or per-channel reads.
    p->pair = 0;
    if (!p->window && d.kernel != ICONV_KERNEL_UMMA_IM2COL && p->kc == 128 && p->kg == 1 && !p->resident_b && !d.proj_weights &&
        p->block_n % 32 == 0 && (p->epi == EPI_FAST || p->epi == EPI_FAST_SKIP8 || p->epi == EPI_SAFE || p->epi == EPI_SAFE_SKIP8) &&
        (long long)d.n * p->h_out * p->w_out > 2 * BLOCK_M) {
        const int b_tile = (p->block_n * p->kc + 1023) / 1024 * 1024;
        const int slot = BLOCK_M * p->kc + b_tile / 2;
        int st = p->pipe_room / slot;
        if (st > MAX_STAGES) st = MAX_STAGES;
        if (st >= 3) {
            p->pair = 1;
            p->stages = st;
            rc = umma_encode_weight_map(p);
            if (rc != ICONV_OK) return rc;
        }
    }
    if (p->group_uniform && !p->window) {
        // the im2col kernel reads per-channel parameters channel by channel
        p->group_uniform = 0;
        if (!d.proj_weights && p->epi != EPI_NARROW) p->epi = choose_epilogue(d, p->c_out_pad, c_a, p->tail, false);
    }
    std::vector<int32_t> par((size_t)5 * p->c_out_pad, 0);
    for (int co = 0; co < p->c_out_pad; ++co) {
        const int q = d.per_channel && co < d.c_out ? co : 0;
        par[co] = c_a[co];
        par[(size_t)4 * p->c_out_pad + co] = c_b[co];
        par[(size_t)p->c_out_pad + co] = d.out_dtype != ICONV_I32 ? d.mul[q] : 1;
        par[(size_t)2 * p->c_out_pad + co] = d.out_dtype != ICONV_I32 ? d.shift[q] : 1;
        par[(size_t)3 * p->c_out_pad + co] = d.out_dtype != ICONV_I32 ? d.h_i[q] : 0;
    }
    ICONV_CUDA_TRY(cudaMalloc((void **)&p->params_packed, par.size() * sizeof(int32_t)));
    ICONV_CUDA_TRY(cudaMemcpy(p->params_packed, par.data(), par.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    p->q_mul = d.out_dtype != ICONV_I32 ? d.mul[0] : 1;
    p->q_shift = d.out_dtype != ICONV_I32 ? d.shift[0] : 0;
    p->q_h = d.out_dtype != ICONV_I32 ? d.h_i[0] : 0;

    if (p->epi == EPI_NARROW && !p->window) {
        set_error("tensor-core path: a narrow or unaligned 8-bit output needs window mode");
        return ICONV_ERR_UNSUPPORTED;
    }
    if (p->pair16 && !p->window) {
        set_error("tensor-core path: paired taps need window mode");
        return ICONV_ERR_UNSUPPORTED;
    }
    return ICONV_OK;
}

// Every TMA descriptor one launch of the layer needs, for these tensor addresses: the input
// (patch map in window mode, im2col map otherwise), the output rows and the skip rows (or the
// fused projection's input).
int encode_launch_maps(const iconv_plan_t *p, const void *x, const void *skip, void *out, CUtensorMap *tmap_x, CUtensorMap *tmap_out,
                       CUtensorMap *tmap_skip)
{
    const iconv_desc &d = p->d;
    int rc = p->window ? encode_patch_map(p, x, tmap_x) : encode_activation_map(p, x, tmap_x);
    if (rc != ICONV_OK) return rc;
    const long long m_total = (long long)d.n * p->h_out * p->w_out;
    const int esz = d.out_dtype == ICONV_I32 ? 4 : 1;
    memset(tmap_out, 0, sizeof(*tmap_out));
    if (!p->window) {       // window mode stores from registers
        rc = encode_rows_map((uint8_t *)out + (size_t)d.out_c_offset * esz, esz, d.c_out, d.out_c_total, m_total, p->piece_bytes, tmap_out);
        if (rc != ICONV_OK) return rc;
    }
    *tmap_skip = *tmap_out;
    if (p->epi == EPI_PROJ) {
        rc = encode_projection_map(p, skip, tmap_skip);      // the slot of the skip map carries the projection's input
        if (rc != ICONV_OK) return rc;
    }
    if (!p->window && (p->epi == EPI_FAST_SKIP8 || p->epi == EPI_SAFE_SKIP8)) {
        rc = encode_rows_map((const uint8_t *)skip + d.skip_c_offset, 1, d.c_out, d.skip_c_total, m_total, p->piece_bytes, tmap_skip);
        if (rc != ICONV_OK) return rc;
    }
    return ICONV_OK;
}

int umma_encode_2d(CUtensorMap *map, const void *base, long long inner, long long rows, long long row_stride, int box_inner, int box_rows, int swizzle)
{
    const int rc = load_driver_entry_points();
    if (rc != ICONV_OK) return rc;
    const cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_stride};
    const cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapSwizzle sw = swizzle == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : swizzle == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                  : swizzle == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
    const CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void *)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled (2-D map) failed with %d", (int)r); return ICONV_ERR_UNSUPPORTED; }
    return ICONV_OK;
}

// ICONV_OK when every descriptor of a launch on these addresses can be encoded (nothing is enqueued).
int umma_check_maps(const iconv_plan_t *p, const void *x, void *out)
{
    if (((uintptr_t)x % 16) || ((uintptr_t)out % 16)) { set_error("tensor pointers must be 16-byte aligned"); return ICONV_ERR_ALIGN; }
    const int rc = umma_init_once();
    if (rc != ICONV_OK) return rc;
    CUtensorMap mx, mo, ms;
    return encode_launch_maps(p, x, out, out, &mx, &mo, &ms);
}

int launch_umma(const iconv_plan_t *p, const ConvArgs &a, cudaStream_t stream)
{
    const iconv_desc &d = p->d;
    if (((uintptr_t)a.x % 16) || ((uintptr_t)a.out % 16) || (a.skip && ((uintptr_t)a.skip % 16))) {
        set_error("iconv_forward: tensor pointers must be 16-byte aligned");
        return ICONV_ERR_ALIGN;
    }
    CUtensorMap tmap_x, tmap_out, tmap_skip;
    int rc = encode_launch_maps(p, a.x, a.skip, a.out, &tmap_x, &tmap_out, &tmap_skip);
    if (rc != ICONV_OK) return rc;

    UmmaArgs u;
    u.win_vw = p->win_vw; u.win_bw = p->win_bw; u.win_bh = p->win_bh; u.win_full_width = p->win_full_width; u.win_tpi = p->win_tpi;
    u.win_blocks = p->win_blocks;
    u.win_issuers = p->win_issuers;
    find_divisor((unsigned)(p->win_tpi > 0 ? p->win_tpi : 1), u.div_tpi_mul, u.div_tpi_shr);
    find_divisor((unsigned)(p->win_vw > 0 ? p->win_vw : 1), u.div_vw_mul, u.div_vw_shr);
    u.m_total = (long long)d.n * p->h_out * p->w_out;
    u.m_tiles = (int)((u.m_total + BLOCK_M - 1) / BLOCK_M);
    u.n_tiles = p->c_out_pad / p->block_n;
    u.block_n = p->block_n;
    u.kc = p->kc;
    u.cchunks = p->c_in_pad / p->kc;
    u.taps = plan_taps(p);
    u.win_tap_step = p->pair16 ? 2 : 1;
    u.p_iters = p->proj_iters;
    u.p_taps = p->proj_iters ? d.proj_k * d.proj_k : 0;
    u.p_cchunks = p->proj_iters ? p->proj_c_in_pad / p->kc : 0;
    u.p_kw = d.proj_k;
    u.p_stride = d.proj_stride;
    u.p_pad = d.proj_pad;
    u.proj32 = p->proj32;
    u.stages = p->stages;
    u.kg = p->kg;
    u.slot_a_bytes = BLOCK_M * p->kc;
    u.b_tile_bytes = (p->block_n * p->kc + 1023) / 1024 * 1024;
    u.resident_b = p->resident_b;
    u.slot_bytes = u.slot_a_bytes + (p->resident_b ? 0 : (p->pair ? u.b_tile_bytes / 2 : u.b_tile_bytes));
    u.stage_bytes = u.kg * u.slot_bytes;
    u.producers = p->stages * p->kg < NUM_PRODUCERS ? p->stages * p->kg : NUM_PRODUCERS;
    u.nbuf = p->window ? p->win_nbuf : p->nbuf;
    u.lg_nbuf = u.nbuf == 8 ? 3 : u.nbuf == 4 ? 2 : 1;
    int cols = 32;
    u.acc_cols = p->block_n * (p->proj_iters ? 2 : 1);
    while (cols < u.nbuf * u.acc_cols) cols *= 2;
    u.tmem_cols = cols;
    u.epi_warps = p->epi_warps;
    u.cs = p->cs;
    u.bi = p->bi;
    u.part_n = p->half_n;
    u.piece_bytes = p->piece_bytes;
    u.epi_warp_bytes = p->epi_warp_bytes;
    u.skip_ring = p->skip_ring;
    // instruction descriptor: D = s32, A = u8 or s8, B = s8, both K-major, N/8, M/16
    u.idesc = (2u << 4) | ((d.in_dtype == ICONV_S8 ? 1u : 0u) << 7) | (1u << 10) | ((unsigned)(p->block_n >> 3) << 17) |
              ((unsigned)((p->pair ? 2 * BLOCK_M : BLOCK_M) >> 4) << 24);      // pairs: one instruction spans both CTAs' rows (M = 256)
    u.idesc_p = (u.idesc & ~(7u << 7)) | ((d.skip_dtype == ICONV_S8 ? 1u : 0u) << 7);
    // matrix descriptor, upper half: stride between 8-row groups (8 * KC bytes, in 16-byte
    // units), descriptor version 1, swizzle mode (128B = 2, 64B = 4, 32B = 6)
    const unsigned long long layout = p->kc == 128 ? 2ull : (p->kc == 64 ? 4ull : 6ull);
    u.desc_hi = ((unsigned long long)((8 * p->kc) >> 4) << 32) | (1ull << 46) | (layout << 61);
    u.desc_hi_a = (unsigned)((((unsigned long long)((p->win_bw * p->kc) >> 4) << 32) | (1ull << 46) | (layout << 61)) >> 32);
    u.q_mul = p->q_mul;
    u.q_shift = p->q_shift;
    u.q_half = p->q_shift > 0 && p->q_shift <= 31 ? (int)(1u << (p->q_shift - 1)) : 0;
    u.q_h = p->q_h;
    u.skip_half = (d.skip_dtype >= 0 && d.skip_shift > 0 && d.skip_shift <= 31) ? (int)(1u << (d.skip_shift - 1)) : 0;
    u.skip_xor = d.skip_dtype == ICONV_S8 ? 0x80808080u : 0u;
    u.tail = p->tail;
    u.group_uniform = p->group_uniform;
    u.c_a = p->params_packed;
    u.c_mul = p->params_packed + p->c_out_pad;
    u.c_shift = p->params_packed + 2 * (size_t)p->c_out_pad;
    u.c_h = p->params_packed + 3 * (size_t)p->c_out_pad;
    u.c_b = p->params_packed + 4 * (size_t)p->c_out_pad;
    find_divisor((unsigned)u.n_tiles, u.div_nt_mul, u.div_nt_shr);
    find_divisor((unsigned)p->w_out, u.div_w_mul, u.div_w_shr);
    find_divisor((unsigned)(p->h_out * p->w_out), u.div_hw_mul, u.div_hw_shr);
    u.status = device_status_ptr();
    if (!u.status) { set_error("device status word not available"); return ICONV_ERR_CUDA; }

    // shared-memory opt-in and SM count of the device this launch goes to (a plan made on one
    // device may run on another)
    rc = umma_init_once();
    if (rc != ICONV_OK) return rc;
    const int sms = g_device_init[current_device_slot()].sms;
    if (p->window) {
        u.m_tiles = p->win_tpi * d.n;
        u.stages = p->win_stages;
        u.stage_bytes = p->win_patch_bytes;
        const unsigned wgrid = (unsigned)(u.m_tiles < sms ? u.m_tiles : sms);
        const size_t wsmem = 1024 + (size_t)u.stages * u.stage_bytes + (size_t)u.b_tile_bytes * u.taps + sizeof(Shared);
        if (wsmem > (size_t)MAX_SMEM) { set_error("tensor-core path: shared-memory plan exceeds the limit"); return ICONV_ERR_UNSUPPORTED; }
        const UmmaLaunch l = {wgrid, wsmem, stream, &tmap_x, &p->tmap_w, &tmap_out, &tmap_skip, &a, &u, 1};
        const int wepi = (p->epi == EPI_FAST || p->epi == EPI_NARROW || p->epi == EPI_FAST_SKIP8 || p->epi == EPI_SAFE_SKIP8) ? p->epi : EPI_SAFE;
        ICONV_CUDA_TRY(umma_window_launch(wepi, d.kh, d.kw, p->kc >> 5, p->pair16, l));
        return ICONV_OK;
    }
    if (p->pair) u.m_tiles = (u.m_tiles + 1) / 2;                // pixel-tile pairs
    const long long tiles = (long long)u.m_tiles * u.n_tiles;
    unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    if (p->pair) grid = 2u * (unsigned)(tiles < sms / 2 ? tiles : sms / 2);     // clusters of two CTAs
    const size_t smem = 1024 + (size_t)u.stages * u.stage_bytes +
                        (p->resident_b ? (size_t)u.b_tile_bytes * (u.p_iters + u.taps * u.cchunks) * u.n_tiles : 0) + sizeof(Shared) + 1024 +
                        (size_t)p->epi_warps * p->epi_warp_bytes;
    if (smem > (size_t)MAX_SMEM) { set_error("tensor-core path: shared-memory plan exceeds the limit"); return ICONV_ERR_UNSUPPORTED; }
    const int kj_l = p->kc >> 5;
    const int issue = p->pair ? 3 : (kj_l == 4 && p->kg == 1 && !p->resident_b) ? 1
                      : (kj_l == 4 && p->resident_b && u.p_iters + u.taps * u.cchunks <= p->kg && u.p_iters == 0) ? 2 : 0;
    const UmmaLaunch l = {grid, smem, stream, &tmap_x, &p->tmap_w, &tmap_out, &tmap_skip, &a, &u, p->pair ? 2 : 1};
    ICONV_CUDA_TRY(umma_conv_launch(p->epi >= EPI_WIDE && p->epi <= EPI_PROJ ? p->epi : EPI_WIDE, issue, l));
    return ICONV_OK;
}

int launch_wait_selftest(int which, long long limit_cycles, cudaStream_t stream)
{
    int *status = device_status_ptr();
    if (!status) { set_error("device status word not available"); return ICONV_ERR_CUDA; }
    wait_timeout_selftest_kernel<<<1, 64, 0, stream>>>(which, limit_cycles, status);
    ICONV_CUDA_TRY(cudaGetLastError());
    return ICONV_OK;
}

}  // namespace iconv
