// The stem: a 7x7 stride-2 pad-3 convolution over a 3-channel image (the first layer of
// the ResNet-shaped networks).  Three channels are far too narrow for TMA (16-byte rows at
// least) and K = 147 is awkward for the tensor cores, so the layer runs in two steps:
//
//   1. a repack kernel rewrites the image as T[n][Y][X][16]: a 2x2 space-to-depth, which
//      turns the stride-2 7x7 filter into a stride-1 4x4 filter over 12 channels (padded to
//      16), with the re-normalisation (raw - 128, Section 3.4.1) and the zero padding applied
//      on the way:   T[n][Y][X][(dy*2+dx)*3 + c] = in[n][2(Y-2)+dy][2(X-2)+dx][c]
//   2. the tensor-core kernel runs a 4x4, 16-channel, stride-1, unpadded convolution on T
//      (in window mode: one patch of T per tile) with weights rearranged the same way:
//      out(oh, ow) = sum_{R,S} T[oh+R][ow+S] . W'[R][S],  W'[R][S][(dy*2+dx)*3+c] = W[2R+dy-1][2S+dx-1][c].
//
// The sum is the same integers in another order, so the result is bit-identical.
//
// A single-channel image under a stride-1 kh x kw filter (the first layer of the regression
// networks) takes the same two steps with another repack: T[n][Y][x][j] = in[n][Y-pad][x-pad+j],
// j < kw (the kw input bytes an output column needs, side by side as "channels"), after which
// the layer is a kh x 1 filter over 16 channels: out(oh, ow) = sum_r T[oh+r][ow] . W'[r],
// W'[r][j] = W[r][j].  Sixteen bytes per position instead of one, but the arithmetic moves
// to the tensor cores and the CUDA cores keep only the epilogue.
#include <atomic>
#include <cstring>
#include <vector>

#include "plan.h"

namespace iconv {

namespace {

// One thread writes the 16 bytes of one position (n, Y, X) of T.  The six input bytes of one image row
// that a position holds (two pixels x three channels) are contiguous and start on an even address:
// three 16-bit loads where both pixels are inside the image, byte loads at a ragged right edge.
__global__ void __launch_bounds__(256)
stem_repack_kernel(const uint8_t *__restrict__ in, uint8_t *__restrict__ T, int n, int h, int w, int hp, int wp,
                   int raw128, int slack)
{
    const unsigned total = (unsigned)n * (unsigned)hp * (unsigned)wp;     // < 2^31 (checked by the caller)
    const unsigned flip = raw128 ? 0x8080u : 0u;                           // raw - 128 as int8
    for (unsigned pos = blockIdx.x * blockDim.x + threadIdx.x; pos < total; pos += gridDim.x * blockDim.x) {
        const unsigned row = pos / (unsigned)wp;
        const int X = (int)(pos - row * (unsigned)wp);
        const unsigned img = row / (unsigned)hp;
        const int Y = (int)(row - img * (unsigned)hp);
        unsigned hw[6] = {0, 0, 0, 0, 0, 0};          // the twelve bytes as six 16-bit halves
        const int iw = 2 * (X - 2);
#pragma unroll
        for (int dy = 0; dy < 2; ++dy) {
            const int ih = 2 * (Y - 2) + dy;
            if (ih < 0 || ih >= h || iw < 0 || iw >= w) continue;            // zero padding (iw is even: iw < 0 puts both pixels outside)
            const uint8_t *p = in + (((size_t)img * h + ih) * w + iw) * 3;
            if (iw + 1 < w && ((uintptr_t)p & 1) == 0) {
                const unsigned short *q = (const unsigned short *)p;
                hw[dy * 3] = (unsigned)__ldg(q) ^ flip;
                hw[dy * 3 + 1] = (unsigned)__ldg(q + 1) ^ flip;
                hw[dy * 3 + 2] = (unsigned)__ldg(q + 2) ^ flip;
            } else {                          // rows of an odd width that start on an odd address, and their last pixel
                const unsigned f = flip & 0xffu;
                hw[dy * 3] = ((unsigned)p[0] ^ f) | (((unsigned)p[1] ^ f) << 8);
                hw[dy * 3 + 1] = (unsigned)p[2] ^ f;
                if (iw + 1 < w) {
                    hw[dy * 3 + 1] |= ((unsigned)p[3] ^ f) << 8;
                    hw[dy * 3 + 2] = ((unsigned)p[4] ^ f) | (((unsigned)p[5] ^ f) << 8);
                }
            }
        }
        *(uint4 *)(T + (size_t)pos * 16) = make_uint4(hw[0] | (hw[1] << 16), hw[2] | (hw[3] << 16), hw[4] | (hw[5] << 16), 0u);
        if (slack && pos == total - 1) *(uint4 *)(T + (size_t)total * 16) = make_uint4(0, 0, 0, 0);   // the 16 bytes of slack behind T
    }
}

// One thread writes the 16 bytes of one position (n, Y, x) of T for a single-channel image:
// bytes 0 .. kw-1 are in[n][Y - pad][x - pad + j] (0 outside the image), the rest 0.
__global__ void __launch_bounds__(256)
rows_repack_kernel(const uint8_t *__restrict__ in, uint8_t *__restrict__ T, int n, int h, int w, int hp, int wo, int pad, int kw,
                   int raw128)
{
    const long long total = (long long)n * hp * wo;
    for (long long pos = (long long)blockIdx.x * blockDim.x + threadIdx.x; pos < total;
         pos += (long long)gridDim.x * blockDim.x) {
        const int x = (int)(pos % wo);
        const int Y = (int)((pos / wo) % hp);
        const int img = (int)(pos / ((long long)wo * hp));
        const int ih = Y - pad;
        unsigned wds[4] = {0, 0, 0, 0};
        if (ih >= 0 && ih < h) {
            const uint8_t *row = in + ((long long)img * h + ih) * w;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int iw = x - pad + j;
                if (j < kw && iw >= 0 && iw < w) {
                    unsigned v = row[iw];
                    if (raw128) v ^= 0x80u;                              // raw - 128 as int8
                    wds[j >> 2] |= v << (8 * (j & 3));
                }
            }
        }
        *(uint4 *)(T + pos * 16) = make_uint4(wds[0], wds[1], wds[2], wds[3]);
    }
}

// 1: the 7x7 stride-2 stem over 3 channels; 2: a stride-1 filter over a single-channel image
int stem_kind(const iconv_desc &d)
{
    if (d.c_in == 3 && d.in_c_total == 3 && d.in_c_offset == 0 && d.kh == 7 && d.kw == 7 && d.stride == 2 &&
        d.pad == 3 && d.c_out >= 16)
        return 1;
    if (d.c_in == 1 && d.in_c_total == 1 && d.in_c_offset == 0 && d.stride == 1 && d.kw <= 16 && d.kh * d.kw > 1 &&
        d.c_out >= 32 && d.skip_dtype < 0)
        return 2;
    return 0;
}

}  // namespace

int stem_supported(const iconv_plan_t *p)
{
    if (stem_kind(p->d)) return ICONV_OK;
    set_error("stem path: needs a 7x7 stride-2 pad-3 layer over a 3-channel tensor, or a stride-1 filter at most 16 wide "
              "over a single-channel tensor with at least 32 output channels and no skip");
    return ICONV_ERR_UNSUPPORTED;
}

namespace {

int rows_setup(iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    const int hp = d.h + 2 * d.pad, wo = p->w_out;
    std::vector<int8_t> w2((size_t)d.c_out * d.kh * 16, 0);
    for (int co = 0; co < d.c_out; ++co)
        for (int r = 0; r < d.kh; ++r)
            for (int s = 0; s < d.kw; ++s)
                w2[((size_t)co * d.kh + r) * 16 + s] = d.weights[((size_t)co * d.kh + r) * d.kw + s];
    iconv_desc in = d;
    in.h = hp;
    in.w = wo;
    in.c_in = 16;
    in.in_c_total = 16;
    in.in_c_offset = 0;
    in.kw = 1;
    in.stride = 1;
    in.pad = 0;
    in.in_dtype = d.in_dtype == ICONV_U8 ? ICONV_U8 : ICONV_S8;
    in.kernel = ICONV_KERNEL_UMMA;
    in.weights = w2.data();
    int rc = iconv_plan(&in, &p->inner);
    if (rc != ICONV_OK) return rc;
    if (!p->inner->window) {
        // only worth the repack when the layer then runs from one patch per tile
        iconv_plan_destroy(p->inner);
        p->inner = nullptr;
        set_error("stem path: the repacked single-channel layer does not fit the tensor-core window mode");
        return ICONV_ERR_UNSUPPORTED;
    }
    p->workspace_bytes = (size_t)d.n * hp * wo * 16;
    return ICONV_OK;
}

}  // namespace

int stem_setup(iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    if (stem_kind(d) == 2) return rows_setup(p);
    const int hp = p->h_out + 3, wp = p->w_out + 3;
    // W'[co][R][S][(dy*2+dx)*3 + c] = W[co][2R+dy-1][2S+dx-1][c]  (0 where an index is -1)
    std::vector<int8_t> w2((size_t)d.c_out * 16 * 16, 0);
    for (int co = 0; co < d.c_out; ++co)
        for (int R = 0; R < 4; ++R)
            for (int S = 0; S < 4; ++S)
                for (int dy = 0; dy < 2; ++dy)
                    for (int dx = 0; dx < 2; ++dx) {
                        const int r = 2 * R + dy - 1, s = 2 * S + dx - 1;
                        if (r < 0 || s < 0) continue;
                        for (int c = 0; c < 3; ++c)
                            w2[(((size_t)co * 4 + R) * 4 + S) * 16 + (dy * 2 + dx) * 3 + c] =
                                d.weights[(((size_t)co * 7 + r) * 7 + s) * 3 + c];
                    }
    iconv_desc in = d;
    in.h = hp;
    in.w = wp;
    in.c_in = 16;
    in.in_c_total = 16;
    in.in_c_offset = 0;
    in.kh = 4;
    in.kw = 4;
    in.stride = 1;
    in.pad = 0;
    in.in_dtype = d.in_dtype == ICONV_U8 ? ICONV_U8 : ICONV_S8;
    in.kernel = ICONV_KERNEL_UMMA;
    in.weights = w2.data();
    // two horizontally adjacent taps per K step where the driver accepts the overlapping view
    // of T (half the MMAs); T gets 16 bytes of slack for the last position's neighbour
    int rc = plan_create(&in, 1, &p->inner);
    if (rc != ICONV_OK) rc = iconv_plan(&in, &p->inner);
    if (rc != ICONV_OK) return rc;
    // (the slack is only ever the right-hand neighbour of the last position, which no real output
    // pixel reads; the repack kernel zeroes it so that the workspace holds no stale bytes)
    p->workspace_bytes = (size_t)d.n * hp * wp * 16 + 16;
    return ICONV_OK;
}

int launch_stem(const iconv_plan_t *p, const ConvArgs &a, void *workspace, cudaStream_t stream)
{
    const iconv_desc &d = p->d;
    if (stem_kind(d) == 2) {
        const int hp = d.h + 2 * d.pad, wo = p->w_out;
        const long long total = (long long)d.n * hp * wo;
        long long blocks = (total + 255) / 256;
        if (blocks > 148ll * 32) blocks = 148ll * 32;
        if (blocks > 0)
            rows_repack_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const uint8_t *)a.x, (uint8_t *)workspace, d.n, d.h, d.w, hp, wo,
                                                                     d.pad, d.kw, d.in_dtype == ICONV_U8_RAW128);
        ICONV_CUDA_TRY(cudaGetLastError());
        return iconv_forward(p->inner, workspace, a.skip, a.out, nullptr, (void *)stream);
    }
    const int hp = p->h_out + 3, wp = p->w_out + 3;
    const long long total = (long long)d.n * hp * wp;
    if (total >= (1ll << 31)) { set_error("first-layer repack: more than 2^31 positions"); return ICONV_ERR_SHAPE; }
    long long blocks = (total + 255) / 256;
    if (blocks > 148ll * 32) blocks = 148ll * 32;
    stem_repack_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const uint8_t *)a.x, (uint8_t *)workspace, d.n, d.h, d.w,
                                                             hp, wp, d.in_dtype == ICONV_U8_RAW128, 1);
    ICONV_CUDA_TRY(cudaGetLastError());
    return iconv_forward(p->inner, workspace, a.skip, a.out, nullptr, (void *)stream);
}

}  // namespace iconv

// ---------------------------------------------------------------- allocation-free variant
//
// The same two steps for callers that may not allocate device memory (see iconv.h): the
// repacked image, the rearranged weights and the epilogue constants live in one file-scope
// device array instead of plan-owned buffers, and the caller hands in weights and bias that
// are already on the device.  In host code `g_stem_static` names a host-side stand-in of the
// array, not its device address: the address every kernel and TMA descriptor receives is the
// one cudaGetSymbolAddress returns, looked up once per device.
namespace iconv {

namespace {

constexpr size_t STEM_STATIC_W_BYTES = 128 * 1024;      // rearranged weights: 256 channels x 16 taps x 32 bytes
constexpr size_t STEM_STATIC_PAR_BYTES = 64 * 1024;     // {c_a, mul, shift, h_i} x 256 int32 (+ slack)
constexpr size_t STEM_STATIC_T_OFFSET = STEM_STATIC_W_BYTES + STEM_STATIC_PAR_BYTES;

static __device__ __align__(256) unsigned char g_stem_static[ICONV_STEM_STATIC_BYTES];

std::atomic<unsigned char *> g_stem_static_ptr[MAX_DEVICES];

// Device address of the array on the current device (looked up on the first call per device).
int stem_static_base(unsigned char **base)
{
    const int dev = current_device_slot();
    if (dev < 0) { set_error("iconv_stem_forward_static: no current device, or its index is beyond %d", MAX_DEVICES - 1); return ICONV_ERR_UNSUPPORTED; }
    unsigned char *ptr = g_stem_static_ptr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        ICONV_CUDA_TRY(cudaGetSymbolAddress((void **)&ptr, g_stem_static));
        if (!ptr) { set_error("iconv_stem_forward_static: the scratch array has no device address"); return ICONV_ERR_CUDA; }
        g_stem_static_ptr[dev].store(ptr, std::memory_order_release);
    }
    *base = ptr;
    return ICONV_OK;
}

// Writes W'[co][R][S][(dy*2+dx)*3 + c] = W[co][2R+dy-1][2S+dx-1][c], 32 bytes per tap (0 where an index is
// -1, in the padding lanes and in the padded channels) and the epilogue constants.  Every
// byte the GEMM reads is written here, so the array's previous contents never matter.
__global__ void __launch_bounds__(256)
stem_static_prepare_kernel(const int8_t *__restrict__ w, const int32_t *__restrict__ bias, int8_t *__restrict__ w2,
                           int32_t *__restrict__ par, int c_out, int c_out_pad, int mul, int shift, int h_i, int *status)
{
    const int total = c_out_pad * 512;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const int k = e & 31, S = (e >> 5) & 3, R = (e >> 7) & 3, co = e >> 9;
        int8_t v = 0;
        if (co < c_out && k < 12) {
            const int tap = k / 3, c = k - 3 * tap;
            const int r = 2 * R + (tap >> 1) - 1, s = 2 * S + (tap & 1) - 1;
            if (r >= 0 && s >= 0) v = w[((co * 7 + r) * 7 + s) * 3 + c];
        }
        w2[e] = v;
        if (e < c_out_pad) {
            int b = e < c_out ? bias[e] : 0;
            if (b > (1 << 30) || b < -(1 << 30)) { atomicCAS(status, 0, 8); b = 0; }   // U + b must stay inside int32
            par[e] = b;
            par[c_out_pad + e] = mul;
            par[2 * c_out_pad + e] = shift;
            par[3 * c_out_pad + e] = h_i;
        }
    }
}

}  // namespace

}  // namespace iconv

using namespace iconv;

extern "C" int iconv_stem_forward_static(const istem_desc *sd, const void *x, const int8_t *weights, const int32_t *bias,
                                         void *out, void *cuda_stream)
{
    if (!sd) { set_error("iconv_stem_forward_static: null descriptor"); return ICONV_ERR_ARG; }
    if (sd->n < 0 || sd->h < 1 || sd->w < 1 || sd->c_out < 16 || sd->c_out > 256 || sd->c_out % 16) {
        set_error("iconv_stem_forward_static: need n >= 0, h, w >= 1 and c_out a multiple of 16 in [16, 256]");
        return ICONV_ERR_ARG;
    }
    if (!(sd->in_dtype == ICONV_U8 || sd->in_dtype == ICONV_S8 || sd->in_dtype == ICONV_U8_RAW128)) {
        set_error("iconv_stem_forward_static: in_dtype must be U8, S8 or U8_RAW128");
        return ICONV_ERR_ARG;
    }
    if (sd->out_c_offset < 0 || sd->out_c_offset + sd->c_out > sd->out_c_total || sd->out_c_total % 16 || sd->out_c_offset % 16) {
        set_error("iconv_stem_forward_static: output slice outside its tensor or not a multiple of 16 channels");
        return ICONV_ERR_SHAPE;
    }
    if (sd->mul < 1 || sd->shift < 1 || sd->shift > 31 || sd->h_i < 0 || sd->out_lo > sd->out_hi || sd->out_lo < 0 || sd->out_hi > 255 ||
        (unsigned long long)sd->h_i * (unsigned long long)sd->mul + (1ull << (sd->shift - 1)) >= (1ull << 32)) {
        set_error("iconv_stem_forward_static: need mul >= 1, 1 <= shift <= 31, h_i * mul + 2^(shift-1) < 2^32, 0 <= out_lo <= out_hi <= 255");
        return ICONV_ERR_ARG;
    }
    const int h_out = (sd->h + 6 - 7) / 2 + 1, w_out = (sd->w + 6 - 7) / 2 + 1;
    const int hp = h_out + 3, wp = w_out + 3;
    const unsigned long long t_bytes = (unsigned long long)sd->n * hp * wp * 16ull;
    if (STEM_STATIC_T_OFFSET + t_bytes > (unsigned long long)ICONV_STEM_STATIC_BYTES) {
        set_error("iconv_stem_forward_static: %d images of %d x %d need %llu bytes of scratch, the static array holds %llu",
                  sd->n, sd->h, sd->w, STEM_STATIC_T_OFFSET + t_bytes, (unsigned long long)ICONV_STEM_STATIC_BYTES);
        return ICONV_ERR_SHAPE;
    }
    if (sd->n == 0) return ICONV_OK;
    if (!x || !weights || !bias || !out) { set_error("iconv_stem_forward_static: null tensor pointer"); return ICONV_ERR_ARG; }
    if (((uintptr_t)x % 16) || ((uintptr_t)out % 16)) { set_error("iconv_stem_forward_static: x and out must be 16-byte aligned"); return ICONV_ERR_ALIGN; }

    unsigned char *base = nullptr;
    int rc = stem_static_base(&base);
    if (rc != ICONV_OK) return rc;
    rc = umma_init_once();
    if (rc != ICONV_OK) return rc;
    int *status = device_status_ptr();
    if (!status) { set_error("device status word not available"); return ICONV_ERR_CUDA; }
    int8_t *w2 = (int8_t *)base;
    int32_t *par = (int32_t *)(base + STEM_STATIC_W_BYTES);
    uint8_t *T = base + STEM_STATIC_T_OFFSET;
    cudaStream_t stream = (cudaStream_t)cuda_stream;

    // a plan that lives on this call's stack and owns nothing: the GEMM over T
    iconv_plan_s tmp;
    iconv_desc &d = tmp.d;
    memset(&d, 0, sizeof(d));
    d.n = sd->n; d.h = hp; d.w = wp; d.c_in = 16; d.c_out = sd->c_out; d.kh = 4; d.kw = 4; d.stride = 1; d.pad = 0;
    d.in_dtype = sd->in_dtype == ICONV_U8 ? ICONV_U8 : ICONV_S8; d.in_c_total = 16; d.in_c_offset = 0;
    d.out_dtype = ICONV_U8; d.out_c_total = sd->out_c_total; d.out_c_offset = sd->out_c_offset;
    d.brelu = 1; d.per_channel = 0; d.out_lo = sd->out_lo; d.out_hi = sd->out_hi; d.out_zero = sd->out_zero;
    d.skip_dtype = -1; d.kernel = ICONV_KERNEL_UMMA;
    tmp.h_out = h_out; tmp.w_out = w_out; tmp.kernel = ICONV_KERNEL_UMMA;
    rc = umma_geometry(&tmp);
    if (rc != ICONV_OK) return rc;
    if ((size_t)tmp.c_out_pad * 16 * tmp.c_in_pad > STEM_STATIC_W_BYTES || tmp.c_in_pad != 32 || (size_t)tmp.c_out_pad * 20 > STEM_STATIC_PAR_BYTES) {
        set_error("iconv_stem_forward_static: channel count beyond the static array's weight region");
        return ICONV_ERR_SHAPE;
    }
    tmp.w_packed = w2;
    rc = umma_encode_weight_map(&tmp);
    if (rc == ICONV_OK) {
        tmp.params_packed = par;
        tmp.epi = umma_epilogue_safe();      // explicit clamps: no bound on the weights is known on the host
        tmp.tail = 1;
        tmp.q_mul = sd->mul; tmp.q_shift = sd->shift; tmp.q_h = sd->h_i;
        window_plan(&tmp);                   // one patch of T per tile where the geometry allows
        rc = umma_check_maps(&tmp, T, out);  // every descriptor the launch will need, before anything is enqueued
    }
    if (rc == ICONV_OK) {
        stem_static_prepare_kernel<<<(tmp.c_out_pad * 512 + 255) / 256, 256, 0, stream>>>(weights, bias, w2, par, sd->c_out, tmp.c_out_pad,
                                                                                    sd->mul, sd->shift, sd->h_i, status);
        const long long total = (long long)sd->n * hp * wp;
        long long blocks = (total + 255) / 256;
        if (blocks > 148ll * 32) blocks = 148ll * 32;
        stem_repack_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const uint8_t *)x, T, sd->n, sd->h, sd->w, hp, wp,
                                                                 sd->in_dtype == ICONV_U8_RAW128, 0);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) rc = cuda_fail(e, "iconv_stem_forward_static launches");
    }
    if (rc == ICONV_OK) {
        ConvArgs a;
        memset(&a, 0, sizeof(a));
        a.x = T; a.skip = nullptr; a.out = out;
        a.w = w2; a.bias = par; a.mul = par + tmp.c_out_pad; a.shift = par + 2 * tmp.c_out_pad; a.h_i = par + 3 * tmp.c_out_pad;
        a.n = d.n; a.h = d.h; a.w_ = d.w; a.c_in = 16; a.c_out = d.c_out; a.kh = 4; a.kw = 4; a.stride = 1; a.pad = 0;
        a.h_out = h_out; a.w_out = w_out;
        a.in_dtype = d.in_dtype; a.in_c_total = 16; a.in_c_offset = 0;
        a.out_dtype = ICONV_U8; a.out_c_total = d.out_c_total; a.out_c_offset = d.out_c_offset;
        a.brelu = 1; a.per_channel = 0; a.out_lo = d.out_lo; a.out_hi = d.out_hi; a.out_zero = d.out_zero;
        a.skip_dtype = -1; a.skip_mul = 1;
        rc = launch_umma(&tmp, a, stream);
    }
    // the stack plan owns nothing: keep its destructor-free fields from being mistaken for allocations
    tmp.w_packed = nullptr;
    tmp.params_packed = nullptr;
    return rc;
}
