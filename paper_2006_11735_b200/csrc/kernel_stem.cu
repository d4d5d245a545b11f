// The stem: a 7x7 stride-2 pad-3 convolution over a 3-channel image (the first layer of
// the ResNet-shaped networks).  Three channels are far too narrow for TMA (16-byte rows at
// least) and K = 147 is awkward for the tensor cores, so the layer runs in two steps:
//
//   1. a repack kernel rewrites the image as T[n][Y][X][64]: a 2x2 space-to-depth (which
//      turns the stride-2 7x7 filter into a stride-1 4x4 filter over 12 channels, padded to
//      16) with the four filter columns of every output position laid side by side, and
//      the re-normalisation (raw - 128, Section 3.4.1) and the zero padding applied on the
//      way:   T[n][Y][X][S*16 + (dy*2+dx)*3 + c] = in[n][2(Y-2)+dy][2(X+S-2)+dx][c]
//   2. the tensor-core kernel runs a kh=4, kw=1, c_in=64, stride-1, unpadded convolution on
//      T with weights rearranged the same way: out(oh, ow) = sum_R T[oh+R][ow] . W'[R].
//
// The sum is the same integers in another order, so the result is bit-identical.
#include <vector>

#include "plan.h"

namespace iconv {

namespace {

// One thread writes 16 bytes: position (n, Y, X) and filter column S of T.
__global__ void __launch_bounds__(256)
stem_repack_kernel(const uint8_t *__restrict__ in, uint8_t *__restrict__ T, int n, int h, int w, int hp, int wp,
                   int raw128)
{
    const long long total = (long long)n * hp * wp * 4;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int S = (int)(e & 3);
        const long long pos = e >> 2;
        const int X = (int)(pos % wp);
        const int Y = (int)((pos / wp) % hp);
        const int img = (int)(pos / ((long long)wp * hp));
        unsigned wds[4] = {0, 0, 0, 0};
#pragma unroll
        for (int dy = 0; dy < 2; ++dy) {
            const int ih = 2 * (Y - 2) + dy;
#pragma unroll
            for (int dx = 0; dx < 2; ++dx) {
                const int iw = 2 * (X + S - 2) + dx;
                if (ih < 0 || ih >= h || iw < 0 || iw >= w) continue;    // zero padding
                const uint8_t *p = in + (((long long)img * h + ih) * w + iw) * 3;
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    const int k = (dy * 2 + dx) * 3 + c;
                    unsigned v = p[c];
                    if (raw128) v ^= 0x80u;                              // raw - 128 as int8
                    wds[k >> 2] |= v << (8 * (k & 3));
                }
            }
        }
        *(uint4 *)(T + pos * 64 + S * 16) = make_uint4(wds[0], wds[1], wds[2], wds[3]);
    }
}

}  // namespace

int stem_supported(const iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    if (d.c_in == 3 && d.in_c_total == 3 && d.in_c_offset == 0 && d.kh == 7 && d.kw == 7 && d.stride == 2 &&
        d.pad == 3 && d.c_out >= 16)
        return ICONV_OK;
    set_error("stem path: needs a 7x7 stride-2 pad-3 layer over a 3-channel tensor");
    return ICONV_ERR_UNSUPPORTED;
}

int stem_setup(iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    const int hp = p->h_out + 3, wp = p->w_out;
    // W'[co][R][0][S*16 + (dy*2+dx)*3 + c] = W[co][2R+dy-1][2S+dx-1][c]  (0 where an index is -1)
    std::vector<int8_t> w2((size_t)d.c_out * 4 * 64, 0);
    for (int co = 0; co < d.c_out; ++co)
        for (int R = 0; R < 4; ++R)
            for (int S = 0; S < 4; ++S)
                for (int dy = 0; dy < 2; ++dy)
                    for (int dx = 0; dx < 2; ++dx) {
                        const int r = 2 * R + dy - 1, s = 2 * S + dx - 1;
                        if (r < 0 || s < 0) continue;
                        for (int c = 0; c < 3; ++c)
                            w2[((size_t)co * 4 + R) * 64 + S * 16 + (dy * 2 + dx) * 3 + c] =
                                d.weights[(((size_t)co * 7 + r) * 7 + s) * 3 + c];
                    }
    iconv_desc in = d;
    in.h = hp;
    in.w = wp;
    in.c_in = 64;
    in.in_c_total = 64;
    in.in_c_offset = 0;
    in.kh = 4;
    in.kw = 1;
    in.stride = 1;
    in.pad = 0;
    in.in_dtype = d.in_dtype == ICONV_U8 ? ICONV_U8 : ICONV_S8;
    in.kernel = ICONV_KERNEL_UMMA;
    in.weights = w2.data();
    int rc = iconv_plan(&in, &p->inner);
    if (rc != ICONV_OK) return rc;
    p->workspace_bytes = (size_t)d.n * hp * wp * 64;
    if (p->workspace_bytes) ICONV_CUDA_TRY(cudaMalloc(&p->workspace, p->workspace_bytes));
    return ICONV_OK;
}

int launch_stem(const iconv_plan_t *p, const ConvArgs &a, cudaStream_t stream)
{
    const iconv_desc &d = p->d;
    const int hp = p->h_out + 3, wp = p->w_out;
    const long long total = (long long)d.n * hp * wp * 4;
    long long blocks = (total + 255) / 256;
    if (blocks > 148ll * 32) blocks = 148ll * 32;
    stem_repack_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const uint8_t *)a.x, (uint8_t *)p->workspace, d.n, d.h, d.w,
                                                             hp, wp, d.in_dtype == ICONV_U8_RAW128);
    ICONV_CUDA_TRY(cudaGetLastError());
    return iconv_forward(p->inner, p->workspace, a.skip, a.out, (void *)stream);
}

}  // namespace iconv
