// CUDA-core kernels: the any-shape direct convolution (the path of last resort and the
// home of shapes no faster kernel takes), the stand-alone add-rescale, and the pooling
// layers of the ResNet-shaped networks.
#include "common.cuh"

namespace iconv {

__device__ __forceinline__ int dp4a_u8s8(unsigned a, int b, int c)
{
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ int dp4a_s8s8(int a, int b, int c)
{
    int d;
    asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// One thread per output element (pixel-major, channel fastest).  VEC: the channel slice of
// every pixel starts on a 4-byte boundary and c_in is a multiple of 4, so the reduction
// runs on dp4a; otherwise byte by byte.
template <int IN_DTYPE, bool VEC>
__global__ void __launch_bounds__(256) direct_conv_kernel(const __grid_constant__ ConvArgs a)
{
    const long long total = (long long)a.n * a.h_out * a.w_out * a.c_out;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int co = (int)(e % a.c_out);
        const long long pix = e / a.c_out;
        const int ow = (int)(pix % a.w_out);
        const int oh = (int)((pix / a.w_out) % a.h_out);
        const int n = (int)(pix / ((long long)a.w_out * a.h_out));
        int U = 0;
        for (int r = 0; r < a.kh; ++r) {
            const int ih = oh * a.stride - a.pad + r;
            if (ih < 0 || ih >= a.h) continue;
            for (int s = 0; s < a.kw; ++s) {
                const int iw = ow * a.stride - a.pad + s;
                if (iw < 0 || iw >= a.w_) continue;
                const long long xb = (((long long)n * a.h + ih) * a.w_ + iw) * a.in_c_total + a.in_c_offset;
                const long long wb = (((long long)co * a.kh + r) * a.kw + s) * a.c_in;
                if (VEC) {
                    const unsigned *xp = (const unsigned *)((const uint8_t *)a.x + xb);
                    const int *wp = (const int *)(a.w + wb);
                    for (int c4 = 0; c4 < a.c_in / 4; ++c4) {
                        unsigned xv = __ldg(xp + c4);
                        const int wv = __ldg(wp + c4);
                        if (IN_DTYPE == ICONV_U8) {
                            U = dp4a_u8s8(xv, wv, U);
                        } else {
                            if (IN_DTYPE == ICONV_U8_RAW128) xv ^= 0x80808080u;   // u8 - 128 as s8
                            U = dp4a_s8s8((int)xv, wv, U);
                        }
                    }
                } else {
                    for (int ci = 0; ci < a.c_in; ++ci) {
                        int xv;
                        if (IN_DTYPE == ICONV_S8) xv = ((const int8_t *)a.x)[xb + ci];
                        else xv = (int)((const uint8_t *)a.x)[xb + ci] - (IN_DTYPE == ICONV_U8_RAW128 ? 128 : 0);
                        U += xv * (int)a.w[wb + ci];
                    }
                }
            }
        }
        long long Y = (long long)U + a.bias[co];
        if (a.skip_dtype >= 0) {
            const int sv = load_skip(a.skip, pix * a.skip_c_total + a.skip_c_offset + co, a.skip_dtype);
            Y += round_shift64((long long)sv * a.skip_mul, a.skip_shift);
        }
        const long long oi = pix * a.out_c_total + a.out_c_offset + co;
        if (a.out_dtype == ICONV_I32) {
            ((int32_t *)a.out)[oi] = (int32_t)Y;
        } else {
            const int q = a.per_channel ? co : 0;
            const int V = requant_tail(Y, a.brelu, a.h_i[q], a.mul[q], a.shift[q], a.out_zero, a.out_lo, a.out_hi);
            if (a.out_dtype == ICONV_U8) ((uint8_t *)a.out)[oi] = (uint8_t)V;
            else ((int8_t *)a.out)[oi] = (int8_t)V;
        }
    }
}

int launch_direct(const ConvArgs &a, cudaStream_t stream)
{
    const long long total = (long long)a.n * a.h_out * a.w_out * a.c_out;
    if (total == 0) return ICONV_OK;
    const bool vec = (a.c_in % 4 == 0) && (a.in_c_total % 4 == 0) && (a.in_c_offset % 4 == 0) &&
                     (((uintptr_t)a.x) % 4 == 0) && (((uintptr_t)a.w) % 4 == 0);
    long long blocks = (total + 255) / 256;
    const long long cap = 148ll * 8 * 16;
    if (blocks > cap) blocks = cap;
#define LAUNCH(DT)                                                                         \
    if (vec) direct_conv_kernel<DT, true><<<(unsigned)blocks, 256, 0, stream>>>(a);        \
    else direct_conv_kernel<DT, false><<<(unsigned)blocks, 256, 0, stream>>>(a)
    switch (a.in_dtype) {
    case ICONV_U8: LAUNCH(ICONV_U8); break;
    case ICONV_S8: LAUNCH(ICONV_S8); break;
    default: LAUNCH(ICONV_U8_RAW128); break;
    }
#undef LAUNCH
    ICONV_CUDA_TRY(cudaGetLastError());
    return ICONV_OK;
}

// ---------------------------------------------------------------- add-rescale
__device__ __forceinline__ int load_elem(const void *p, long long i, int dtype)
{
    if (dtype == ICONV_U8) return ((const uint8_t *)p)[i];
    if (dtype == ICONV_S8) return ((const int8_t *)p)[i];
    return ((const int32_t *)p)[i];
}

// Loads 16 consecutive elements starting at i (a multiple of 16) with 16-byte accesses.
__device__ __forceinline__ void load16(const void *p, long long i, int dtype, int (&v)[16])
{
    if (dtype == ICONV_I32) {
        const int4 *q = (const int4 *)((const int32_t *)p + i);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int4 t = __ldg(q + k);
            v[4 * k] = t.x; v[4 * k + 1] = t.y; v[4 * k + 2] = t.z; v[4 * k + 3] = t.w;
        }
    } else {
        const uint4 t = __ldg((const uint4 *)((const uint8_t *)p + i));
        const unsigned wds[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const unsigned b = (wds[k >> 2] >> (8 * (k & 3))) & 0xffu;
            v[k] = dtype == ICONV_U8 ? (int)b : (int)(int8_t)b;
        }
    }
}

__device__ __forceinline__ int add_one(const iadd_desc &d, int av, int bv)
{
    const long long Y = round_shift64((long long)(av - d.a_zero) * d.mul_a, d.sh_a) +
                        round_shift64((long long)(bv - d.b_zero) * d.mul_b, d.sh_b);
    return requant_tail(Y, d.brelu, d.h_i, d.mul, d.shift, d.out_zero, d.out_lo, d.out_hi);
}

__global__ void __launch_bounds__(256) add_requant_kernel(const __grid_constant__ iadd_desc d, const void *A,
                                                          const void *B, void *out, int vec_ok)
{
    const long long groups = d.n_elems / 16;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nthreads = (long long)gridDim.x * blockDim.x;
    if (vec_ok) {
        for (long long g = tid; g < groups; g += nthreads) {
            int av[16], bv[16], ov[16];
            load16(A, g * 16, d.a_dtype, av);
            load16(B, g * 16, d.b_dtype, bv);
#pragma unroll
            for (int k = 0; k < 16; ++k) ov[k] = add_one(d, av[k], bv[k]);
            if (d.out_dtype == ICONV_I32) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    ((int4 *)((int32_t *)out + g * 16))[k] = make_int4(ov[4 * k], ov[4 * k + 1], ov[4 * k + 2], ov[4 * k + 3]);
            } else {
                unsigned wds[4];
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    wds[k] = (ov[4 * k] & 0xff) | ((ov[4 * k + 1] & 0xff) << 8) | ((ov[4 * k + 2] & 0xff) << 16) |
                             ((unsigned)(ov[4 * k + 3] & 0xff) << 24);
                *(uint4 *)((uint8_t *)out + g * 16) = make_uint4(wds[0], wds[1], wds[2], wds[3]);
            }
        }
    }
    // ragged tail (or everything when the pointers are not 16-byte aligned)
    for (long long i = (vec_ok ? groups * 16 : 0) + tid; i < d.n_elems; i += nthreads) {
        const int V = add_one(d, load_elem(A, i, d.a_dtype), load_elem(B, i, d.b_dtype));
        if (d.out_dtype == ICONV_I32) ((int32_t *)out)[i] = V;
        else if (d.out_dtype == ICONV_U8) ((uint8_t *)out)[i] = (uint8_t)V;
        else ((int8_t *)out)[i] = (int8_t)V;
    }
}

int launch_add_requant(const iadd_desc &d, const void *a, const void *b, void *out, cudaStream_t stream)
{
    if (d.n_elems == 0) return ICONV_OK;
    const int vec_ok = ((uintptr_t)a % 16 == 0) && ((uintptr_t)b % 16 == 0) && ((uintptr_t)out % 16 == 0);
    long long blocks = (d.n_elems / 16 + 255) / 256 + 1;
    if (blocks > 148ll * 32) blocks = 148ll * 32;
    add_requant_kernel<<<(unsigned)blocks, 256, 0, stream>>>(d, a, b, out, vec_ok);
    ICONV_CUDA_TRY(cudaGetLastError());
    return ICONV_OK;
}

// ---------------------------------------------------------------- pooling
// One thread per (output pixel, group of 16 channels): 16-byte loads, byte-wise unsigned max.
__global__ void __launch_bounds__(256) maxpool_kernel(const uint8_t *x, uint8_t *out, int n, int h, int w, int c,
                                                      int k, int stride, int pad, int h_out, int w_out)
{
    const int cg = c / 16;
    const long long total = (long long)n * h_out * w_out * cg;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int g = (int)(e % cg);
        const long long pix = e / cg;
        const int ow = (int)(pix % w_out);
        const int oh = (int)((pix / w_out) % h_out);
        const int in = (int)(pix / ((long long)w_out * h_out));
        uint4 m = make_uint4(0, 0, 0, 0);
        for (int r = 0; r < k; ++r) {
            const int ih = oh * stride - pad + r;
            if (ih < 0 || ih >= h) continue;
            for (int s = 0; s < k; ++s) {
                const int iw = ow * stride - pad + s;
                if (iw < 0 || iw >= w) continue;
                const uint4 v = __ldg((const uint4 *)(x + (((long long)in * h + ih) * w + iw) * c) + g);
                m.x = __vmaxu4(m.x, v.x); m.y = __vmaxu4(m.y, v.y);
                m.z = __vmaxu4(m.z, v.z); m.w = __vmaxu4(m.w, v.w);
            }
        }
        *((uint4 *)(out + pix * c) + g) = m;
    }
}

// The 3x3 stride-2 pad-1 pooling of the ResNet-shaped networks: the nine loads carry no branch
// (a tap outside the image re-reads the nearest row or column inside it, which the window
// holds anyway, so the maximum is unchanged) and are all in flight together; one thread per
// (output pixel, group of 16 channels), 32-bit index arithmetic.
__global__ void __launch_bounds__(256) maxpool_3x3s2_kernel(const uint8_t *__restrict__ x, uint8_t *__restrict__ out, unsigned total,
                                                            int h, int w, int cg, int h_out, int w_out)
{
    const unsigned e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= total) return;
    const unsigned pix = e / (unsigned)cg;
    const int g = (int)(e - pix * (unsigned)cg);
    const unsigned row = pix / (unsigned)w_out;               // image * h_out + oh
    const int ow = (int)(pix - row * (unsigned)w_out);
    const unsigned in = row / (unsigned)h_out;
    const int oh = (int)(row - in * (unsigned)h_out);
    const uint4 *base = (const uint4 *)x + (size_t)in * h * w * cg + g;
    uint4 v[9];
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int ih = min(max(2 * oh - 1 + r, 0), h - 1);
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            const int iw = min(max(2 * ow - 1 + s, 0), w - 1);
            v[r * 3 + s] = __ldg(base + (size_t)(ih * w + iw) * cg);
        }
    }
    uint4 m = v[0];
#pragma unroll
    for (int t = 1; t < 9; ++t) {
        m.x = __vmaxu4(m.x, v[t].x); m.y = __vmaxu4(m.y, v[t].y);
        m.z = __vmaxu4(m.z, v[t].z); m.w = __vmaxu4(m.w, v[t].w);
    }
    ((uint4 *)out)[e] = m;
}

int launch_maxpool(const void *x, void *out, int n, int h, int w, int c, int k, int stride, int pad,
                   cudaStream_t stream)
{
    const int h_out = (h + 2 * pad - k) / stride + 1, w_out = (w + 2 * pad - k) / stride + 1;
    const long long total = (long long)n * h_out * w_out * (c / 16);
    if (total == 0) return ICONV_OK;
    if (k == 3 && stride == 2 && pad == 1 && total < (1ll << 31) && (long long)n * h * w * (c / 16) < (1ll << 31)) {
        maxpool_3x3s2_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>((const uint8_t *)x, (uint8_t *)out, (unsigned)total, h, w,
                                                                                c / 16, h_out, w_out);
        ICONV_CUDA_TRY(cudaGetLastError());
        return ICONV_OK;
    }
    long long blocks = (total + 255) / 256;
    if (blocks > 148ll * 64) blocks = 148ll * 64;
    maxpool_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const uint8_t *)x, (uint8_t *)out, n, h, w, c, k, stride,
                                                         pad, h_out, w_out);
    ICONV_CUDA_TRY(cudaGetLastError());
    return ICONV_OK;
}

// One thread per (image, channel); consecutive threads take consecutive channels, so every
// pixel row is read coalesced.  Sum, then Eq. 4 and a clamp to [0, max_int].
__global__ void __launch_bounds__(256) avgpool_kernel(const uint8_t *x, uint8_t *out, int n, int hw, int c, int mul,
                                                      int shift, int max_int)
{
    const long long total = (long long)n * c;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int ch = (int)(e % c);
        const long long in = e / c;
        const uint8_t *p = x + in * hw * c + ch;
        long long sum = 0;
        for (int i = 0; i < hw; ++i) sum += p[(long long)i * c];
        long long V = round_shift64(sum * mul, shift);
        V = V < 0 ? 0 : (V > max_int ? max_int : V);
        out[e] = (uint8_t)V;
    }
}

// Sixteen channels per thread (16-byte loads, a warp reads 512 contiguous bytes of every pixel),
// byte lanes widened into 16 int sums; for channel counts that are multiples of 16 and 16-byte
// aligned tensors.  The sums stay far inside int32 (at most hw * 255).
__global__ void __launch_bounds__(128) avgpool16_kernel(const uint8_t *__restrict__ x, uint8_t *__restrict__ out, int n, int hw, int cg,
                                                        int mul, int shift, int max_int)
{
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n * cg) return;
    const int img = e / cg, g = e - img * cg;
    const uint4 *p = (const uint4 *)x + (size_t)img * hw * cg + g;
    int sum[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) sum[k] = 0;
#pragma unroll 7
    for (int i = 0; i < hw; ++i) {
        const uint4 v = __ldg(p + (size_t)i * cg);
        const unsigned wds[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 16; ++k) sum[k] += (int)((wds[k >> 2] >> (8 * (k & 3))) & 0xffu);
    }
    unsigned o[4] = {0, 0, 0, 0};
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        long long V = round_shift64((long long)sum[k] * mul, shift);
        V = V < 0 ? 0 : (V > max_int ? max_int : V);
        o[k >> 2] |= (unsigned)V << (8 * (k & 3));
    }
    ((uint4 *)out)[e] = make_uint4(o[0], o[1], o[2], o[3]);
}

int launch_avgpool(const void *x, void *out, int n, int h, int w, int c, int mul, int shift, int max_int,
                   cudaStream_t stream)
{
    const long long total = (long long)n * c;
    if (total == 0) return ICONV_OK;
    if (c % 16 == 0 && (uintptr_t)x % 16 == 0 && (uintptr_t)out % 16 == 0 && total / 16 < (1ll << 31) && max_int <= 255 &&
        (long long)h * w * 255 < (1ll << 31)) {
        const int groups = (int)(total / 16);
        avgpool16_kernel<<<(unsigned)((groups + 127) / 128), 128, 0, stream>>>((const uint8_t *)x, (uint8_t *)out, n, h * w, c / 16, mul,
                                                                             shift, max_int);
        ICONV_CUDA_TRY(cudaGetLastError());
        return ICONV_OK;
    }
    long long blocks = (total + 255) / 256;
    avgpool_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const uint8_t *)x, (uint8_t *)out, n, h * w, c, mul, shift,
                                                         max_int);
    ICONV_CUDA_TRY(cudaGetLastError());
    return ICONV_OK;
}

}  // namespace iconv
