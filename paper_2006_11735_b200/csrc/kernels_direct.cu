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

// The usual case in 32-bit arithmetic: 8-bit operands, an 8-bit result, and bounds (checked on the
// host from the descriptor alone) under which every product and sum below stays inside int32:
//   a' = (A * mul_a + ca) >> sh_a   with ca = 2^(sh_a-1) - a_zero * mul_a   (the zero point folded in)
//   b' likewise,  Y = a' + b',  clamp, V = (Y * mul + 2^(shift-1)) >> shift, zero point, saturation.
// Sixteen elements per thread and step, 16-byte accesses, two steps in flight per thread.
struct AddFast {
    int mul_a, ca, sh_a, mul_b, cb, sh_b;
    int y_lo, y_hi;          // BReLU's clamp, or the (unreachable) bounds of Y when there is none
    int mul, half, shift, out_zero, out_lo, out_hi;
    unsigned xor_a, xor_b;   // 0x80808080 turns int8 bytes into offset-binary (the offset rides in ca / cb)
    int out_signed;
};

__device__ __forceinline__ void add_fast16(const AddFast &f, uint4 ta, uint4 tb, uint4 &o)
{
    const unsigned wa[4] = {ta.x ^ f.xor_a, ta.y ^ f.xor_a, ta.z ^ f.xor_a, ta.w ^ f.xor_a};
    const unsigned wb[4] = {tb.x ^ f.xor_b, tb.y ^ f.xor_b, tb.z ^ f.xor_b, tb.w ^ f.xor_b};
    int V[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const int av = (int)__byte_perm(wa[k >> 2], 0, 0x4440 + (k & 3));
        const int bv = (int)__byte_perm(wb[k >> 2], 0, 0x4440 + (k & 3));
        int y = ((av * f.mul_a + f.ca) >> f.sh_a) + ((bv * f.mul_b + f.cb) >> f.sh_b);
        y = min(max(y, f.y_lo), f.y_hi);
        const int v = ((y * f.mul + f.half) >> f.shift) + f.out_zero;
        V[k] = min(max(v, f.out_lo), f.out_hi);
    }
    unsigned wds[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
        wds[k] = (V[4 * k] & 0xff) | ((V[4 * k + 1] & 0xff) << 8) | ((V[4 * k + 2] & 0xff) << 16) | ((unsigned)(V[4 * k + 3] & 0xff) << 24);
    o = make_uint4(wds[0], wds[1], wds[2], wds[3]);
}

__global__ void __launch_bounds__(256) add_requant_fast_kernel(const __grid_constant__ AddFast f, const uint4 *__restrict__ A,
                                                               const uint4 *__restrict__ B, uint4 *__restrict__ out, long long groups)
{
    const long long nthreads = (long long)gridDim.x * blockDim.x;
    long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    for (; g + nthreads < groups; g += 2 * nthreads) {
        const uint4 a0 = __ldcs(A + g), b0 = __ldcs(B + g), a1 = __ldcs(A + g + nthreads), b1 = __ldcs(B + g + nthreads);
        uint4 o0, o1;
        add_fast16(f, a0, b0, o0);
        add_fast16(f, a1, b1, o1);
        __stcs(out + g, o0);
        __stcs(out + g + nthreads, o1);
    }
    if (g < groups) {
        uint4 o0;
        add_fast16(f, __ldcs(A + g), __ldcs(B + g), o0);
        __stcs(out + g, o0);
    }
}

// Fills `f` and returns true when the 32-bit form is exact for every possible operand value.
static bool add_fast_plan(const iadd_desc &d, AddFast &f)
{
    const auto eight = [](int t) { return t == ICONV_U8 || t == ICONV_S8; };
    if (!eight(d.a_dtype) || !eight(d.b_dtype) || !eight(d.out_dtype)) return false;
    if (d.sh_a > 30 || d.sh_b > 30 || d.shift > 30) return false;
    const long long LIM = 1ll << 31;
    // stored byte as an unsigned number sv in [0, 255]; value = sv - z with z = zero (u8) or zero + 128 (offset-binary int8)
    const long long za = d.a_zero + (d.a_dtype == ICONV_S8 ? 128 : 0), zb = d.b_zero + (d.b_dtype == ICONV_S8 ? 128 : 0);
    const long long half_a = d.sh_a ? 1ll << (d.sh_a - 1) : 0, half_b = d.sh_b ? 1ll << (d.sh_b - 1) : 0, half = d.shift ? 1ll << (d.shift - 1) : 0;
    const long long ca = half_a - za * d.mul_a, cb = half_b - zb * d.mul_b;
    const auto mag = [](long long v) { return v < 0 ? -v : v; };
    if (mag(ca) + 255ll * d.mul_a >= LIM || mag(cb) + 255ll * d.mul_b >= LIM) return false;
    const long long a_lo = ca >> d.sh_a, a_hi = (255ll * d.mul_a + ca) >> d.sh_a, b_lo = cb >> d.sh_b, b_hi = (255ll * d.mul_b + cb) >> d.sh_b;
    long long y_lo = a_lo + b_lo, y_hi = a_hi + b_hi;
    if (d.brelu) { y_lo = 0; y_hi = d.h_i; }
    if (mag(y_lo) >= LIM || mag(y_hi) >= LIM) return false;
    if (mag(y_lo) * d.mul + half >= LIM || mag(y_hi) * d.mul + half >= LIM) return false;
    if (mag((long long)d.out_zero) >= (1ll << 30)) return false;
    f.mul_a = d.mul_a; f.ca = (int)ca; f.sh_a = d.sh_a; f.mul_b = d.mul_b; f.cb = (int)cb; f.sh_b = d.sh_b;
    f.y_lo = (int)y_lo; f.y_hi = (int)y_hi;
    f.mul = d.mul; f.half = (int)half; f.shift = d.shift; f.out_zero = d.out_zero; f.out_lo = d.out_lo; f.out_hi = d.out_hi;
    f.xor_a = d.a_dtype == ICONV_S8 ? 0x80808080u : 0u; f.xor_b = d.b_dtype == ICONV_S8 ? 0x80808080u : 0u;
    f.out_signed = d.out_dtype == ICONV_S8;
    return true;
}

int launch_add_requant(const iadd_desc &d, const void *a, const void *b, void *out, cudaStream_t stream)
{
    if (d.n_elems == 0) return ICONV_OK;
    const int vec_ok = ((uintptr_t)a % 16 == 0) && ((uintptr_t)b % 16 == 0) && ((uintptr_t)out % 16 == 0);
    AddFast f;
    if (vec_ok && d.n_elems >= 16 && add_fast_plan(d, f)) {
        const long long groups = d.n_elems / 16;
        long long fblocks = (groups + 511) / 512;                 // two groups per thread and round
        if (fblocks > 148ll * 16) fblocks = 148ll * 16;           // a whole number of waves: 8 resident blocks of 256 threads per SM
        if (fblocks < 1) fblocks = 1;
        add_requant_fast_kernel<<<(unsigned)fblocks, 256, 0, stream>>>(f, (const uint4 *)a, (const uint4 *)b, (uint4 *)out, groups);
        ICONV_CUDA_TRY(cudaGetLastError());
        const long long done = groups * 16;
        if (done == d.n_elems) return ICONV_OK;
        // the ragged tail (fewer than 16 elements) through the general kernel
        iadd_desc t = d;
        t.n_elems = d.n_elems - done;
        const size_t ea = 1, eo = 1;
        add_requant_kernel<<<1, 32, 0, stream>>>(t, (const uint8_t *)a + done * ea, (const uint8_t *)b + done * ea, (uint8_t *)out + done * eo, 0);
        ICONV_CUDA_TRY(cudaGetLastError());
        return ICONV_OK;
    }
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

// The same with 32 channels per thread (32-byte loads and one 32-byte store: half the memory
// instructions, every store a whole sector), for channel counts that are multiples of 32 and
// 32-byte aligned tensors.
struct Bytes32 {
    unsigned v[8];
};
__device__ __forceinline__ Bytes32 ld_global_32(const void *p)
{
    Bytes32 r;
    asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]), "=r"(r.v[4]), "=r"(r.v[5]), "=r"(r.v[6]), "=r"(r.v[7])
                 : "l"(p));
    return r;
}
__global__ void __launch_bounds__(256) maxpool_3x3s2_wide_kernel(const uint8_t *__restrict__ x, uint8_t *__restrict__ out, unsigned total,
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
    const uint8_t *base = x + ((size_t)in * h * w * cg + g) * 32;
    Bytes32 v[9];
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int ih = min(max(2 * oh - 1 + r, 0), h - 1);
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            const int iw = min(max(2 * ow - 1 + s, 0), w - 1);
            v[r * 3 + s] = ld_global_32(base + (size_t)(ih * w + iw) * cg * 32);
        }
    }
    Bytes32 m = v[0];
#pragma unroll
    for (int t = 1; t < 9; ++t)
#pragma unroll
        for (int k = 0; k < 8; ++k) m.v[k] = __vmaxu4(m.v[k], v[t].v[k]);
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(out + (size_t)e * 32), "r"(m.v[0]), "r"(m.v[1]), "r"(m.v[2]),
                 "r"(m.v[3]), "r"(m.v[4]), "r"(m.v[5]), "r"(m.v[6]), "r"(m.v[7])
                 : "memory");
}

int launch_maxpool(const void *x, void *out, int n, int h, int w, int c, int k, int stride, int pad,
                   cudaStream_t stream)
{
    const int h_out = (h + 2 * pad - k) / stride + 1, w_out = (w + 2 * pad - k) / stride + 1;
    const long long total = (long long)n * h_out * w_out * (c / 16);
    if (total == 0) return ICONV_OK;
    if (k == 3 && stride == 2 && pad == 1 && c % 32 == 0 && ((uintptr_t)x % 32) == 0 && ((uintptr_t)out % 32) == 0 && total < (1ll << 31) &&
        (long long)n * h * w * (c / 16) < (1ll << 31)) {
        const unsigned wide_total = (unsigned)(total / 2);
        maxpool_3x3s2_wide_kernel<<<(wide_total + 255) / 256, 256, 0, stream>>>((const uint8_t *)x, (uint8_t *)out, wide_total, h, w, c / 32, h_out,
                                                                                w_out);
        ICONV_CUDA_TRY(cudaGetLastError());
        return ICONV_OK;
    }
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
