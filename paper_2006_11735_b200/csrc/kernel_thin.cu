// Bandwidth-bound thin layers on the CUDA cores (the first and last layers of the
// regression networks): too little reduction per output byte for the tensor cores to matter,
// so the kernels are built around coalesced 16-byte accesses and dp4a.
//
//   thin_in   c_in = 1 (e.g. 3x3 or 5x5, 1 -> 64).  Four threads share a pixel, each owning 16
//             output channels: the kh*kw input bytes of the pixel are packed four to a word,
//             the filter bank sits in shared memory packed the same way, every output costs
//             ceil(kh*kw / 4) dp4a plus the epilogue, and a warp stores 512 contiguous bytes.
//   thin_out  c_out = 1 (e.g. 3x3, 64 -> 1, with the global residual).  c_in / 16 lanes share a
//             pixel, each reading 16 channels per tap with one 16-byte load (a warp reads 512
//             contiguous bytes per tap when c_in = 64); partial sums meet by warp shuffles and
//             the group's first lane applies the epilogue.
#include "plan.h"

namespace iconv {

namespace {

constexpr int THIN_MAX_W4 = 7;          // packed filter words per output channel: kh * kw <= 28
constexpr int THIN_IN_THREADS = 256;

__device__ __forceinline__ int dp4a_us(unsigned a, int b, int c)
{
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ int dp4a_ss(int a, int b, int c)
{
    int d;
    asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

struct ThinArgs {
    int groups;        // thin_in: threads per pixel (c_out / 16)
    int w4;            // thin_in: packed words per output channel
    int narrow;        // thin_in: 1 when BReLU + Eq. 4 provably fit 32 bits for every channel
    int lpp;           // thin_out: lanes per pixel (c_in / 16)
    // x / w_out and x / (h_out * w_out) as umulhi(x, mul) >> shr (x < 2^31; mul == 0: divisor 1)
    unsigned div_w_mul, div_w_shr, div_hw_mul, div_hw_shr;
};

__device__ __forceinline__ unsigned thin_div(unsigned x, unsigned mul, unsigned shr) { return mul ? (__umulhi(x, mul) >> shr) : x; }

// SIGNED: the packed input bytes are int8 (stored int8, or raw uint8 turned into raw - 128 by
// flipping bit 7); otherwise uint8.  KH, KW: the filter size when known at compile time (0:
// read from the arguments).  FAST: per-layer parameters and a proven 32-bit Eq. 4 (then the
// thread keeps its 16 biases in registers: it serves the same channel group for every pixel).
template <bool SIGNED, int KH, int KW, bool FAST>
__global__ void __launch_bounds__(THIN_IN_THREADS) thin_in_kernel(const __grid_constant__ ConvArgs a, const __grid_constant__ ThinArgs t)
{
    extern __shared__ int ws[];                       // [w4][c_out + c_out / 16]: word j of channel co at j * pitch + co + co / 16
    const int pitch = a.c_out + a.c_out / 16;         // one pad word per 16 channels: the groups of a pixel hit distinct banks
    const int kh = KH ? KH : a.kh, kw = KW ? KW : a.kw;
    const int K = kh * kw;
    const int w4 = KH ? (KH * KW + 3) / 4 : t.w4;
    for (int e = threadIdx.x; e < w4 * a.c_out; e += blockDim.x) {
        const int co = e % a.c_out, j = e / a.c_out;
        unsigned word = 0;
        for (int b = 0; b < 4; ++b) {
            const int k = 4 * j + b;
            if (k < K) word |= (unsigned)(uint8_t)a.w[(long long)co * K + k] << (8 * b);
        }
        ws[j * pitch + co + co / 16] = (int)word;
    }
    __syncthreads();

    const int g = threadIdx.x % t.groups;              // this thread's 16-channel group
    const int ppb = blockDim.x / t.groups;             // pixels per block and pass
    const unsigned m_total = (unsigned)((long long)a.n * a.h_out * a.w_out);
    const unsigned hw = (unsigned)(a.h_out * a.w_out);
    const unsigned flip = a.in_dtype == ICONV_U8_RAW128 ? 0x80u : 0u;
    const uint8_t *x = (const uint8_t *)a.x;
    const int *wg = ws + g * 17;                       // word j of this group's channel c at wg[j * pitch + c]
    int b16[16];
    int q_mul = 0, q_shift = 1, q_h = 0;
    unsigned q_half = 0;
    if (FAST) {
#pragma unroll
        for (int c = 0; c < 16; ++c) b16[c] = __ldg(a.bias + g * 16 + c);
        q_mul = __ldg(a.mul); q_shift = __ldg(a.shift); q_h = __ldg(a.h_i); q_half = 1u << (q_shift - 1);
    }
    for (unsigned m = blockIdx.x * ppb + threadIdx.x / t.groups; m < m_total; m += gridDim.x * ppb) {
        const unsigned img = thin_div(m, t.div_hw_mul, t.div_hw_shr);
        const unsigned rem = m - img * hw;
        const int oh = (int)thin_div(rem, t.div_w_mul, t.div_w_shr);
        const int ow = (int)rem - oh * a.w_out;
        const uint8_t *ximg = x + (size_t)img * a.h * a.w_;
        unsigned xw[THIN_MAX_W4];
#pragma unroll
        for (int j = 0; j < THIN_MAX_W4; ++j) xw[j] = 0;
        if (KH) {
#pragma unroll
            for (int r = 0; r < (KH ? KH : 1); ++r) {
                const int ih = oh * a.stride - a.pad + r;
                const bool row_in = ih >= 0 && ih < a.h;
#pragma unroll
                for (int s = 0; s < (KW ? KW : 1); ++s) {
                    const int k = r * KW + s;
                    const int iw = ow * a.stride - a.pad + s;
                    unsigned v = 0;                    // zero padding, after the re-normalisation
                    if (row_in && iw >= 0 && iw < a.w_) v = (unsigned)__ldg(ximg + ih * a.w_ + iw) ^ flip;
                    xw[k >> 2] |= v << ((k & 3) * 8);
                }
            }
        } else {
            int k = 0;
            for (int r = 0; r < kh; ++r) {
                const int ih = oh * a.stride - a.pad + r;
                for (int s = 0; s < kw; ++s, ++k) {
                    const int iw = ow * a.stride - a.pad + s;
                    unsigned v = 0;
                    if (ih >= 0 && ih < a.h && iw >= 0 && iw < a.w_) v = (unsigned)__ldg(ximg + ih * a.w_ + iw) ^ flip;
                    const unsigned sh = (unsigned)(k & 3) * 8u;
#pragma unroll
                    for (int j = 0; j < THIN_MAX_W4; ++j)
                        if (j == (k >> 2)) xw[j] |= v << sh;
                }
            }
        }
        unsigned packed[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int V[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int c = 4 * q + e, co = g * 16 + c;
                int U = 0;
#pragma unroll
                for (int j = 0; j < THIN_MAX_W4; ++j)
                    if (j < w4) {
                        const int wv = wg[j * pitch + c];
                        U = SIGNED ? dp4a_ss((int)xw[j], wv, U) : dp4a_us(xw[j], wv, U);
                    }
                if (FAST) {
                    const int y = max(min(U + b16[c], q_h), 0);
                    const int v = (int)(((unsigned)y * (unsigned)q_mul + q_half) >> q_shift);
                    V[e] = min(max(v + a.out_zero, a.out_lo), a.out_hi);
                } else {
                    const int pc = a.per_channel ? co : 0;
                    if (t.narrow) {
                        int y = U + __ldg(a.bias + co);
                        const int shift = __ldg(a.shift + pc);
                        y = max(min(y, __ldg(a.h_i + pc)), 0);
                        const int v = (int)(((unsigned)y * (unsigned)__ldg(a.mul + pc) + (1u << (shift - 1))) >> shift);
                        V[e] = min(max(v + a.out_zero, a.out_lo), a.out_hi);
                    } else {
                        V[e] = requant_tail((long long)U + __ldg(a.bias + co), a.brelu, __ldg(a.h_i + pc), __ldg(a.mul + pc),
                                            __ldg(a.shift + pc), a.out_zero, a.out_lo, a.out_hi);
                    }
                }
            }
            packed[q] = (V[0] & 0xff) | ((V[1] & 0xff) << 8) | ((V[2] & 0xff) << 16) | ((unsigned)(V[3] & 0xff) << 24);
        }
        *(uint4 *)((uint8_t *)a.out + (size_t)m * a.out_c_total + a.out_c_offset + g * 16) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    }
}

// K3: a 3x3 filter, whose nine 16-byte weight slices the lane keeps in registers.
template <bool SIGNED, bool K3>
__global__ void __launch_bounds__(256) thin_out_kernel(const __grid_constant__ ConvArgs a, const __grid_constant__ ThinArgs t)
{
    const int lane = threadIdx.x & 31;
    const int ppw = 32 / t.lpp;                        // pixels per warp and pass
    const int lp = lane / t.lpp, part = lane - lp * t.lpp;
    const bool active = lp < ppw;
    const unsigned m_total = (unsigned)((long long)a.n * a.h_out * a.w_out);
    const unsigned hw = (unsigned)(a.h_out * a.w_out);
    const unsigned warps = gridDim.x * (blockDim.x >> 5);
    const unsigned warp_id = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const uint8_t *x = (const uint8_t *)a.x + a.in_c_offset + part * 16;
    const int8_t *w = a.w + part * 16;
    int4 wr[9];
    if (K3) {
#pragma unroll
        for (int tap = 0; tap < 9; ++tap) wr[tap] = __ldg((const int4 *)(w + tap * a.c_in));
    }
    const int bias = __ldg(a.bias);
    for (unsigned m0 = warp_id * ppw; m0 < m_total; m0 += warps * ppw) {      // the same trip count for every lane of a warp
        const unsigned m = m0 + lp;
        const bool live = active && m < m_total;
        int U = 0;
        if (live) {
            const unsigned img = thin_div(m, t.div_hw_mul, t.div_hw_shr);
            const unsigned rem = m - img * hw;
            const int oh = (int)thin_div(rem, t.div_w_mul, t.div_w_shr);
            const int ow = (int)rem - oh * a.w_out;
            const uint8_t *ximg = x + (size_t)img * a.h * a.w_ * a.in_c_total;
            if (K3) {
                // nine loads with no branch between them (a tap outside the image reads the
                // image's first pixel instead and is zeroed afterwards), so that all nine are
                // in flight together
                uint4 xv[9];
#pragma unroll
                for (int r = 0; r < 3; ++r) {
                    const int ih = oh * a.stride - a.pad + r;
#pragma unroll
                    for (int s = 0; s < 3; ++s) {
                        const int iw = ow * a.stride - a.pad + s;
                        const bool in = ih >= 0 && ih < a.h && iw >= 0 && iw < a.w_;
                        const size_t off = in ? (size_t)(ih * a.w_ + iw) * a.in_c_total : 0;
                        uint4 v = __ldg((const uint4 *)(ximg + off));
                        if (!in) v = make_uint4(0, 0, 0, 0);
                        xv[r * 3 + s] = v;
                    }
                }
#pragma unroll
                for (int tap = 0; tap < 9; ++tap) {
                    const int4 wv = wr[tap];
                    if (SIGNED) {
                        U = dp4a_ss((int)xv[tap].x, wv.x, U); U = dp4a_ss((int)xv[tap].y, wv.y, U);
                        U = dp4a_ss((int)xv[tap].z, wv.z, U); U = dp4a_ss((int)xv[tap].w, wv.w, U);
                    } else {
                        U = dp4a_us(xv[tap].x, wv.x, U); U = dp4a_us(xv[tap].y, wv.y, U);
                        U = dp4a_us(xv[tap].z, wv.z, U); U = dp4a_us(xv[tap].w, wv.w, U);
                    }
                }
            } else {
                for (int r = 0; r < a.kh; ++r) {
                    const int ih = oh * a.stride - a.pad + r;
                    if (ih < 0 || ih >= a.h) continue;
                    for (int s = 0; s < a.kw; ++s) {
                        const int iw = ow * a.stride - a.pad + s;
                        if (iw < 0 || iw >= a.w_) continue;
                        const uint4 xv = __ldg((const uint4 *)(ximg + (size_t)(ih * a.w_ + iw) * a.in_c_total));
                        const int4 wv = __ldg((const int4 *)(w + (r * a.kw + s) * a.c_in));
                        if (SIGNED) {
                            U = dp4a_ss((int)xv.x, wv.x, U); U = dp4a_ss((int)xv.y, wv.y, U);
                            U = dp4a_ss((int)xv.z, wv.z, U); U = dp4a_ss((int)xv.w, wv.w, U);
                        } else {
                            U = dp4a_us(xv.x, wv.x, U); U = dp4a_us(xv.y, wv.y, U);
                            U = dp4a_us(xv.z, wv.z, U); U = dp4a_us(xv.w, wv.w, U);
                        }
                    }
                }
            }
        }
        int total = U;
        for (int k = 1; k < t.lpp; ++k) total += __shfl_down_sync(0xffffffffu, U, k);
        if (live && part == 0) {
            long long Y = (long long)total + bias;
            if (a.skip_dtype >= 0)
                Y += round_shift64((long long)load_skip(a.skip, (long long)m * a.skip_c_total + a.skip_c_offset, a.skip_dtype) * a.skip_mul, a.skip_shift);
            const long long oi = (long long)m * a.out_c_total + a.out_c_offset;
            if (a.out_dtype == ICONV_I32) {
                ((int32_t *)a.out)[oi] = (int32_t)Y;
            } else {
                const int V = requant_tail(Y, a.brelu, __ldg(a.h_i), __ldg(a.mul), __ldg(a.shift), a.out_zero, a.out_lo, a.out_hi);
                if (a.out_dtype == ICONV_U8) ((uint8_t *)a.out)[oi] = (uint8_t)V;
                else ((int8_t *)a.out)[oi] = (int8_t)V;
            }
        }
    }
}

void thin_divisor(unsigned d, unsigned &mul, unsigned &shr)
{
    if (d <= 1) { mul = 0; shr = 0; return; }
    unsigned lg = 0;
    while ((1ull << lg) < d) ++lg;
    mul = (unsigned)(((1ull << (31 + lg)) + d - 1) / d);
    shr = lg - 1;
}

bool is_thin_in(const iconv_desc &d)
{
    const int groups = d.c_out / 16;
    return d.c_in == 1 && d.in_c_total == 1 && d.in_c_offset == 0 && d.c_out % 16 == 0 && d.c_out <= 256 &&
           (groups & (groups - 1)) == 0 && d.out_dtype != ICONV_I32 && d.out_c_total % 16 == 0 && d.out_c_offset % 16 == 0 &&
           d.skip_dtype < 0 && d.kh * d.kw <= 4 * THIN_MAX_W4;
}

bool is_thin_out(const iconv_desc &d)
{
    return d.c_out == 1 && d.c_in % 16 == 0 && d.c_in <= 512 && d.in_c_total % 16 == 0 && d.in_c_offset % 16 == 0 &&
           d.in_dtype != ICONV_U8_RAW128;
}

}  // namespace

int thin_supported(const iconv_plan_t *p)
{
    if (is_thin_in(p->d) || is_thin_out(p->d)) return ICONV_OK;
    set_error("thin kernels: need c_in = 1 (8-bit output, no skip, c_out a power-of-two multiple of 16, kh*kw <= 28) "
              "or c_out = 1 (c_in a multiple of 16)");
    return ICONV_ERR_UNSUPPORTED;
}

int thin_setup(iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    p->thin_narrow = 0;
    if (is_thin_in(d) && d.brelu) {
        // BReLU + Eq. 4 in 32 bits when h_i * mul + 2^(shift-1) < 2^32 for every channel
        const int np = d.per_channel ? d.c_out : 1;
        bool ok = true;
        for (int i = 0; i < np && ok; ++i)
            ok = d.shift[i] >= 1 && d.shift[i] <= 31 &&
                 (unsigned long long)d.h_i[i] * (unsigned long long)d.mul[i] + (1ull << (d.shift[i] - 1)) < (1ull << 32);
        // U + b must stay in int32 as well: the plan's overflow check already bounds |Y|
        p->thin_narrow = ok ? 1 : 0;
    }
    return ICONV_OK;
}

int launch_thin(const iconv_plan_t *p, const ConvArgs &a, cudaStream_t stream)
{
    const iconv_desc &d = p->d;
    if (is_thin_in(d) ? ((uintptr_t)a.out % 16) != 0 : ((uintptr_t)a.x % 16) != 0) {
        set_error("iconv_forward: tensor pointers must be 16-byte aligned");
        return ICONV_ERR_ALIGN;
    }
    const long long m_total = (long long)d.n * p->h_out * p->w_out;
    if (m_total == 0) return ICONV_OK;
    ThinArgs t;
    t.groups = d.c_out / 16;
    t.w4 = (d.kh * d.kw + 3) / 4;
    t.narrow = p->thin_narrow;
    t.lpp = d.c_in / 16;
    const bool is_signed = d.in_dtype != ICONV_U8;
    if (m_total >= (1ll << 31) - 65536) { set_error("thin kernels: more than 2^31 output pixels"); return ICONV_ERR_UNSUPPORTED; }
    thin_divisor((unsigned)p->w_out, t.div_w_mul, t.div_w_shr);
    thin_divisor((unsigned)(p->h_out * p->w_out), t.div_hw_mul, t.div_hw_shr);
    if (is_thin_in(d)) {
        const int ppb = THIN_IN_THREADS / t.groups;
        long long blocks = (m_total + ppb - 1) / ppb;
        if (blocks > 148ll * 16) blocks = 148ll * 16;
        const size_t smem = (size_t)t.w4 * (d.c_out + d.c_out / 16) * sizeof(int);
        const bool fast = p->thin_narrow && !d.per_channel;
        const int k = d.kh == d.kw ? d.kh : 0;
#define ICONV_THIN_IN(S, KH, KW, F) thin_in_kernel<S, KH, KW, F><<<(unsigned)blocks, THIN_IN_THREADS, smem, stream>>>(a, t)
#define ICONV_THIN_IN_K(S, F)                                    \
    do {                                                         \
        if (k == 3) ICONV_THIN_IN(S, 3, 3, F);                   \
        else if (k == 5) ICONV_THIN_IN(S, 5, 5, F);              \
        else ICONV_THIN_IN(S, 0, 0, F);                          \
    } while (0)
        if (is_signed) { if (fast) ICONV_THIN_IN_K(true, true); else ICONV_THIN_IN_K(true, false); }
        else { if (fast) ICONV_THIN_IN_K(false, true); else ICONV_THIN_IN_K(false, false); }
#undef ICONV_THIN_IN_K
#undef ICONV_THIN_IN
    } else {
        if (t.lpp > 32) { set_error("thin kernels: c_in too wide"); return ICONV_ERR_UNSUPPORTED; }
        const int ppw = 32 / t.lpp;
        long long blocks = (m_total + 8ll * ppw - 1) / (8ll * ppw);
        if (blocks > 148ll * 16) blocks = 148ll * 16;
        const bool k3 = d.kh == 3 && d.kw == 3;
        if (is_signed) { if (k3) thin_out_kernel<true, true><<<(unsigned)blocks, 256, 0, stream>>>(a, t); else thin_out_kernel<true, false><<<(unsigned)blocks, 256, 0, stream>>>(a, t); }
        else { if (k3) thin_out_kernel<false, true><<<(unsigned)blocks, 256, 0, stream>>>(a, t); else thin_out_kernel<false, false><<<(unsigned)blocks, 256, 0, stream>>>(a, t); }
    }
    ICONV_CUDA_TRY(cudaGetLastError());
    return ICONV_OK;
}

}  // namespace iconv
