// Shared declarations of the CUDA path: kernel argument block, the integer epilogue
// (bias, rescaled skip, BReLU, Eq. 4, zero point, saturation) and host-side error helpers.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>

#include "iconv.h"

namespace iconv {

// Everything a convolution kernel needs, passed by value as a __grid_constant__.
struct ConvArgs {
    const void *x;
    const void *skip;
    void *out;
    const int8_t *w;        // [c_out][kh][kw][c_in]
    const int32_t *bias;
    const int32_t *mul;
    const int32_t *shift;
    const int32_t *h_i;
    int n, h, w_, c_in, c_out, kh, kw, stride, pad, h_out, w_out;
    int in_dtype, in_c_total, in_c_offset;
    int out_dtype, out_c_total, out_c_offset;
    int brelu, per_channel, out_lo, out_hi, out_zero;
    int skip_dtype, skip_c_total, skip_c_offset, skip_mul, skip_shift;
};

// [v / 2^s], ties toward +infinity (the bracket of Eq. 4); >> on a signed 64-bit value is
// an arithmetic shift in CUDA C++, i.e. a floor.
__device__ __forceinline__ long long round_shift64(long long v, int s)
{
    return s == 0 ? v : ((v + (1ll << (s - 1))) >> s);
}

// Value of one skip element in the integer domain of the addition (Section 4.1).
__device__ __forceinline__ int load_skip(const void *skip, long long idx, int dtype)
{
    switch (dtype) {
    case ICONV_U8:        return (int)((const uint8_t *)skip)[idx];
    case ICONV_S8:        return (int)((const int8_t *)skip)[idx];
    case ICONV_I32:       return ((const int32_t *)skip)[idx];
    default:              return (int)((const uint8_t *)skip)[idx] - 128;   // ICONV_U8_RAW128
    }
}

// BReLU (Eq. 5, l = 0), requantisation (Eq. 4), zero point, saturation.  64-bit product.
__device__ __forceinline__ int requant_tail(long long Y, int brelu, int h_i, int mul, int shift,
                                            int out_zero, int out_lo, int out_hi)
{
    if (brelu) {
        Y = Y < 0 ? 0 : Y;
        Y = Y > (long long)h_i ? (long long)h_i : Y;
    }
    long long V = round_shift64(Y * (long long)mul, shift) + out_zero;
    V = V < out_lo ? out_lo : V;
    V = V > out_hi ? out_hi : V;
    return (int)V;
}

// Host helpers -------------------------------------------------------------------------
void set_error(const char *fmt, ...);
int cuda_fail(cudaError_t e, const char *what);   // records the text, returns ICONV_ERR_CUDA

#define ICONV_CUDA_TRY(expr)                                         \
    do {                                                             \
        cudaError_t e__ = (expr);                                    \
        if (e__ != cudaSuccess) return ::iconv::cuda_fail(e__, #expr); \
    } while (0)

// Launchers implemented by the kernel files.
int launch_direct(const ConvArgs &a, cudaStream_t stream);

}  // namespace iconv
