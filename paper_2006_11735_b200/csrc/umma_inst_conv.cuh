// Body of one im2col-kernel translation unit: define ICONV_INST_EPI (0..7) before including.
#include "umma_inst.h"

namespace iconv {

#define ICONV_CAT2(a, b) a##b
#define ICONV_CAT(a, b) ICONV_CAT2(a, b)

cudaError_t ICONV_CAT(umma_conv_launch_, ICONV_INST_EPI)(int issue, const UmmaLaunch &l)
{
    constexpr int E = ICONV_INST_EPI;
    constexpr bool HAS_PAIR = E == EPI_FAST || E == EPI_FAST_SKIP8 || E == EPI_SAFE || E == EPI_SAFE_SKIP8;
    if (issue == 3) {
        if (!HAS_PAIR) return cudaErrorInvalidValue;
        return umma_launch_pdl(umma_conv_kernel<E, HAS_PAIR ? 3 : 0>, l, *l.tmap_x, *l.tmap_w, *l.tmap_out, *l.tmap_skip, *l.a, *l.u);
    }
    if (issue == 1) return umma_launch_pdl(umma_conv_kernel<E, 1>, l, *l.tmap_x, *l.tmap_w, *l.tmap_out, *l.tmap_skip, *l.a, *l.u);
    if (issue == 2) return umma_launch_pdl(umma_conv_kernel<E, 2>, l, *l.tmap_x, *l.tmap_w, *l.tmap_out, *l.tmap_skip, *l.a, *l.u);
    return umma_launch_pdl(umma_conv_kernel<E, 0>, l, *l.tmap_x, *l.tmap_w, *l.tmap_out, *l.tmap_skip, *l.a, *l.u);
}

cudaError_t ICONV_CAT(umma_conv_opt_in_, ICONV_INST_EPI)()
{
    constexpr int E = ICONV_INST_EPI;
    cudaError_t e = cudaFuncSetAttribute(umma_conv_kernel<E, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(umma_conv_kernel<E, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(umma_conv_kernel<E, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM);
    constexpr bool HAS_PAIR = E == EPI_FAST || E == EPI_FAST_SKIP8 || E == EPI_SAFE || E == EPI_SAFE_SKIP8;
    if (HAS_PAIR && e == cudaSuccess) e = cudaFuncSetAttribute(umma_conv_kernel<E, HAS_PAIR ? 3 : 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM);
    return e;
}

}  // namespace iconv
