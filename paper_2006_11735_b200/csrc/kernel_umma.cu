// tcgen05.mma kind::i8 implicit-GEMM convolution.
#include "plan.h"

namespace iconv {

int umma_supported(const iconv_plan_t *p)
{
    (void)p;
    set_error("tensor-core path: not built yet");
    return ICONV_ERR_UNSUPPORTED;
}
int umma_setup(iconv_plan_t *p) { (void)p; return ICONV_ERR_UNSUPPORTED; }

int launch_umma(const iconv_plan_t *p, const ConvArgs &a, cudaStream_t stream)
{
    (void)p; (void)a; (void)stream;
    set_error("tensor-core path: not built yet");
    return ICONV_ERR_UNSUPPORTED;
}

}  // namespace iconv
