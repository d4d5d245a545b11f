// Bandwidth-bound thin layers (c_in <= 4 or c_out == 1).
#include "plan.h"

namespace iconv {

int thin_supported(const iconv_plan_t *p)
{
    (void)p;
    set_error("thin kernels: not built yet");
    return ICONV_ERR_UNSUPPORTED;
}

int launch_thin(const iconv_plan_t *p, const ConvArgs &a, cudaStream_t stream)
{
    (void)p; (void)a; (void)stream;
    set_error("thin kernels: not built yet");
    return ICONV_ERR_UNSUPPORTED;
}

}  // namespace iconv
