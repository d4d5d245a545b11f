// Kernel selection for a planned layer.
#include "plan.h"

namespace iconv {

int choose_kernel(iconv_plan_t *p)
{
    const int want = p->d.kernel;
    if (p->d.proj_weights) {
        // a fused projection skip exists on the tensor-core path only
        if (want != ICONV_KERNEL_AUTO && want != ICONV_KERNEL_UMMA && want != ICONV_KERNEL_UMMA_IM2COL) {
            set_error("iconv_plan: a fused projection needs the tensor-core kernel");
            return ICONV_ERR_UNSUPPORTED;
        }
        const int rc = umma_supported(p);
        if (rc != ICONV_OK) return rc;
        p->kernel = ICONV_KERNEL_UMMA;
        return umma_setup(p);
    }
    if (want == ICONV_KERNEL_DIRECT || p->d.n == 0) {
        p->kernel = ICONV_KERNEL_DIRECT;
        return ICONV_OK;
    }
    if (want == ICONV_KERNEL_UMMA || want == ICONV_KERNEL_UMMA_IM2COL) {
        const int rc = umma_supported(p);
        if (rc != ICONV_OK) return rc;
        p->kernel = ICONV_KERNEL_UMMA;
        return umma_setup(p);
    }
    if (want == ICONV_KERNEL_THIN) {
        const int rc = thin_supported(p);
        if (rc != ICONV_OK) return rc;
        p->kernel = ICONV_KERNEL_THIN;
        return thin_setup(p);
    }
    if (want == ICONV_KERNEL_STEM) {
        const int rc = stem_supported(p);
        if (rc != ICONV_OK) return rc;
        p->kernel = ICONV_KERNEL_STEM;
        return stem_setup(p);
    }
    // AUTO: the repacking paths of the first layers (tensor cores), then the thin layers on
    // the CUDA cores, then the tensor-core path proper, the direct kernel for whatever is left.
    if (stem_supported(p) == ICONV_OK) {
        const int rc = stem_setup(p);
        if (rc == ICONV_OK) {
            p->kernel = ICONV_KERNEL_STEM;
            return ICONV_OK;
        }
        if (rc != ICONV_ERR_UNSUPPORTED) return rc;
    }
    if (umma_narrow(p->d) && umma_supported(p) == ICONV_OK) {
        // a narrow output whose reduction is wide enough for the tensor cores (window mode, byte stores)
        const int rc = umma_setup(p);
        if (rc == ICONV_OK) {
            p->kernel = ICONV_KERNEL_UMMA;
            return ICONV_OK;
        }
        if (rc != ICONV_ERR_UNSUPPORTED) return rc;
        cudaFree(p->w_packed);
        p->w_packed = nullptr;
        cudaFree(p->params_packed);
        p->params_packed = nullptr;
    }
    if (thin_supported(p) == ICONV_OK) {
        p->kernel = ICONV_KERNEL_THIN;
        return thin_setup(p);
    }
    if (umma_supported(p) == ICONV_OK) {
        const int rc = umma_setup(p);
        if (rc == ICONV_OK) {
            p->kernel = ICONV_KERNEL_UMMA;
            return ICONV_OK;
        }
        if (rc != ICONV_ERR_UNSUPPORTED) return rc;
        cudaFree(p->w_packed);               // geometry the TMA descriptor cannot express
        p->w_packed = nullptr;
    }
    p->kernel = ICONV_KERNEL_DIRECT;
    return ICONV_OK;
}

}  // namespace iconv
