// Launch and shared-memory opt-in functions of the tensor-core kernel instances.  Each group of
// instances (one epilogue variant of the im2col kernel; one family of the window kernel) is
// compiled in a translation unit of its own (umma_inst_*.cu), so that the library builds in
// parallel; the host side (kernel_umma.cu) reaches the kernels only through these functions.
#pragma once

#include "umma_device.cuh"

namespace iconv {

struct UmmaLaunch {
    unsigned grid;
    size_t smem;
    cudaStream_t stream;
    const CUtensorMap *tmap_x, *tmap_w, *tmap_out, *tmap_skip;
    const ConvArgs *a;
    const UmmaArgs *u;
    int cluster;                    // CTAs per cluster: 2 for the CTA-pair form, else 1
};

// Launch with programmatic stream serialisation (see grid_dep_wait in umma_device.cuh).
template <typename... KArgs, typename... Args>
cudaError_t umma_launch_pdl(void (*kernel)(KArgs...), const UmmaLaunch &l, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(l.grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = l.smem;
    cfg.stream = l.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (l.cluster > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)l.cluster;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// im2col kernel: epi = EPI_* (EPI_NARROW excluded), issue = 0 / 1 / 2, or 3 (CTA pairs; the 8-bit-output forms without a fused projection: EPI_FAST, EPI_FAST_SKIP8, EPI_SAFE, EPI_SAFE_SKIP8)
cudaError_t umma_conv_launch(int epi, int issue, const UmmaLaunch &l);
cudaError_t umma_conv_opt_in(int epi);
// window kernel: kh, kw, kj as planned (the instance with compile-time sizes where one exists)
cudaError_t umma_window_launch(int epi, int kh, int kw, int kj, int pair16, const UmmaLaunch &l);
cudaError_t umma_window_opt_in(int epi);

// per-variant entry points behind the dispatchers above
#define ICONV_DECLARE_CONV(E) cudaError_t umma_conv_launch_##E(int issue, const UmmaLaunch &l); cudaError_t umma_conv_opt_in_##E();
ICONV_DECLARE_CONV(0) ICONV_DECLARE_CONV(1) ICONV_DECLARE_CONV(2) ICONV_DECLARE_CONV(3)
ICONV_DECLARE_CONV(4) ICONV_DECLARE_CONV(5) ICONV_DECLARE_CONV(6) ICONV_DECLARE_CONV(7)
#undef ICONV_DECLARE_CONV
#define ICONV_DECLARE_WIN(E) cudaError_t umma_window_launch_##E(int kh, int kw, int kj, int pair16, const UmmaLaunch &l); cudaError_t umma_window_opt_in_##E();
ICONV_DECLARE_WIN(2) ICONV_DECLARE_WIN(3) ICONV_DECLARE_WIN(4) ICONV_DECLARE_WIN(5) ICONV_DECLARE_WIN(8)
#undef ICONV_DECLARE_WIN

}  // namespace iconv
