// Body of one window-kernel translation unit: define ICONV_INST_EPI (2, 3, 4, 5 or 8) before including.
// The no-skip variants (2, 4) carry every compile-time filter size; the skip variants 3x3 only;
// the narrow variant 3x3 with 64-byte rows only.  Everything else runs the generic instance.
#include "umma_inst.h"

namespace iconv {

#define ICONV_CAT2(a, b) a##b
#define ICONV_CAT(a, b) ICONV_CAT2(a, b)
#define ICONV_WIN_GO(KH, KW, KJ) return umma_launch_pdl(umma_window_kernel<E, KH, KW, KJ>, l, *l.tmap_x, *l.tmap_w, *l.a, *l.u)
#define ICONV_WIN_ATTR(KH, KW, KJ) if (e == cudaSuccess) e = cudaFuncSetAttribute(umma_window_kernel<E, KH, KW, KJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM)

cudaError_t ICONV_CAT(umma_window_launch_, ICONV_INST_EPI)(int kh, int kw, int kj, int pair16, const UmmaLaunch &l)
{
    constexpr int E = ICONV_INST_EPI;
    constexpr bool ALL = E == EPI_FAST || E == EPI_SAFE, SKIP = E == EPI_FAST_SKIP8 || E == EPI_SAFE_SKIP8;
    if (kh == 3 && kw == 3 && kj == 2) ICONV_WIN_GO(3, 3, 2);
    else if ((ALL || SKIP) && kh == 3 && kw == 3 && kj == 4) ICONV_WIN_GO((ALL || SKIP) ? 3 : 0, (ALL || SKIP) ? 3 : 0, (ALL || SKIP) ? 4 : 0);
    else if (ALL && kh == 5 && kw == 5 && kj == 2) ICONV_WIN_GO(ALL ? 5 : 0, ALL ? 5 : 0, ALL ? 2 : 0);
    else if (ALL && kh == 4 && kw == 4 && kj == 1 && pair16) ICONV_WIN_GO(ALL ? 4 : 0, ALL ? 2 : 0, ALL ? 1 : 0);
    else if (ALL && kh == 4 && kw == 4 && kj == 1) ICONV_WIN_GO(ALL ? 4 : 0, ALL ? 4 : 0, ALL ? 1 : 0);
    else ICONV_WIN_GO(0, 0, 0);
}

cudaError_t ICONV_CAT(umma_window_opt_in_, ICONV_INST_EPI)()
{
    constexpr int E = ICONV_INST_EPI;
    constexpr bool ALL = E == EPI_FAST || E == EPI_SAFE, SKIP = E == EPI_FAST_SKIP8 || E == EPI_SAFE_SKIP8;
    cudaError_t e = cudaSuccess;
    ICONV_WIN_ATTR(3, 3, 2);
    ICONV_WIN_ATTR(0, 0, 0);
    if (ALL || SKIP) ICONV_WIN_ATTR((ALL || SKIP) ? 3 : 0, (ALL || SKIP) ? 3 : 0, (ALL || SKIP) ? 4 : 0);
    if (ALL) {
        ICONV_WIN_ATTR(ALL ? 5 : 0, ALL ? 5 : 0, ALL ? 2 : 0);
        ICONV_WIN_ATTR(ALL ? 4 : 0, ALL ? 2 : 0, ALL ? 1 : 0);
        ICONV_WIN_ATTR(ALL ? 4 : 0, ALL ? 4 : 0, ALL ? 1 : 0);
    }
    return e;
}

}  // namespace iconv
