// im2col-kernel instances of epilogue variant 6 (see umma_inst.h)
#define ICONV_INST_EPI 6
#include "umma_inst_conv.cuh"
