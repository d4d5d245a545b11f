// im2col-kernel instances of epilogue variant 3 (see umma_inst.h)
#define ICONV_INST_EPI 3
#include "umma_inst_conv.cuh"
