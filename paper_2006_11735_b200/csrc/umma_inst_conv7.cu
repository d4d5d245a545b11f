// im2col-kernel instances of epilogue variant 7 (see umma_inst.h)
#define ICONV_INST_EPI 7
#include "umma_inst_conv.cuh"
