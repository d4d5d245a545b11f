// im2col-kernel instances of epilogue variant 1 (see umma_inst.h)
#define ICONV_INST_EPI 1
#include "umma_inst_conv.cuh"
