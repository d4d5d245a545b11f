// im2col-kernel instances of epilogue variant 4 (see umma_inst.h)
#define ICONV_INST_EPI 4
#include "umma_inst_conv.cuh"
