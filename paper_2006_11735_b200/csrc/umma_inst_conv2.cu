// im2col-kernel instances of epilogue variant 2 (see umma_inst.h)
#define ICONV_INST_EPI 2
#include "umma_inst_conv.cuh"
