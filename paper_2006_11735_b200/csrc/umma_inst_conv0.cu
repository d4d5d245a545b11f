// im2col-kernel instances of epilogue variant 0 (see umma_inst.h)
#define ICONV_INST_EPI 0
#include "umma_inst_conv.cuh"
