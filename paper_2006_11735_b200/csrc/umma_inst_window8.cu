// window-kernel instances of epilogue variant 8 (see umma_inst.h)
#define ICONV_INST_EPI 8
#include "umma_inst_window.cuh"
