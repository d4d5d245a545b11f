// window-kernel instances of epilogue variant 5 (see umma_inst.h)
#define ICONV_INST_EPI 5
#include "umma_inst_window.cuh"
