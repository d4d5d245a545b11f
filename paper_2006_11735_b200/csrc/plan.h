// The opaque plan behind iconv_plan_t and the launchers each kernel family provides.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include "common.cuh"

struct iconv_plan_s {
    iconv_desc d;            // host pointers cleared after planning
    int h_out = 0, w_out = 0;
    int kernel = ICONV_KERNEL_DIRECT;
    // plain device copies (direct and thin kernels)
    int8_t *w_dev = nullptr;
    int32_t *bias_dev = nullptr, *mul_dev = nullptr, *shift_dev = nullptr, *h_i_dev = nullptr;
    // tensor-core path: weights repacked [c_out_pad][taps][c_in_pad], per-channel epilogue
    // parameters interleaved {bias, mul, shift, h_i}, TMA descriptors
    int8_t *w_packed = nullptr;
    int32_t *params_packed = nullptr;
    CUtensorMap tmap_w;      // 2-D tiled map over the packed weights
    int block_n = 0, kc = 0, c_in_pad = 0, c_out_pad = 0, stages = 0, swizzle_bytes = 0;
    int epi = 0;             // epilogue variant of the tensor-core kernel
    int half_n = 0, piece_bytes = 0;   // columns per epilogue warp and staged piece width
    int proj_c_in_pad = 0, proj_iters = 0, proj32 = 0;   // fused projection: padded channels, k-iterations, 32-bit rescale proven
    // window mode of the tensor-core kernel (stride-1 filters: one patch load per tile)
    int window = 0, win_vw = 0, win_bw = 0, win_bh = 0, win_full_width = 0, win_blocks = 0, win_tpi = 0, win_patch_bytes = 0, win_stages = 0, win_nbuf = 0, win_issuers = 2;
    int thin_narrow = 0;     // thin kernels: BReLU + Eq. 4 provably fit 32 bits
    int kg = 1;              // k-iterations grouped behind one pair of pipeline barriers
    int nbuf = 2;            // TMEM accumulator buffers
    int resident_b = 0;      // 1: the packed filter bank stays in shared memory for the whole kernel
    int epi_warps = 8, cs = 1, bi = 1;   // epilogue warps; column split per tile; tiles in flight
    int tail = 1;            // 0: zero point and output range are provably no-ops
    int q_mul = 1, q_shift = 0, q_h = 0; // per-layer Eq. 4 / BReLU scalars
    int epi_warp_bytes = 8192;           // staging memory per epilogue warp (im2col kernel)
    int skip_ring = 3;                   // staged 8-bit skip pieces per epilogue warp (2 or 3)
    int pair = 0;                        // long reductions on CTA pairs (tcgen05 cta_group::2): 256-pixel tiles, each CTA holds half of every B tile
    int pipe_room = 0;                   // shared memory left to the pipeline stages (bytes)
    int group_uniform = 0;               // per-channel parameters equal within every 16-channel group
    int pair16 = 0;                      // internal (stem): 16-channel positions read in pairs, two taps per K step
    // stem path: the plan of the GEMM that follows the repack, and the size of the repacked image,
    // which lives in the caller's workspace (iconv_workspace_bytes)
    iconv_plan_s *inner = nullptr;
    size_t workspace_bytes = 0;
};

namespace iconv {

int choose_kernel(iconv_plan_t *p);      // fills p->kernel and the kernel-specific fields
// iconv_plan with the internal options: pair16 plans a 16-channel layer with paired taps (the
// input must be followed by 16 readable bytes; the tensor-core window path or failure)
int plan_create(const iconv_desc *desc, int pair16, iconv_plan_t **plan_out);

int launch_umma(const iconv_plan_t *p, const ConvArgs &a, cudaStream_t stream);
int launch_thin(const iconv_plan_t *p, const ConvArgs &a, cudaStream_t stream);
int umma_supported(const iconv_plan_t *p);   // ICONV_OK or the reason it is not
bool umma_narrow(const iconv_desc &d);      // an 8-bit output too narrow or unaligned for 16-byte stores that window mode could still take
int umma_setup(iconv_plan_t *p);
int umma_init_once();                        // driver entry points, shared-memory opt-in of the current device; allocates nothing
int umma_device_ready(int device);           // the device's SM count once umma_init_once ran on it, else -1
// 2-D tiled TMA map over uint8 rows: `inner` bytes per row of which a box takes box_inner, `rows` rows `row_stride`
// bytes apart of which a box takes box_rows; swizzle span in bytes (32, 64, 128; 0 none)
int umma_encode_2d(CUtensorMap *map, const void *base, long long inner, long long rows, long long row_stride, int box_inner, int box_rows, int swizzle);
int umma_chain_opt_in();                     // shared-memory opt-in of the two-layer kernel on the current device
int umma_check_maps(const iconv_plan_t *p, const void *x, void *out);   // can every TMA descriptor of a launch be encoded?
int umma_geometry(iconv_plan_t *p);           // host-only tile / pipeline / epilogue geometry
int umma_encode_weight_map(iconv_plan_t *p);  // TMA map over p->w_packed
void window_plan(iconv_plan_t *p);            // window mode if the layer allows (needs p->epi); host only
int umma_epilogue_safe();                     // id of the explicit-clamp 32-bit epilogue variant
int thin_supported(const iconv_plan_t *p);
int thin_setup(iconv_plan_t *p);
int stem_supported(const iconv_plan_t *p);
int stem_setup(iconv_plan_t *p);
int launch_stem(const iconv_plan_t *p, const ConvArgs &a, void *workspace, cudaStream_t stream);

int launch_add_requant(const iadd_desc &d, const void *a, const void *b, void *out, cudaStream_t stream);
int launch_maxpool(const void *x, void *out, int n, int h, int w, int c, int k, int stride, int pad,
                   cudaStream_t stream);
int launch_avgpool(const void *x, void *out, int n, int h, int w, int c, int mul, int shift, int max_int,
                   cudaStream_t stream);
constexpr int MAX_DEVICES = 64;               // per-device tables (shared-memory opt-in, SM count, status word) have this many slots
int current_device_slot();                    // index of the current device in those tables, or -1
int *device_status_ptr();                     // the status word of the current device
int launch_wait_selftest(int which, long long limit_cycles, cudaStream_t stream);

}  // namespace iconv
