// Implicit-GEMM integer convolution on the 5th-generation tensor cores.
//
//   GEMM view   M = n*h_out*w_out output pixels, N = c_out, K = kh*kw*c_in.
//   A operand   activations, fetched by TMA in im2col mode: one load per (filter tap,
//               channel chunk) brings 128 consecutive output pixels x KC channels into
//               shared memory, K-major, hardware-swizzled; out-of-image taps arrive as 0.
//   B operand   int8 weights, repacked at plan time to [c_out_pad][tap][c_in_pad] and
//               fetched by tiled TMA into the same K-major swizzled layout.
//   D           int32 accumulators in tensor memory (TMEM), two buffers of BLOCK_N columns,
//               so the epilogue of one tile overlaps the MMAs of the next.
//   MMA         tcgen05.mma.cta_group::1.kind::i8, M=128, N=BLOCK_N, K=32 per instruction,
//               u8 (or s8) x s8 -> s32, issued by one thread.
//   Epilogue    four warps read TMEM (32 lanes each), add the bias and the rescaled skip,
//               apply BReLU, Eq. 4, zero point and saturation, and store 16 output
//               channels per 16-byte store at the layer's channel offset.
//
// Persistent CTAs (one per SM) walk the tiles round-robin.  Warp 0 produces (TMA), warp 1
// issues MMAs and owns the TMEM allocation, warps 2-5 run the epilogue.  All mbarrier
// waits are bounded: on expiry the CTA records a code in the device status word, drains
// its copies in flight, frees its TMEM and returns.
#include <cuda.h>

#include <vector>

#include "plan.h"

namespace iconv {

namespace {

constexpr int BLOCK_M = 128;
constexpr int NUM_THREADS = 320;          // TMA warp, MMA warp, eight epilogue warps
constexpr int WARP_COLS = 128;            // columns one epilogue warp handles per tile (256 / 2)

// Epilogue variants, chosen at plan time.
enum { EPI_WIDE = 0,             // any descriptor: 64-bit products, run-time branches
       EPI_RAW = 1,              // int32 Y out, no skip: bias add only
       EPI_NARROW_NOSKIP = 2,    // BReLU + Eq. 4 proven to fit 32 bits
       EPI_NARROW_SKIP8 = 3,     // ... with an 8-bit skip whose rescale fits 32 bits
       EPI_NARROW_SKIPWIDE = 4   // ... with an int32 (or unproven) skip added in 64 bits
};
constexpr int MAX_STAGES = 8;
constexpr unsigned long long WAIT_LIMIT_NS = 4000000000ull;
constexpr int EPI_SMEM = 8 * 8192;        // per epilogue warp: output staging + skip staging
constexpr int SMEM_BUDGET = 140 * 1024;    // pipeline stages; barriers, parameters and epilogue staging come on top
constexpr int MAX_SMEM = 225 * 1024;

struct UmmaArgs {
    long long m_total;
    int m_tiles, n_tiles;
    int block_n, kc, cchunks, taps;
    int stages, stage_a_bytes, stage_bytes;
    int tmem_cols;
    unsigned idesc;
    unsigned long long desc_hi;     // upper 32 bits of the shared-memory matrix descriptors
    int skip_half;                  // 2^(skip_shift-1), or 0
    int half_n;                     // columns of the tile taken by the first epilogue warp of a quadrant
    int piece_bytes;                // row width of one staged output piece (16, 32, 64 or 128 bytes)
    int *status;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer();
    for (uint32_t i = 1;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 0) {
            if (*abort_flag) return false;
            if (globaltimer() - t0 > WAIT_LIMIT_NS) return false;
        }
    }
}

__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c, int w,
                                                   int h, int n, unsigned short off_w, unsigned short off_h)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                        uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier receives one arrival once every MMA issued so far by this thread is done.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major, hardware-swizzled tile whose rows are one
// swizzle span wide: start address, stride between 8-row groups, descriptor version 1
// and the swizzle mode (the constant upper half comes from the host).
__device__ __forceinline__ unsigned long long smem_desc(uint32_t addr, unsigned long long hi)
{
    return hi | (unsigned long long)((addr & 0x3FFFFu) >> 4) | (1ull << 16);
}

struct WarpParams {
    int bias[WARP_COLS], mul[WARP_COLS], shift[WARP_COLS], h_i[WARP_COLS];
};

struct Shared {
    WarpParams params[8];
    unsigned long long skip_full[8];
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    unsigned long long drain;
    uint32_t tmem_base;
    volatile int abort_flag;
};

__device__ __forceinline__ void give_up(Shared *sh, int *status, int code)
{
    sh->abort_flag = 1;
    atomicCAS(status, 0, code);
}

}  // namespace

template <int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_conv_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                 const __grid_constant__ CUtensorMap tmap_out, const __grid_constant__ CUtensorMap tmap_skip,
                 const __grid_constant__ ConvArgs a, const __grid_constant__ UmmaArgs u)
{
    extern __shared__ uint8_t smem_raw[];
    // tiles need the alignment of the widest swizzle pattern (8 rows x 128 bytes)
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    Shared *sh = (Shared *)(tiles + (size_t)u.stages * u.stage_bytes);
    // per epilogue warp: 4 KB output staging + 4 KB skip staging, 1024-byte aligned
    uint8_t *epi_smem = (uint8_t *)(((uintptr_t)(sh + 1) + 1023) & ~(uintptr_t)1023);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int num_tiles = u.m_tiles * u.n_tiles;
    const int k_iters = u.taps * u.cchunks;

    if (threadIdx.x == 0) {
        for (int s = 0; s < u.stages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh->tmem_full[b]), 1);
            mbar_init(smem_u32(&sh->tmem_empty[b]), 8);
        }
        for (int w = 0; w < 8; ++w) mbar_init(smem_u32(&sh->skip_full[w]), 1);
        mbar_init(smem_u32(&sh->drain), 1);
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&sh->tmem_base), (uint32_t)u.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    int issued = 0;        // producer: k-iterations whose loads were issued
    int skip_issued = 0;   // epilogue lane 0: skip prefetches issued

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            int it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m_tile = tile / u.n_tiles, n_tile = tile % u.n_tiles;
                const long long m0 = (long long)m_tile * BLOCK_M;
                const int q = (int)(m0 % a.w_out);
                const int p = (int)((m0 / a.w_out) % a.h_out);
                const int img = (int)(m0 / ((long long)a.w_out * a.h_out));
                const int cw = q * a.stride - a.pad, ch = p * a.stride - a.pad;
                for (int tap = 0; tap < u.taps && ok; ++tap) {
                    const unsigned short r = (unsigned short)(tap / a.kw), s = (unsigned short)(tap % a.kw);
                    for (int cc = 0; cc < u.cchunks; ++cc, ++it) {
                        const int stage = it % u.stages;
                        const uint32_t parity = (uint32_t)((it / u.stages) & 1);
                        if (!mbar_wait(smem_u32(&sh->empty[stage]), parity ^ 1u, &sh->abort_flag)) {
                            give_up(sh, u.status, 1);
                            ok = false;
                            break;
                        }
                        const uint32_t full = smem_u32(&sh->full[stage]);
                        const uint32_t sa = smem_u32(tiles + (size_t)stage * u.stage_bytes);
                        mbar_expect_tx(full, (uint32_t)(BLOCK_M * u.kc + u.block_n * u.kc));
                        tma_load_im2col_4d(sa, &tmap_x, full, cc * u.kc, cw, ch, img, s, r);
                        tma_load_2d(sa + u.stage_a_bytes, &tmap_w, full, (tap * u.cchunks + cc) * u.kc,
                                    n_tile * u.block_n);
                        issued = it + 1;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            int it = 0, t = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++t) {
                const int buf = t & 1;
                if (!mbar_wait(smem_u32(&sh->tmem_empty[buf]), (uint32_t)(((t >> 1) & 1) ^ 1), &sh->abort_flag)) {
                    give_up(sh, u.status, 2);
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * u.block_n);
                for (int ki = 0; ki < k_iters; ++ki, ++it) {
                    const int stage = it % u.stages;
                    if (!mbar_wait(smem_u32(&sh->full[stage]), (uint32_t)((it / u.stages) & 1), &sh->abort_flag)) {
                        give_up(sh, u.status, 3);
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(tiles + (size_t)stage * u.stage_bytes);
                    const unsigned long long da = smem_desc(sa, u.desc_hi);
                    const unsigned long long db = smem_desc(sa + u.stage_a_bytes, u.desc_hi);
                    for (int j = 0; j < u.kc / 32; ++j)   // 32 bytes of K per instruction: +2 in 16-byte units
                        umma_i8(d_tmem, da + 2ull * j, db + 2ull * j, u.idesc, (uint32_t)((ki | j) != 0));
                    umma_commit(smem_u32(&sh->empty[stage]));   // frees the stage when these MMAs are done
                }
                if (ok) umma_commit(smem_u32(&sh->tmem_full[buf]));
            }
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------------------- epilogue
        // Eight warps.  warp % 4 fixes the TMEM lane quadrant (32 output pixels) a warp may
        // read; the two warps of a quadrant split the tile's columns in halves.  A warp
        // works alone: it keeps its own copy of its channels' parameters, prefetches its
        // own part of an 8-bit skip tensor by TMA, stages its outputs in its own swizzled
        // shared-memory buffer and writes them with its own TMA stores (which also clip
        // the ragged last tile), so no cross-warp barrier exists that a warp which gave up
        // could strand.
        const int ew = warp - 2;
        const int quad = warp & 3;
        const int half = ew >> 2;
        const int col_lo = half * u.half_n;
        const int ncols = min(u.block_n - col_lo, u.half_n);          // may be <= 0 for narrow tiles
        WarpParams *wp = &sh->params[ew];
        uint8_t *obuf = epi_smem + (size_t)ew * 8192;                 // 32 rows x 128 bytes, 1024-aligned
        uint8_t *sbuf = obuf + 4096;
        const uint32_t skip_bar = smem_u32(&sh->skip_full[ew]);
        const int esz = a.out_dtype == ICONV_I32 ? 4 : 1;
        const int pcols = u.piece_bytes / esz;                        // columns per staged piece
        const int swz_shift = u.piece_bytes == 128 ? 0 : (u.piece_bytes == 64 ? 1 : 2);
        const int swz_mask = u.piece_bytes / 16 - 1;
        const int q_mul = __ldg(a.mul), q_shift = __ldg(a.shift), q_h_i = __ldg(a.h_i);
        const unsigned row_off = (unsigned)lane * (unsigned)u.piece_bytes;
        const unsigned row_swz = u.piece_bytes >= 32 ? (((unsigned)lane >> swz_shift) & (unsigned)swz_mask) : 0u;
        int t = 0, staged_n_tile = -1;
        bool ok = ncols > 0;

        // first skip prefetch
        if (EPI == EPI_NARROW_SKIP8 && ok && lane == 0 && (int)blockIdx.x < num_tiles) {
            const int tile0 = blockIdx.x;
            mbar_expect_tx(skip_bar, (uint32_t)(32 * ncols));
            for (int c = 0; c < ncols; c += pcols)
                tma_load_2d(smem_u32(sbuf + (size_t)(c / pcols) * 32 * u.piece_bytes), &tmap_skip, skip_bar,
                            (tile0 % u.n_tiles) * u.block_n + col_lo + c, (tile0 / u.n_tiles) * BLOCK_M + quad * 32);
            skip_issued = 1;
        }

        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++t) {
            const int m_tile = tile / u.n_tiles, n_tile = tile % u.n_tiles;
            const int buf = t & 1;
            const int n0 = n_tile * u.block_n + col_lo;                // first channel of this warp
            if (n_tile != staged_n_tile) {
                __syncwarp();
                for (int lc = lane; lc < ncols; lc += 32) {
                    const int co = n0 + lc;
                    const bool in = co < a.c_out;
                    wp->bias[lc] = in ? __ldg(a.bias + co) : 0;
                    if (a.per_channel) {
                        wp->mul[lc] = in ? __ldg(a.mul + co) : 1;
                        wp->shift[lc] = in ? __ldg(a.shift + co) : 1;
                        wp->h_i[lc] = in ? __ldg(a.h_i + co) : 0;
                    }
                }
                __syncwarp();
                staged_n_tile = n_tile;
            }
            if (!mbar_wait(smem_u32(&sh->tmem_full[buf]), (uint32_t)((t >> 1) & 1), &sh->abort_flag)) {
                give_up(sh, u.status, 4);
                break;
            }
            tc_fence_after();
            if (EPI == EPI_NARROW_SKIP8) {
                if (!mbar_wait(skip_bar, (uint32_t)(t & 1), &sh->abort_flag)) {
                    give_up(sh, u.status, 5);
                    break;
                }
            }
            const long long m = (long long)m_tile * BLOCK_M + quad * 32 + lane;
            const bool row_ok = m < u.m_total;

            for (int pc = 0; pc < ncols; pc += pcols) {
                // the previous TMA store must have finished reading the staging buffer
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                __syncwarp();
                for (int cc = 0; cc < pcols; cc += 16) {
                    const int lc0 = pc + cc;                           // column within this warp's range
                    uint32_t acc[16];
                    tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * u.block_n + col_lo + lc0), acc);
                    const int co0 = n0 + lc0;
                    uint4 sk8 = make_uint4(0, 0, 0, 0);
                    int4 sk32[4];
                    if (EPI == EPI_NARROW_SKIP8) {
                        const unsigned chunk = (unsigned)(cc >> 4);
                        sk8 = *(const uint4 *)(sbuf + (size_t)(pc / pcols) * 32 * u.piece_bytes + row_off + ((chunk ^ row_swz) << 4));
                    } else if ((EPI == EPI_NARROW_SKIPWIDE || EPI == EPI_WIDE) && row_ok && co0 < a.c_out) {
                        if (a.skip_dtype == ICONV_I32) {
#pragma unroll
                            for (int g = 0; g < 4; ++g)
                                if (co0 + 4 * g < a.c_out)
                                    sk32[g] = __ldg((const int4 *)((const int32_t *)a.skip + m * a.skip_c_total + a.skip_c_offset + co0) + g);
                        } else if (a.skip_dtype >= 0) {
                            sk8 = __ldg((const uint4 *)((const uint8_t *)a.skip + m * a.skip_c_total + a.skip_c_offset + co0));
                        }
                    }
                    tmem_ld_wait();
                    const unsigned skw[4] = {sk8.x, sk8.y, sk8.z, sk8.w};
                    unsigned packed[4];
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const int4 b4 = *(const int4 *)(wp->bias + lc0 + 4 * g);
                        const int bias4[4] = {b4.x, b4.y, b4.z, b4.w};
                        int mul4[4] = {q_mul, q_mul, q_mul, q_mul}, shift4[4] = {q_shift, q_shift, q_shift, q_shift};
                        int h4[4] = {q_h_i, q_h_i, q_h_i, q_h_i};
                        if (EPI != EPI_RAW && a.per_channel) {
                            const int4 m4 = *(const int4 *)(wp->mul + lc0 + 4 * g);
                            const int4 s4 = *(const int4 *)(wp->shift + lc0 + 4 * g);
                            const int4 hh = *(const int4 *)(wp->h_i + lc0 + 4 * g);
                            mul4[0] = m4.x; mul4[1] = m4.y; mul4[2] = m4.z; mul4[3] = m4.w;
                            shift4[0] = s4.x; shift4[1] = s4.y; shift4[2] = s4.z; shift4[3] = s4.w;
                            h4[0] = hh.x; h4[1] = hh.y; h4[2] = hh.z; h4[3] = hh.w;
                        }
                        const int s32v[4] = {sk32[g].x, sk32[g].y, sk32[g].z, sk32[g].w};
                        int V[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int k = 4 * g + e;
                            int sv = 0;   // skip value in the integer domain of the addition
                            if (EPI == EPI_NARROW_SKIP8 || EPI == EPI_NARROW_SKIPWIDE || EPI == EPI_WIDE) {
                                if (a.skip_dtype == ICONV_I32) {
                                    sv = s32v[e];
                                } else {
                                    const unsigned byte = (skw[g] >> (8 * e)) & 0xffu;
                                    sv = a.skip_dtype == ICONV_S8 ? (int)(int8_t)byte
                                                                  : (int)byte - (a.skip_dtype == ICONV_U8_RAW128 ? 128 : 0);
                                }
                            }
                            if (EPI == EPI_RAW) {
                                V[e] = (int)acc[k] + bias4[e];
                            } else if (EPI == EPI_NARROW_NOSKIP || EPI == EPI_NARROW_SKIP8) {
                                // every intermediate is proven at plan time to fit 32 bits
                                int y = (int)acc[k] + bias4[e];
                                if (EPI == EPI_NARROW_SKIP8) y += (sv * a.skip_mul + u.skip_half) >> a.skip_shift;
                                y = max(min(y, h4[e]), 0);
                                const unsigned v = ((unsigned)y * (unsigned)mul4[e] + (1u << (shift4[e] - 1))) >> shift4[e];
                                V[e] = min(max((int)v + a.out_zero, a.out_lo), a.out_hi);
                            } else if (EPI == EPI_NARROW_SKIPWIDE) {
                                long long Y = (long long)(int)acc[k] + bias4[e] + round_shift64((long long)sv * a.skip_mul, a.skip_shift);
                                Y = Y < 0 ? 0 : (Y > (long long)h4[e] ? (long long)h4[e] : Y);
                                const unsigned v = ((unsigned)Y * (unsigned)mul4[e] + (1u << (shift4[e] - 1))) >> shift4[e];
                                V[e] = min(max((int)v + a.out_zero, a.out_lo), a.out_hi);
                            } else {
                                long long Y = (long long)(int)acc[k] + bias4[e];
                                if (a.skip_dtype >= 0) Y += round_shift64((long long)sv * a.skip_mul, a.skip_shift);
                                V[e] = a.out_dtype == ICONV_I32
                                           ? (int)Y
                                           : requant_tail(Y, a.brelu, h4[e], mul4[e], shift4[e], a.out_zero, a.out_lo, a.out_hi);
                            }
                        }
                        if (a.out_dtype == ICONV_I32) {
                            const unsigned chunk = (unsigned)((cc >> 2) + g);          // 4 columns = 16 bytes
                            *(int4 *)(obuf + row_off + ((chunk ^ row_swz) << 4)) = make_int4(V[0], V[1], V[2], V[3]);
                        } else {
                            packed[g] = (V[0] & 0xff) | ((V[1] & 0xff) << 8) | ((V[2] & 0xff) << 16) | ((unsigned)(V[3] & 0xff) << 24);
                        }
                    }
                    if (a.out_dtype != ICONV_I32) {
                        const unsigned chunk = (unsigned)(cc >> 4);
                        *(uint4 *)(obuf + row_off + ((chunk ^ row_swz) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    }
                }
                // hand the staged piece to the TMA unit (the store clips rows beyond the last
                // pixel and columns beyond c_out)
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                 ::"l"(&tmap_out), "r"(smem_u32(obuf)), "r"(n0 + pc), "r"(m_tile * BLOCK_M + quad * 32)
                                 : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&sh->tmem_empty[buf]));
                const int next = tile + gridDim.x;
                if (EPI == EPI_NARROW_SKIP8 && next < num_tiles) {     // prefetch the next tile's skip rows
                    mbar_expect_tx(skip_bar, (uint32_t)(32 * ncols));
                    for (int c = 0; c < ncols; c += pcols)
                        tma_load_2d(smem_u32(sbuf + (size_t)(c / pcols) * 32 * u.piece_bytes), &tmap_skip, skip_bar,
                                    (next % u.n_tiles) * u.block_n + col_lo + c, (next / u.n_tiles) * BLOCK_M + quad * 32);
                    ++skip_issued;
                }
            }
        }
        // a warp with no columns still has to release the accumulators it never reads
        if (ncols <= 0) {
            for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++t) {
                const int buf = t & 1;
                if (!mbar_wait(smem_u32(&sh->tmem_full[buf]), (uint32_t)((t >> 1) & 1), &sh->abort_flag)) break;
                if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty[buf]));
            }
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        __syncwarp();
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (sh->abort_flag) {
        // Something gave up: wait (bounded) for the copies and MMAs still in flight so that
        // nothing touches this CTA's shared memory or TMEM after it returns.
        volatile int never = 0;
        if (warp == 0 && lane == 0) {
            for (int s = 0; s < u.stages; ++s) {
                int last = -1;
                for (int i = issued - 1; i >= 0 && i >= issued - u.stages; --i)
                    if (i % u.stages == s) { last = i; break; }
                if (last >= 0) mbar_wait(smem_u32(&sh->full[s]), (uint32_t)((last / u.stages) & 1), &never);
            }
        }
        if (warp == 1 && lane == 0) {
            umma_commit(smem_u32(&sh->drain));
            mbar_wait(smem_u32(&sh->drain), 0, &never);
        }
        if (warp >= 2 && lane == 0 && skip_issued > 0)
            mbar_wait(smem_u32(&sh->skip_full[warp - 2]), (uint32_t)((skip_issued - 1) & 1), &never);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)u.tmem_cols);
    }
}

// ---------------------------------------------------------------- host side
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const int *, const int *, cuuint32_t, cuuint32_t,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;

int load_driver_entry_points()
{
    if (g_encode_tiled && g_encode_im2col) return ICONV_OK;
    cudaDriverEntryPointQueryResult q;
    void *f = nullptr;
    ICONV_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q));
    if (q != cudaDriverEntryPointSuccess || !f) { set_error("cuTensorMapEncodeTiled not available"); return ICONV_ERR_CUDA; }
    g_encode_tiled = (EncodeTiledFn)f;
    ICONV_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f, cudaEnableDefault, &q));
    if (q != cudaDriverEntryPointSuccess || !f) { set_error("cuTensorMapEncodeIm2col not available"); return ICONV_ERR_CUDA; }
    g_encode_im2col = (EncodeIm2colFn)f;
    return ICONV_OK;
}

CUtensorMapSwizzle swizzle_of(int kc)
{
    return kc == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (kc == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

// im2col-mode map over the activation slice: dims {c_in, w, h, n}; the box is KC channels
// of 128 consecutive output pixels; base-pixel coordinates run over [-pad, dim + pad - k].
int encode_activation_map(const iconv_plan_t *p, const void *x, CUtensorMap *map)
{
    const iconv_desc &d = p->d;
    const cuuint64_t dims[4] = {(cuuint64_t)d.c_in, (cuuint64_t)d.w, (cuuint64_t)d.h, (cuuint64_t)d.n};
    const cuuint64_t strides[3] = {(cuuint64_t)d.in_c_total, (cuuint64_t)d.in_c_total * d.w,
                                   (cuuint64_t)d.in_c_total * d.w * d.h};
    const int lower[2] = {-d.pad, -d.pad};
    const int upper[2] = {d.pad - (d.kw - 1), d.pad - (d.kh - 1)};
    const cuuint32_t estr[4] = {1, (cuuint32_t)d.stride, (cuuint32_t)d.stride, 1};
    const CUresult r = g_encode_im2col(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, (void *)((const uint8_t *)x + d.in_c_offset),
                                       dims, strides, lower, upper, (cuuint32_t)p->kc, (cuuint32_t)BLOCK_M, estr,
                                       CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(p->kc),
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeIm2col failed with %d", (int)r);
        return ICONV_ERR_UNSUPPORTED;
    }
    return ICONV_OK;
}

}  // namespace

// Picks the cheapest epilogue whose 32-bit arithmetic is provably exact for this layer.
// After the BReLU clamp 0 <= Y <= h_i, so Y * mul + 2^(shift-1) fits an unsigned 32-bit
// word whenever h_i * mul + 2^(shift-1) < 2^32; an 8-bit skip's rescale fits a signed word
// whenever 255 * skip_mul + 2^(skip_shift-1) < 2^31.
static int choose_epilogue(const iconv_desc &d)
{
    if (d.out_dtype == ICONV_I32) return d.skip_dtype < 0 ? EPI_RAW : EPI_WIDE;
    if (!d.brelu) return EPI_WIDE;
    const int np = d.per_channel ? d.c_out : 1;
    for (int i = 0; i < np; ++i) {
        if (d.shift[i] < 1 || d.shift[i] > 31) return EPI_WIDE;
        if ((unsigned long long)d.h_i[i] * (unsigned long long)d.mul[i] + (1ull << (d.shift[i] - 1)) >= (1ull << 32)) return EPI_WIDE;
    }
    if (d.skip_dtype < 0) return EPI_NARROW_NOSKIP;
    if (d.skip_dtype != ICONV_I32 && d.skip_shift <= 30 &&
        255ll * d.skip_mul + (d.skip_shift ? (1ll << (d.skip_shift - 1)) : 0) < (1ll << 31))
        return EPI_NARROW_SKIP8;
    return EPI_NARROW_SKIPWIDE;
}

// Tiled 2-D map over a channel slice of an NHWC tensor seen as [pixels][channels]; the box
// is one staged piece: 32 pixels x piece_bytes.
static int encode_rows_map(const void *base, int elem_bytes, int c_slice, int c_total, long long pixels,
                           int piece_bytes, CUtensorMap *map)
{
    const cuuint64_t dims[2] = {(cuuint64_t)c_slice, (cuuint64_t)pixels};
    const cuuint64_t strides[1] = {(cuuint64_t)c_total * elem_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)(piece_bytes / elem_bytes), 32};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapSwizzle sw = piece_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : piece_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                  : piece_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
    const CUresult r = g_encode_tiled(map, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_INT32 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
                                      (void *)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                                      CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled (rows map) failed with %d", (int)r);
        return ICONV_ERR_UNSUPPORTED;
    }
    return ICONV_OK;
}

int umma_supported(const iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    const char *why = nullptr;
    if (d.in_dtype == ICONV_U8_RAW128) why = "raw-128 inputs are not GEMM operands";
    else if (d.c_in % 16 || d.in_c_total % 16 || d.in_c_offset % 16) why = "input channels must be multiples of 16";
    else if (d.c_out < 16) why = "c_out below 16";
    else if (d.out_dtype == ICONV_I32 && (d.c_out % 4 || d.out_c_total % 4 || d.out_c_offset % 4)) why = "int32 output channels must be multiples of 4";
    else if (d.out_dtype != ICONV_I32 && (d.c_out % 16 || d.out_c_total % 16 || d.out_c_offset % 16)) why = "8-bit output channels must be multiples of 16";
    else if (d.skip_dtype == ICONV_I32 && (d.skip_c_total % 4 || d.skip_c_offset % 4)) why = "int32 skip channels must be multiples of 4";
    else if (d.skip_dtype >= 0 && d.skip_dtype != ICONV_I32 && (d.skip_c_total % 16 || d.skip_c_offset % 16)) why = "8-bit skip channels must be multiples of 16";
    else if (d.kh > 16 || d.kw > 16 || d.pad > 16 || d.stride > 8) why = "filter, padding or stride beyond the im2col descriptor's range";
    else if ((long long)d.kh * d.kw * ((d.c_in + 127) / 128 * 128) >= (1ll << 24)) why = "reduction too long";
    if (why) {
        set_error("tensor-core path: %s", why);
        return ICONV_ERR_UNSUPPORTED;
    }
    return ICONV_OK;
}

int umma_setup(iconv_plan_t *p)
{
    const iconv_desc &d = p->d;
    int rc = load_driver_entry_points();
    if (rc != ICONV_OK) return rc;

    // channel chunk per pipeline stage: the padded reduction should be as short as possible,
    // ties go to the wider chunk (fewer, larger TMA transactions)
    int best_kc = 0, best_pad = 0;
    for (int kc = 128; kc >= 32; kc /= 2) {
        const int padded = (d.c_in + kc - 1) / kc * kc;
        if (best_kc == 0 || padded < best_pad) { best_kc = kc; best_pad = padded; }
    }
    p->kc = best_kc;
    p->c_in_pad = best_pad;
    p->swizzle_bytes = best_kc;
    const int n_tiles = (d.c_out + 255) / 256;
    p->block_n = ((d.c_out + n_tiles - 1) / n_tiles + 15) / 16 * 16;
    p->c_out_pad = p->block_n * n_tiles;
    // epilogue split: the two warps of a TMEM lane quadrant take the two halves of the tile's
    // columns; a staged piece is the widest power of two (up to 128 bytes) dividing both
    p->half_n = (p->block_n / 2 + 15) / 16 * 16;
    {
        const int esz = d.out_dtype == ICONV_I32 ? 4 : 1;
        const int w0 = p->half_n * esz, w1 = (p->block_n - p->half_n) * esz;
        int pb = 128;
        while (pb > 16 && (w0 % pb || w1 % pb)) pb /= 2;
        p->piece_bytes = pb;
    }
    const int stage_a = BLOCK_M * p->kc;
    const int stage_b = (p->block_n * p->kc + 1023) / 1024 * 1024;
    int stages = SMEM_BUDGET / (stage_a + stage_b);
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    if (stages < 2) { set_error("tensor-core path: tile does not fit shared memory"); return ICONV_ERR_UNSUPPORTED; }
    p->stages = stages;

    // repack weights [c_out][tap][c_in] -> [c_out_pad][tap][c_in_pad], zero filled
    const int taps = d.kh * d.kw;
    const size_t k_pad = (size_t)taps * p->c_in_pad;
    std::vector<int8_t> packed((size_t)p->c_out_pad * k_pad, 0);
    for (int co = 0; co < d.c_out; ++co)
        for (int t = 0; t < taps; ++t)
            memcpy(&packed[(size_t)co * k_pad + (size_t)t * p->c_in_pad], d.weights + ((size_t)co * taps + t) * d.c_in, (size_t)d.c_in);
    ICONV_CUDA_TRY(cudaMalloc((void **)&p->w_packed, packed.size()));
    ICONV_CUDA_TRY(cudaMemcpy(p->w_packed, packed.data(), packed.size(), cudaMemcpyHostToDevice));

    const cuuint64_t dims[2] = {(cuuint64_t)k_pad, (cuuint64_t)p->c_out_pad};
    const cuuint64_t strides[1] = {(cuuint64_t)k_pad};
    const cuuint32_t box[2] = {(cuuint32_t)p->kc, (cuuint32_t)p->block_n};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode_tiled(&p->tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, p->w_packed, dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(p->kc), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed with %d", (int)r);
        return ICONV_ERR_UNSUPPORTED;
    }
    // make sure the activation descriptor can be encoded for this geometry (the address is
    // only stored, never read, so the packed weights stand in for it)
    CUtensorMap probe;
    rc = encode_activation_map(p, (const uint8_t *)p->w_packed - d.in_c_offset, &probe);
    if (rc != ICONV_OK) return rc;
    p->epi = choose_epilogue(d);
    static bool attr_set = false;
    if (!attr_set) {
        ICONV_CUDA_TRY(cudaFuncSetAttribute(umma_conv_kernel<EPI_WIDE>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM));
        ICONV_CUDA_TRY(cudaFuncSetAttribute(umma_conv_kernel<EPI_RAW>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM));
        ICONV_CUDA_TRY(cudaFuncSetAttribute(umma_conv_kernel<EPI_NARROW_NOSKIP>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM));
        ICONV_CUDA_TRY(cudaFuncSetAttribute(umma_conv_kernel<EPI_NARROW_SKIP8>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM));
        ICONV_CUDA_TRY(cudaFuncSetAttribute(umma_conv_kernel<EPI_NARROW_SKIPWIDE>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM));
        attr_set = true;
    }
    return ICONV_OK;
}

int launch_umma(const iconv_plan_t *p, const ConvArgs &a, cudaStream_t stream)
{
    const iconv_desc &d = p->d;
    if (((uintptr_t)a.x % 16) || ((uintptr_t)a.out % 16) || (a.skip && ((uintptr_t)a.skip % 16))) {
        set_error("iconv_forward: tensor pointers must be 16-byte aligned");
        return ICONV_ERR_ALIGN;
    }
    CUtensorMap tmap_x;
    int rc = encode_activation_map(p, a.x, &tmap_x);
    if (rc != ICONV_OK) return rc;

    UmmaArgs u;
    u.m_total = (long long)d.n * p->h_out * p->w_out;
    u.m_tiles = (int)((u.m_total + BLOCK_M - 1) / BLOCK_M);
    u.n_tiles = p->c_out_pad / p->block_n;
    u.block_n = p->block_n;
    u.kc = p->kc;
    u.cchunks = p->c_in_pad / p->kc;
    u.taps = d.kh * d.kw;
    u.stages = p->stages;
    u.stage_a_bytes = BLOCK_M * p->kc;
    u.stage_bytes = u.stage_a_bytes + (p->block_n * p->kc + 1023) / 1024 * 1024;
    int cols = 32;
    while (cols < 2 * p->block_n) cols *= 2;
    u.tmem_cols = cols;
    // instruction descriptor: D = s32, A = u8 or s8, B = s8, both K-major, N/8, M/16
    u.idesc = (2u << 4) | ((d.in_dtype == ICONV_S8 ? 1u : 0u) << 7) | (1u << 10) | ((unsigned)(p->block_n >> 3) << 17) |
              ((unsigned)(BLOCK_M >> 4) << 24);
    // matrix descriptor, upper half: stride between 8-row groups (8 * KC bytes, in 16-byte
    // units), descriptor version 1, swizzle mode (128B = 2, 64B = 4, 32B = 6)
    const unsigned long long layout = p->kc == 128 ? 2ull : (p->kc == 64 ? 4ull : 6ull);
    u.desc_hi = ((unsigned long long)((8 * p->kc) >> 4) << 32) | (1ull << 46) | (layout << 61);
    u.half_n = p->half_n;
    u.piece_bytes = p->piece_bytes;
    const int esz = d.out_dtype == ICONV_I32 ? 4 : 1;
    CUtensorMap tmap_out, tmap_skip;
    rc = encode_rows_map((uint8_t *)a.out + (size_t)d.out_c_offset * esz, esz, d.c_out, d.out_c_total, u.m_total,
                         p->piece_bytes, &tmap_out);
    if (rc != ICONV_OK) return rc;
    tmap_skip = tmap_out;
    if (p->epi == EPI_NARROW_SKIP8) {
        rc = encode_rows_map((const uint8_t *)a.skip + d.skip_c_offset, 1, d.c_out, d.skip_c_total, u.m_total,
                             p->piece_bytes, &tmap_skip);
        if (rc != ICONV_OK) return rc;
    }
    u.status = device_status_ptr();
    if (!u.status) { set_error("device status word not available"); return ICONV_ERR_CUDA; }

    int dev = 0, sms = 0;
    ICONV_CUDA_TRY(cudaGetDevice(&dev));
    ICONV_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const long long tiles = (long long)u.m_tiles * u.n_tiles;
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    const size_t smem = (size_t)u.stages * u.stage_bytes + sizeof(Shared) + 2048 + EPI_SMEM;
    u.skip_half = (d.skip_dtype >= 0 && d.skip_shift > 0 && d.skip_shift <= 31) ? (int)(1u << (d.skip_shift - 1)) : 0;
    switch (p->epi) {
    case EPI_RAW: umma_conv_kernel<EPI_RAW><<<grid, NUM_THREADS, smem, stream>>>(tmap_x, p->tmap_w, tmap_out, tmap_skip, a, u); break;
    case EPI_NARROW_NOSKIP: umma_conv_kernel<EPI_NARROW_NOSKIP><<<grid, NUM_THREADS, smem, stream>>>(tmap_x, p->tmap_w, tmap_out, tmap_skip, a, u); break;
    case EPI_NARROW_SKIP8: umma_conv_kernel<EPI_NARROW_SKIP8><<<grid, NUM_THREADS, smem, stream>>>(tmap_x, p->tmap_w, tmap_out, tmap_skip, a, u); break;
    case EPI_NARROW_SKIPWIDE: umma_conv_kernel<EPI_NARROW_SKIPWIDE><<<grid, NUM_THREADS, smem, stream>>>(tmap_x, p->tmap_w, tmap_out, tmap_skip, a, u); break;
    default: umma_conv_kernel<EPI_WIDE><<<grid, NUM_THREADS, smem, stream>>>(tmap_x, p->tmap_w, tmap_out, tmap_skip, a, u); break;
    }
    ICONV_CUDA_TRY(cudaGetLastError());
    return ICONV_OK;
}

}  // namespace iconv
