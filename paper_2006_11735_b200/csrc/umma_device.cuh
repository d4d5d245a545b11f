// Implicit-GEMM integer convolution on the 5th-generation tensor cores.
//
//   GEMM view   M = n*h_out*w_out output pixels, N = c_out, K = kh*kw*c_in.
//   A operand   activations, fetched by TMA in im2col mode: one load per (filter tap,
//               channel chunk) brings 128 consecutive output pixels x KC channels into
//               shared memory, K-major, hardware-swizzled; out-of-image taps arrive as 0.
//   B operand   int8 weights, repacked at plan time to [c_out_pad][tap][c_in_pad] and
//               fetched by tiled TMA into the same K-major swizzled layout.  When the whole
//               packed filter bank fits beside the pipeline it is loaded once per CTA and
//               stays resident; otherwise its tiles travel through the stages with A.
//   D           int32 accumulators in tensor memory (TMEM): two buffers of up to 256 columns
//               or four of up to 128, so the epilogue of one tile overlaps the MMAs of the next.
//   MMA         tcgen05.mma.cta_group::1.kind::i8, M=128, N=BLOCK_N, K=32 per instruction,
//               u8 (or s8) x s8 -> s32, issued by one thread.
//   Epilogue    up to sixteen warps read TMEM (32 lanes = 32 output pixels each), apply bias,
//               rescaled skip, BReLU, Eq. 4, zero point and saturation, stage 16 output
//               channels per 16-byte shared-memory store and hand 32-row pieces to TMA
//               stores aimed at the layer's channel offset.
//
// Persistent CTAs (one per SM) walk the tiles round-robin.  Warps 0-2 produce (TMA; they take
// the pipeline's k-iterations in turn), warp 3 issues MMAs and owns the TMEM allocation, the
// others run the epilogue.  All mbarrier
// waits are bounded: on expiry the CTA records a code in the device status word, drains
// its copies in flight, frees its TMEM and returns.
//
// Measured on B200 and built into the structure: one thread needs 300-400 cycles per TMA
// instruction and per MMA-group + commit round, whatever the box or instruction size, so
// stages are as large as shared memory allows and nothing but the barrier traffic sits in
// the per-stage loops (no divisions: counters and multiply-shift reciprocals).
//
// This header holds the device code; the kernel instances are compiled in several translation
// units (umma_inst_*.cu), each with launch and opt-in functions for its epilogue variants.
#pragma once

#include <cuda.h>

#include "plan.h"

namespace iconv {

constexpr int BLOCK_M = 128;
constexpr int EPI_WARPS_MAX = 16;
constexpr int NUM_PRODUCERS = 3;          // TMA warps: one thread issues a load per 300-400 cycles, the unit takes three times that
constexpr int MMA_WARP = NUM_PRODUCERS;
constexpr int MMA_WARP2 = 1;           // window mode (one TMA warp): a second MMA issuer
constexpr int MMA_WARP3 = 2;           // ... and a third
constexpr int WIN_ISSUERS = 3;
constexpr int EPI_WARP0 = 4;              // first epilogue warp (a multiple of 4: warp % 4 is its TMEM lane quadrant)
constexpr int NUM_THREADS = 32 * (EPI_WARP0 + EPI_WARPS_MAX);
constexpr int FAST_SKIP_SHIFT = 8;         // the skip shift the clamp-free epilogue forms are compiled for (what iq_skip_sync yields unless the skip is scaled down a lot)
constexpr int SKIP_RING = 3;              // staged skip pieces per epilogue warp at most: the load of a piece is issued ring - 1 pieces ahead of its use
constexpr int EPI_WARP_SMEM = 8192;       // per epilogue warp: two output pieces of up to 4 KB together (int32 outputs)
constexpr int EPI_WARP_SMEM_SMALL = 4096; // ... when the output is 8-bit (pieces of 2 KB) and no 8-bit skip is staged
constexpr int MAX_STAGES = 12;
constexpr int MAX_TMEM_BUFS = 8;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // about two seconds at the boost clock
constexpr int MAX_SMEM = 227 * 1024;
constexpr int RESIDENT_B_MAX = 80 * 1024;

// Epilogue variants, chosen at plan time.  "32-bit" variants rely on bounds the plan proves
// from the layer's actual weights and parameters; whatever cannot be proven runs EPI_WIDE.
enum {
    EPI_WIDE = 0,        // any descriptor: 64-bit products, run-time branches, direct skip loads
    EPI_RAW = 1,         // int32 Y out, no skip: bias add only
    EPI_FAST = 2,        // u8 out, no skip: V = sat_u8((U*mul + C) >> shift), clamps folded into the saturation
    EPI_FAST_SKIP8 = 3,  // ... with an 8-bit skip staged by TMA
    EPI_SAFE = 4,        // explicit BReLU clamp, 32-bit Eq. 4, optional zero point / range tail
    EPI_SAFE_SKIP8 = 5,  // ... with an 8-bit skip staged by TMA
    EPI_SAFE_SKIP32 = 6, // ... with an int32 skip (projection), rescaled in 64 bits
    EPI_PROJ = 7,        // ... with the projection convolution fused: a second accumulator tile beside the first
    EPI_NARROW = 8       // window mode only: fewer than 16 output channels (or unaligned ones), any descriptor; byte stores
};

struct UmmaArgs {
    long long m_total;
    int m_tiles, n_tiles;
    int block_n, kc, cchunks, taps;
    // fused projection (segment 0 of the reduction; 0 iterations when absent)
    int p_iters, p_taps, p_cchunks, p_kw, p_stride, p_pad, proj32;
    int acc_cols;                   // TMEM columns per accumulator buffer: block_n, or 2 * block_n with a projection
    int stages, kg;                 // pipeline stages; k-iterations (slots) per stage
    int slot_a_bytes, slot_bytes, stage_bytes, b_tile_bytes, resident_b;
    int producers;                  // active TMA warps: min(NUM_PRODUCERS, stages * kg)
    int tmem_cols, nbuf, lg_nbuf;   // accumulator buffers (2 or 4; window mode up to 8)
    int epi_warps, cs, bi;          // epilogue warps, column split per tile, tiles in flight
    int part_n;                     // columns one epilogue warp handles per tile
    int piece_bytes;                // row width of one staged output piece (16 ... 128 bytes)
    int epi_warp_bytes;             // staging memory per epilogue warp
    int skip_ring;                  // staged skip pieces per epilogue warp: 2 or SKIP_RING
    unsigned idesc, idesc_p;        // instruction descriptors of the layer and of the projection (operand signedness)
    unsigned long long desc_hi;     // upper 32 bits of the shared-memory matrix descriptors
    // per-layer epilogue scalars (per-channel layers read the arrays instead)
    int q_mul, q_shift, q_half, q_h;
    int skip_half;                  // 2^(skip_shift-1), or 0
    unsigned skip_xor;              // 0x80808080 turns int8 skip bytes into offset-binary
    int tail;                       // 1: out_zero / out_lo / out_hi are not provably no-ops
    int group_uniform;              // per-channel parameters that are equal within every group of 16 channels
    const int32_t *c_a;             // [c_out_pad] per-channel additive constant of the variant
    const int32_t *c_b;             // [c_out_pad] projection bias (64-bit form of EPI_PROJ)
    const int32_t *c_mul, *c_shift, *c_h;   // [c_out_pad] copies for per-channel layers
    int *status;
    // window mode (stride-1 filters: one patch load per tile, every tap a shifted view of it)
    int win_vw, win_bw, win_bh, win_full_width, win_tpi;    // virtual row width, patch width / height, mode, tiles per image
    int win_tap_step;               // patch positions between two horizontal taps (2 with paired taps)
    int win_blocks;                 // 1: tiles are blocks of 8 x 16 output pixels (win_vw = blocks per image row)
    int win_issuers;                // MMA-issuing warps (2 or 3): a divisor of the number of stages, see window_plan
    unsigned desc_hi_a;             // upper descriptor word of the A operand in block mode (8-row groups one patch line apart)
    unsigned div_tpi_mul, div_tpi_shr, div_vw_mul, div_vw_shr;
    // exact division of a tile index by n_tiles and of a pixel index by w_out and by
    // h_out * w_out without a divide instruction: q = umulhi(x, mul) >> shr  (x < 2^31)
    unsigned div_nt_mul, div_nt_shr, div_w_mul, div_w_shr, div_hw_mul, div_hw_shr;
};

__device__ __forceinline__ unsigned fast_div(unsigned x, unsigned mul, unsigned shr)
{
    return mul ? (__umulhi(x, mul) >> shr) : x;
}

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

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
// Non-blocking probe of a barrier phase.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Probe that may suspend the thread in hardware until the phase completes or `hint_ns` pass:
// a suspended thread takes no issue slots from the warps that do the arithmetic.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity, uint32_t hint_ns)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}

// 16-byte shared-memory accesses by 32-bit shared address (no generic-pointer arithmetic)
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Bounded wait of a single-thread role (TMA producer, MMA issuer).  Returns false when the
// limit ran out or another role already gave up.  A few plain probes first (the common short
// wait), then suspending probes; the limit is counted on the SM's own cycle counter, read
// only every 64 failed suspending probes, so a wait that succeeds soon costs no timer read.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, long long limit = WAIT_LIMIT_CYCLES)
{
#pragma unroll 1
    for (int i = 0; i < 4; ++i)
        if (mbar_test_wait(bar, parity)) return true;
    long long t0 = 0;
#pragma unroll 1
    for (uint32_t i = 1;; ++i) {
        if (mbar_try_wait(bar, parity, 2000u)) return true;
        if ((i & 63u) == 0) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit) return false;
        }
    }
}

// The wait of an epilogue warp.  Every lane probes the barrier itself (so each has its own acquire
// and no vote or shuffle is needed on the common path): one plain probe, then probes that suspend
// the warp in hardware until the phase completes or the hint runs out -- a suspended warp takes no
// issue slots from the warps that are doing arithmetic on the same scheduler, which a polling
// loop does.  The limit is counted on the SM's cycle counter, read every 16 failed probes.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, int lane,
                                               long long limit = WAIT_LIMIT_CYCLES)
{
    (void)lane;
    if (mbar_test_wait(bar, parity)) return true;
    bool ok = true;
    long long t0 = 0;
#pragma unroll 1
    for (uint32_t i = 1;; ++i) {
        if (mbar_try_wait(bar, parity, 1000u)) break;
        if ((i & 15u) == 0) {
            if (*abort_flag) { ok = false; break; }
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit) { ok = false; break; }
        }
    }
    return __all_sync(0xffffffffu, ok) != 0;
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
__device__ __forceinline__ void tma_load_tile_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c, int w, int h, int n)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n)
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

// Programmatic dependent launch.  The kernels are launched with programmatic stream serialisation:
// the next kernel of the stream may be scheduled while this one still runs (its CTAs take the SMs
// this kernel's CTAs leave, and run their set-up -- barriers, TMEM, the resident filter bank --
// under the tail of this kernel).  grid_dep_wait blocks until every kernel before this one in the
// stream has completed and its writes are visible: every role executes it before it first touches
// a tensor another kernel may have written (activations, skip); plan-owned constants may be read
// before.  grid_dep_launch tells the scheduler that the kernel after this one may be scheduled.
// Ask for a TMA descriptor ahead of its first use (the first copy otherwise waits for the descriptor fetch).
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// One lane of the (fully active) warp, the lowest: the form the compiler recognises as "a single thread", so that what
// the lane does (TMA issue, barrier arrivals) is issued from uniform registers.
__device__ __forceinline__ bool elect_one()
{
    uint32_t p;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(p));
    return p != 0;
}

// ---- CTA pairs (tcgen05 cta_group::2): two CTAs of a cluster work on one 256-row tile.  Each loads
// its own 128 rows of A and its own half of the B tile; one thread of the even ("leader") CTA issues
// the MMAs, which read both CTAs' shared memory and write both CTAs' TMEM.  No load is multicast.
constexpr uint32_t PEER_MASK = 0xFEFFFFFFu;      // a shared::cluster address with this mask applied names the same offset in the leader CTA

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
}
// loads whose completion is counted on the LEADER CTA's barrier (bar already masked)
__device__ __forceinline__ void tma_load_im2col_4d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c, int w, int h, int n,
                                                        unsigned short off_w, unsigned short off_h)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.im2col.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar)      // arrive on the barrier at this offset in the leader CTA
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar & PEER_MASK) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_i8_pair(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
// one arrival on the barrier at this offset in BOTH CTAs once every MMA issued so far is done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"((unsigned short)3) : "memory");
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

// tcgen05.mma kind::i8 with the descriptors given as 32-bit halves: the issuing thread's
// scalar work per instruction is what bounds narrow tiles, so the per-slice address step is a
// 32-bit add on the low half (start address in 16-byte units; it never carries out of its
// 14-bit field because shared memory is smaller than 256 KB).
__device__ __forceinline__ void umma_i8_split(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                              uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same with separate upper descriptor words for A and B (block-mode patches space A's 8-row
// groups one patch line apart).
__device__ __forceinline__ void umma_i8_split2(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                               uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
template <int KJ>
__device__ __forceinline__ void umma_slot2(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                           uint32_t accumulate_first)
{
    umma_i8_split2(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc, accumulate_first);
#pragma unroll
    for (int j = 1; j < KJ; ++j) umma_i8_split2(d_tmem, a_lo + 2u * j, a_hi, b_lo + 2u * j, b_hi, idesc, 1u);
}
// KJ instructions over the KJ 32-byte K slices of one slot (+2 in 16-byte units per slice).
template <int KJ>
__device__ __forceinline__ void umma_slot(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                          uint32_t accumulate_first)
{
    umma_i8_split(d_tmem, a_lo, b_lo, desc_hi, idesc, accumulate_first);
#pragma unroll
    for (int j = 1; j < KJ; ++j) umma_i8_split(d_tmem, a_lo + 2u * j, b_lo + 2u * j, desc_hi, idesc, 1u);
}
// All slots of one pipeline stage (im2col kernel): slot e of the stage is k-iteration ki + e.  A
// fused projection's iterations (ki < p_iters) go to the second accumulator tile.
template <int KJ>
__device__ __forceinline__ void umma_stage(uint32_t d_tmem, uint32_t block_n, uint32_t a_lo, uint32_t b_lo, uint32_t slot_step,
                                           uint32_t b_step, uint32_t desc_hi, uint32_t idesc, uint32_t idesc_p, int ki, int in_stage,
                                           int p_iters)
{
    for (int e = 0; e < in_stage; ++e, ++ki) {
        const bool in_proj = ki < p_iters;
        umma_slot<KJ>(in_proj ? d_tmem + block_n : d_tmem, a_lo, b_lo, desc_hi, in_proj ? idesc_p : idesc,
                      (uint32_t)(ki != 0 && ki != p_iters));
        a_lo += slot_step;
        b_lo += b_step;
    }
}
// The mbarrier receives one arrival once every MMA issued so far by this thread is done.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Position of the MMA issuer in the stage ring, kept as ready-made operands.
struct IssueRing {
    int stage;
    uint32_t parity, a_lo, full_bar, empty_bar;
};
// `rounds` pipeline stages of one 128-byte k-iteration each into the accumulator at d_tmem:
// wait for the stage, four MMAs (A at a_lo, B right behind it in the stage), commit the stage.
// Run by the whole issuing warp (the ring position is warp-uniform and lives in uniform registers,
// where the MMA takes its operands from); one elected lane issues.  Returns false when a wait gave up.
template <bool PAIR_>
__device__ __forceinline__ bool issue_rounds(IssueRing &g, uint32_t d_tmem, uint32_t idesc, int rounds, int stages, uint32_t a_lo0,
                                             uint32_t stage_step, uint32_t slot_a_step, uint32_t desc_hi32, uint32_t full0,
                                             uint32_t empty0, volatile int *abort_flag)
{
    uint32_t acc = 0;
    for (int ki = 0; ki < rounds; ++ki) {
        if (!mbar_wait_warp(g.full_bar, g.parity, abort_flag, 0)) return false;
        if (!elect_one()) {
        } else if (PAIR_) {
            // one instruction covers both CTAs' 128 rows; the stage is released in both CTAs
            umma_i8_pair(d_tmem, g.a_lo, g.a_lo + slot_a_step, desc_hi32, idesc, acc);
#pragma unroll
            for (int j = 1; j < 4; ++j) umma_i8_pair(d_tmem, g.a_lo + 2u * j, g.a_lo + slot_a_step + 2u * j, desc_hi32, idesc, 1u);
            umma_commit_pair(g.empty_bar);
        } else {
            umma_slot<4>(d_tmem, g.a_lo, g.a_lo + slot_a_step, desc_hi32, idesc, acc);
            umma_commit(g.empty_bar);
        }
        acc = 1;
        const bool wrap = ++g.stage == stages;
        g.stage = wrap ? 0 : g.stage;
        g.parity ^= wrap ? 1u : 0u;
        g.a_lo = wrap ? a_lo0 : g.a_lo + stage_step;
        g.full_bar = wrap ? full0 : g.full_bar + 8u;
        g.empty_bar = wrap ? empty0 : g.empty_bar + 8u;
    }
    return true;
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, int *r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
// The load and the wait for it in one statement: the sixteen values are ready when it returns.
// The epilogue keeps no second load in flight (measured: with sixteen epilogue warps the other
// warps of the scheduler cover the TMEM latency, and the second register block a prefetch needs
// cost more -- spills and moves -- than the overlap returned: 64 -> 256 1x1 with skip, batch 256,
// 108 us with the next group's load in flight, 95 us without).
__device__ __forceinline__ void tmem_ld16_sync(uint32_t taddr, int *r, uint4 dep = make_uint4(0, 0, 0, 0))
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr), "r"(dep.x), "r"(dep.y), "r"(dep.z), "r"(dep.w)    // dep: values that must exist before the registers are reloaded
        : "memory");
}
// 32 bytes to a 32-byte-aligned global address in one store
__device__ __forceinline__ void st_global_32(void *p, uint4 a, uint4 b)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x),
                 "r"(b.y), "r"(b.z), "r"(b.w)
                 : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// d = { sat8(v3), sat8(v2), sat8(v1), sat8(v0) } (v0 in the low byte), unsigned or signed saturation
template <bool SIGNED>
__device__ __forceinline__ unsigned pack4_sat(int v0, int v1, int v2, int v3)
{
    unsigned hi, d;
    if (SIGNED) {
        asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(v3), "r"(v2), "r"(0));
        asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(v1), "r"(v0), "r"(hi));
    } else {
        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(v3), "r"(v2), "r"(0));
        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(v1), "r"(v0), "r"(hi));
    }
    return d;
}

struct Shared {
    unsigned long long skip_full[EPI_WARPS_MAX][SKIP_RING];
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long tmem_full[MAX_TMEM_BUFS];
    unsigned long long tmem_empty[MAX_TMEM_BUFS];
    unsigned long long b_full;
    unsigned long long drain;
    uint32_t tmem_base;
    volatile int abort_flag;
};

__device__ __forceinline__ void give_up(Shared *sh, int *status, int code)
{
    sh->abort_flag = 1;
    atomicCAS(status, 0, code);
}

// The scalars the epilogue needs, copied once per thread into registers (read through the kernel
// parameters inside the unrolled element loops they cost an indexed constant load each).
struct EpiScalars {
    int q_mul, q_shift, q_half, q_h;
    int skip_mul, skip_shift;
    unsigned skip_xor;
    int out_zero, out_lo, out_hi, tail;
    int per_channel, group_uniform, proj32, brelu, skip_dtype, out_dtype, c_out;
};

__device__ __forceinline__ EpiScalars epi_scalars(const ConvArgs &a, const UmmaArgs &u)
{
    EpiScalars e;
    e.q_mul = u.q_mul; e.q_shift = u.q_shift; e.q_h = u.q_h;
    // y * q_mul + q_half has two warp-uniform operands and the multiply-add takes only one from a
    // uniform register: left to itself the compiler re-creates the other in a vector register for
    // every element (one move per output).  An opaque move pins q_half in a vector register.
    asm volatile("mov.b32 %0, %1;" : "=r"(e.q_half) : "r"(u.q_half));
    e.skip_mul = a.skip_mul; e.skip_shift = a.skip_shift; e.skip_xor = u.skip_xor;
    e.out_zero = a.out_zero; e.out_lo = a.out_lo; e.out_hi = a.out_hi; e.tail = u.tail;
    e.per_channel = a.per_channel && !u.group_uniform; e.group_uniform = u.group_uniform; e.proj32 = u.proj32; e.brelu = a.brelu; e.skip_dtype = a.skip_dtype;
    e.out_dtype = a.out_dtype; e.c_out = a.c_out;
    return e;
}

// Per-channel parameters that are uniform within each group of 16 channels (merged sibling
// branches): the group's own scalars take the place of the layer's, three loads per group.
__device__ __forceinline__ EpiScalars group_scalars(const EpiScalars &s, const UmmaArgs &u, int co0)
{
    EpiScalars g = s;
    if (s.group_uniform) {
        g.q_mul = __ldg(u.c_mul + co0); g.q_shift = __ldg(u.c_shift + co0); g.q_h = __ldg(u.c_h + co0);
        g.q_half = (int)(1u << (g.q_shift - 1));
    }
    return g;
}

// BReLU clamp + 32-bit Eq. 4 (+ zero point / range when they are not provable no-ops)
__device__ __forceinline__ int requant32(int y, int h, int mul, int half, int shift, const EpiScalars &s)
{
    y = max(min(y, h), 0);
    int v = (int)(((unsigned)y * (unsigned)mul + (unsigned)half) >> shift);
    if (s.tail) v = min(max(v + s.out_zero, s.out_lo), s.out_hi);
    return v;
}

// Eq. 4 parameters of output channel co: the layer's scalars, or (PC) the channel's own.
template <bool PC>
__device__ __forceinline__ void chan_params(const EpiScalars &s, const UmmaArgs &u, int co, int &h, int &mul, int &half, int &shift)
{
    if (PC) {
        h = __ldg(u.c_h + co); mul = __ldg(u.c_mul + co); shift = __ldg(u.c_shift + co); half = (int)(1u << (shift - 1));
    } else {
        h = s.q_h; mul = s.q_mul; shift = s.q_shift; half = s.q_half;
    }
}

// One group of 16 consecutive output channels of one pixel: accumulators in, 16 output
// values (8-bit variants) or 16 int32 (raw) out.  ca4: the variant's per-channel additive
// constants of the group; `sk`: the 16 staged skip bytes; accp: the projection's accumulators.
// PC: per-channel mul / shift / h_i.
template <int EPI, bool PC>
__device__ __forceinline__ void epilogue16_pc(const int *acc, const int *accp, int *V, const int4 *ca4, int co0, long long m, bool row_ok,
                                              uint4 sk, const EpiScalars &s, const ConvArgs &a, const UmmaArgs &u)
{
    int ca[16];
#pragma unroll
    for (int g = 0; g < 4; ++g) { ca[4 * g] = ca4[g].x; ca[4 * g + 1] = ca4[g].y; ca[4 * g + 2] = ca4[g].z; ca[4 * g + 3] = ca4[g].w; }
    int h, mul, half, shift;

    if (EPI == EPI_RAW) {
#pragma unroll
        for (int k = 0; k < 16; ++k) V[k] = acc[k] + ca[k];
        return;
    }
    if (EPI == EPI_FAST) {
        // (U + b) * mul + half = U * mul + C with C = b * mul + half; the shift is arithmetic and the
        // u8 saturation that follows stands for both BReLU clamps (proven at plan time)
#pragma unroll
        for (int k = 0; k < 16; ++k) V[k] = (acc[k] * s.q_mul + ca[k]) >> s.q_shift;
        return;
    }
    if (EPI == EPI_FAST_SKIP8 || EPI == EPI_SAFE_SKIP8) {
        // Y = U + ((sv * skip_mul + C) >> skip_shift) with C = (b << skip_shift) + skip_half - z * skip_mul,
        // where sv is the stored byte as an unsigned number and z its zero (0, or 128 for raw-128 and
        // offset-binary int8): the bias rides inside the rounding shift, which is exact.
        const unsigned w4[4] = {sk.x ^ s.skip_xor, sk.y ^ s.skip_xor, sk.z ^ s.skip_xor, sk.w ^ s.skip_xor};
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const int sv = (int)__byte_perm(w4[k >> 2], 0, 0x4440 + (k & 3));
            // (the fast form is planned only for the usual skip shift of 8: as an immediate, shift and add
            // become one instruction)
            const int y = acc[k] + ((sv * s.skip_mul + ca[k]) >> (EPI == EPI_FAST_SKIP8 ? FAST_SKIP_SHIFT : s.skip_shift));
            if (EPI == EPI_FAST_SKIP8) {
                V[k] = (y * s.q_mul + s.q_half) >> s.q_shift;
            } else {
                chan_params<PC>(s, u, co0 + k, h, mul, half, shift);
                V[k] = requant32(y, h, mul, half, shift, s);
            }
        }
        return;
    }
    if (EPI == EPI_PROJ) {
        // S = accp + b_p is the projection's int32 Y.  32-bit form (bounds proven at plan time):
        // Y = U + ((accp * skip_mul + C) >> skip_shift), C = b_p * skip_mul + 2^(skip_shift-1) + (b << skip_shift);
        // otherwise the rescale runs in 64 bits with the two biases apart.
        if (!PC && s.proj32 == 2) {
            // as EPI_FAST: no clamp before Eq. 4, the u8 saturation that follows stands for both (proven at
            // plan time, and planned only for the usual skip shift of 8)
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const int y = acc[k] + ((accp[k] * s.skip_mul + ca[k]) >> FAST_SKIP_SHIFT);
                V[k] = (y * s.q_mul + s.q_half) >> s.q_shift;
            }
        } else if (s.proj32) {
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                chan_params<PC>(s, u, co0 + k, h, mul, half, shift);
                V[k] = requant32(acc[k] + ((accp[k] * s.skip_mul + ca[k]) >> s.skip_shift), h, mul, half, shift, s);
            }
        } else {
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                chan_params<PC>(s, u, co0 + k, h, mul, half, shift);
                long long Y = (long long)acc[k] + ca[k] +
                              round_shift64(((long long)accp[k] + __ldg(u.c_b + co0 + k)) * s.skip_mul, s.skip_shift);
                Y = Y < 0 ? 0 : (Y > (long long)h ? (long long)h : Y);
                V[k] = requant32((int)Y, h, mul, half, shift, s);
            }
        }
        return;
    }
    if (EPI == EPI_SAFE) {
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            chan_params<PC>(s, u, co0 + k, h, mul, half, shift);
            V[k] = requant32(acc[k] + ca[k], h, mul, half, shift, s);
        }
        return;
    }
    // EPI_SAFE_SKIP32 and EPI_WIDE read the skip straight from global memory
    const bool have = s.skip_dtype >= 0 && row_ok && co0 < s.c_out;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        int ss[4] = {0, 0, 0, 0};
        if (have && s.skip_dtype == ICONV_I32 && co0 + 4 * g < s.c_out) {
            const int4 t = __ldg((const int4 *)((const int32_t *)a.skip + m * a.skip_c_total + a.skip_c_offset + co0) + g);
            ss[0] = t.x; ss[1] = t.y; ss[2] = t.z; ss[3] = t.w;
        } else if (have && s.skip_dtype != ICONV_I32) {
            const unsigned w = __ldg((const unsigned *)((const uint8_t *)a.skip + m * a.skip_c_total + a.skip_c_offset + co0) + g);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const unsigned byte = (w >> (8 * e)) & 0xffu;
                ss[e] = s.skip_dtype == ICONV_S8 ? (int)(int8_t)byte : (int)byte - (s.skip_dtype == ICONV_U8_RAW128 ? 128 : 0);
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int k = 4 * g + e;
            chan_params<PC>(s, u, co0 + k, h, mul, half, shift);
            long long Y = (long long)acc[k] + ca[k];
            if (s.skip_dtype >= 0) Y += round_shift64((long long)ss[e] * s.skip_mul, s.skip_shift);
            if (EPI == EPI_SAFE_SKIP32) {
                Y = Y < 0 ? 0 : (Y > (long long)h ? (long long)h : Y);
                V[k] = requant32((int)Y, h, mul, half, shift, s);
            } else {
                V[k] = s.out_dtype == ICONV_I32 ? (int)Y : requant_tail(Y, s.brelu, h, mul, shift, s.out_zero, s.out_lo, s.out_hi);
            }
        }
    }
}

template <int EPI>
__device__ __forceinline__ void epilogue16(const int *acc, const int *accp, int *V, const int4 *ca4, int co0, long long m, bool row_ok,
                                           uint4 sk, const EpiScalars &s, const ConvArgs &a, const UmmaArgs &u)
{
    // the fast forms are planned for per-layer parameters only
    if (EPI != EPI_RAW && EPI != EPI_FAST && EPI != EPI_FAST_SKIP8 && s.per_channel)
        epilogue16_pc<EPI, true>(acc, accp, V, ca4, co0, m, row_ok, sk, s, a, u);
    else
        epilogue16_pc<EPI, false>(acc, accp, V, ca4, co0, m, row_ok, sk, s, a, u);
}


// ISSUE selects the MMA issuer's code at compile time: 0 the general loop, 1 the long
// reductions (one k-iteration per stage, B in the stage), 2 the tiles that fit one stage with a
// resident filter bank.  The issuer is a lone thread: code it never runs still costs it
// instruction fetches, so each instance carries only its own path.
template <int EPI, int ISSUE>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_conv_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                 const __grid_constant__ CUtensorMap tmap_out, const __grid_constant__ CUtensorMap tmap_skip,
                 const __grid_constant__ ConvArgs a, const __grid_constant__ UmmaArgs u)
{
    constexpr bool SKIP8 = (EPI == EPI_FAST_SKIP8 || EPI == EPI_SAFE_SKIP8);
    // ISSUE 3: the long-reduction path on CTA pairs.  A "tile" is then 256 pixels x block_n: this CTA's
    // pixel tile is 2 * (tile / n_tiles) + rank, u.m_tiles counts pixel-tile pairs, the grid is walked pair by pair.
    constexpr bool PAIR = ISSUE == 3;
    const uint32_t rank = PAIR ? __shfl_sync(0xffffffffu, cluster_rank(), 0) : 0u;    // (known to the compiler as warp-uniform)
    const int tile0 = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, tile_stride = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    extern __shared__ uint8_t smem_raw[];
    // tiles need the alignment of the widest swizzle pattern (8 rows x 128 bytes)
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *b_res = tiles + (size_t)u.stages * u.stage_bytes;                 // resident filter bank (may be empty)
    const int k_iters = u.p_iters + u.taps * u.cchunks;
    Shared *sh = (Shared *)(b_res + (u.resident_b ? (size_t)u.b_tile_bytes * k_iters * u.n_tiles : 0));
    uint8_t *epi_smem = (uint8_t *)(((uintptr_t)(sh + 1) + 1023) & ~(uintptr_t)1023);

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);    // the same value in every lane, and known to the compiler as such: per-warp addresses and coordinates live in uniform registers
    const int lane = threadIdx.x & 31;
    const int num_tiles = u.m_tiles * u.n_tiles;

    if (threadIdx.x == 32) {     // (a lane of a producer warp that has nothing else to do yet)
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_w);
        prefetch_tensormap(&tmap_out);
        if (SKIP8 || EPI == EPI_PROJ) prefetch_tensormap(&tmap_skip);
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < u.stages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), (uint32_t)u.kg);     // one arrival per slot
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < u.nbuf; ++b) {
            mbar_init(smem_u32(&sh->tmem_full[b]), 1);
            mbar_init(smem_u32(&sh->tmem_empty[b]), (uint32_t)((PAIR ? 8 : 4) * u.cs));     // pairs: both CTAs' epilogue warps arrive at the leader
        }
        for (int w = 0; w < EPI_WARPS_MAX * SKIP_RING; ++w) mbar_init(smem_u32(&sh->skip_full[0][0]) + 8u * (uint32_t)w, 1);
        mbar_init(smem_u32(&sh->b_full), 1);
        mbar_init(smem_u32(&sh->drain), 1);
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        grid_dep_launch();
    }
    if (warp == MMA_WARP) {
        if (PAIR) tmem_alloc_pair(smem_u32(&sh->tmem_base), (uint32_t)u.tmem_cols);
        else tmem_alloc(smem_u32(&sh->tmem_base), (uint32_t)u.tmem_cols);
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();            // the peer's barriers exist before anything arrives at them
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    int last_stage = -1;   // producer: stage and phase of the last load this warp issued
    uint32_t last_parity = 0;
    int b_issued = 0;      // producer: resident filter bank requested
    int skip_issued = 0, skip_taken = 0;   // epilogue lane 0: skip pieces requested / waited for

    if (warp < NUM_PRODUCERS) {
        // ---------------------------------------------------------------- TMA producers
        // Producer j of P issues the loads of k-iterations j, j + P, j + 2P, ... (counted across
        // tiles).  A stage holds `kg` k-iterations (slots) behind one pair of barriers, so the MMA
        // issuer pays its wait + commit round once per kg.  P never exceeds stages * kg: a parity
        // wait cannot tell a barrier that is two phases behind from one that is done, and a
        // producer that skips P iterations only knows the consumer's progress up to its own
        // previous iteration.
        if (lane == 0 && warp < u.producers && tile0 < num_tiles) {
            if (u.resident_b && warp == 0) {
                const uint32_t bf = smem_u32(&sh->b_full);
                mbar_expect_tx(bf, (uint32_t)(u.block_n * u.kc * k_iters * u.n_tiles));
                for (int nt = 0; nt < u.n_tiles; ++nt)
                    for (int ki = 0; ki < k_iters; ++ki)
                        tma_load_2d(smem_u32(b_res + (size_t)(nt * k_iters + ki) * u.b_tile_bytes), &tmap_w, bf,
                                    ki * u.kc, nt * u.block_n);
                b_issued = 1;
            }
            grid_dep_wait();                        // the activations may come from the kernel before this one
            int stage = 0, slot = 0, turn = warp;   // turn: iterations until this producer's next one
            uint32_t parity = 0;
            bool ok = true;
            const int hw = a.h_out * a.w_out;
            // (pairs: every CTA brings its own pixel rows and its own half of the B tile; the bytes of both
            // CTAs are counted on the leader's barrier, which the leader arms)
            const uint32_t tx = PAIR ? (uint32_t)(2 * (BLOCK_M * u.kc + (u.block_n >> 1) * u.kc))
                                     : (uint32_t)(BLOCK_M * u.kc + (u.resident_b ? 0 : u.block_n * u.kc));
            for (int tile = tile0; tile < num_tiles && ok; tile += tile_stride) {
                const int m_unit = (int)fast_div((unsigned)tile, u.div_nt_mul, u.div_nt_shr);
                const int n_tile = tile - m_unit * u.n_tiles;
                const int m_tile = PAIR ? 2 * m_unit + (int)rank : m_unit;
                const unsigned m0 = (unsigned)m_tile * BLOCK_M;
                const int img = (int)fast_div(m0, u.div_hw_mul, u.div_hw_shr);
                const unsigned rem = m0 - (unsigned)img * (unsigned)hw;
                const int p = (int)fast_div(rem, u.div_w_mul, u.div_w_shr);
                const int q = (int)rem - p * a.w_out;
                int kx = 0, ki = 0;
                // segment 0: the fused projection (its own input tensor, stride and padding)
                if (EPI == EPI_PROJ) {
                    const int cwp = q * u.p_stride - u.p_pad, chp = p * u.p_stride - u.p_pad;
                    int r = 0, s = 0;
                    for (int tap = 0; tap < u.p_taps && ok; ++tap) {
                        for (int cc = 0; cc < u.p_cchunks; ++cc, ++ki, kx += u.kc) {
                            if (turn == 0) {
                                if (!mbar_wait(smem_u32(&sh->empty[stage]), parity ^ 1u, &sh->abort_flag)) {
                                    give_up(sh, u.status, 1);
                                    ok = false;
                                    break;
                                }
                                const uint32_t full = smem_u32(&sh->full[stage]);
                                const uint32_t sa = smem_u32(tiles + (size_t)stage * u.stage_bytes + (size_t)slot * u.slot_bytes);
                                mbar_expect_tx(full, tx);
                                tma_load_im2col_4d(sa, &tmap_skip, full, cc * u.kc, cwp, chp, img, (unsigned short)s,
                                                   (unsigned short)r);
                                if (!u.resident_b) tma_load_2d(sa + u.slot_a_bytes, &tmap_w, full, kx, n_tile * u.block_n);
                                last_stage = stage;
                                last_parity = parity;
                                turn = u.producers;
                            }
                            --turn;
                            if (++slot == u.kg) {
                                slot = 0;
                                if (++stage == u.stages) { stage = 0; parity ^= 1u; }
                            }
                        }
                        if (++s == u.p_kw) { s = 0; ++r; }
                    }
                }
                const int cw = q * a.stride - a.pad, ch = p * a.stride - a.pad;
                int r = 0, s = 0;
                for (int tap = 0; tap < u.taps && ok; ++tap) {
                    for (int cc = 0; cc < u.cchunks; ++cc, ++ki, kx += u.kc) {
                        const bool tile_end = ki == k_iters - 1;
                        if (turn == 0) {
                            if (!mbar_wait(smem_u32(&sh->empty[stage]), parity ^ 1u, &sh->abort_flag)) {
                                give_up(sh, u.status, 1);
                                ok = false;
                                break;
                            }
                            const uint32_t full = smem_u32(&sh->full[stage]);
                            const uint32_t sa = smem_u32(tiles + (size_t)stage * u.stage_bytes + (size_t)slot * u.slot_bytes);
                            if (PAIR) {
                                if (rank == 0) mbar_expect_tx(full, tx);
                                tma_load_im2col_4d_pair(sa, &tmap_x, full & PEER_MASK, cc * u.kc, cw, ch, img, (unsigned short)s, (unsigned short)r);
                                tma_load_2d_pair(sa + u.slot_a_bytes, &tmap_w, full & PEER_MASK, kx, n_tile * u.block_n + (int)rank * (u.block_n >> 1));
                            } else {
                            mbar_expect_tx(full, tx);
                            tma_load_im2col_4d(sa, &tmap_x, full, cc * u.kc, cw, ch, img, (unsigned short)s,
                                               (unsigned short)r);
                            if (!u.resident_b) tma_load_2d(sa + u.slot_a_bytes, &tmap_w, full, kx, n_tile * u.block_n);
                            }
                            // a tile's last stage may be short: stand in for its missing slots
                            if (tile_end)
                                for (int e = slot + 1; e < u.kg; ++e) mbar_arrive(full);
                            last_stage = stage;
                            last_parity = parity;
                            turn = u.producers;
                        }
                        --turn;
                        if (++slot == u.kg || tile_end) {
                            slot = 0;
                            if (++stage == u.stages) { stage = 0; parity ^= 1u; }
                        }
                    }
                    if (++s == a.kw) { s = 0; ++r; }
                }
            }
        }
        __syncwarp();
    } else if (warp == MMA_WARP) {
        // ---------------------------------------------------------------- MMA issuer
        // The whole warp walks the tiles and waits (warp-uniform control flow: ring positions and
        // descriptors are computed in uniform registers, where the MMA instruction takes them from);
        // one elected lane issues.  (The TMA producers stay single-lane loops: the same change
        // measured no different there.)
        if (tile0 < num_tiles && (!PAIR || rank == 0)) {
            int t = 0, stage = 0;
            uint32_t parity = 0;
            bool ok = true;
            if (u.resident_b && !mbar_wait_warp(smem_u32(&sh->b_full), 0, &sh->abort_flag, lane)) {
                give_up(sh, u.status, 6);
                ok = false;
            }
            const int kj = u.kc >> 5;   // MMAs per k-iteration: 32 bytes of K each
            const uint32_t desc_hi32 = (uint32_t)(u.desc_hi >> 32);
            const uint32_t a_lo0 = ((smem_u32(tiles) & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t stage_step = (uint32_t)u.stage_bytes >> 4, slot_step = (uint32_t)u.slot_bytes >> 4;
            const uint32_t slot_a_step = (uint32_t)u.slot_a_bytes >> 4;
            const uint32_t b_step = (uint32_t)(u.resident_b ? u.b_tile_bytes : u.slot_bytes) >> 4;
            constexpr bool simple = ISSUE == 1 || ISSUE == 3, one_round = ISSUE == 2;
            const uint32_t full0 = smem_u32(&sh->full[0]), empty0 = smem_u32(&sh->empty[0]);
            for (int tile = tile0; tile < num_tiles && ok; tile += tile_stride, ++t) {
                const int buf = t & (u.nbuf - 1);
                if (!mbar_wait_warp(smem_u32(&sh->tmem_empty[buf]), (uint32_t)(((t >> u.lg_nbuf) & 1) ^ 1), &sh->abort_flag, lane)) {
                    give_up(sh, u.status, 2);
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * u.acc_cols);
                uint32_t sb = 0;
                if (u.resident_b) {
                    const int m_tile = (int)fast_div((unsigned)tile, u.div_nt_mul, u.div_nt_shr);
                    sb = ((smem_u32(b_res + (size_t)((tile - m_tile * u.n_tiles) * k_iters) * u.b_tile_bytes) & 0x3FFFFu) >> 4) | (1u << 16);
                }
                if (one_round) {
                    // The short reductions (the whole tile in one stage, the filter bank resident): one
                    // wait, the tile's MMAs, two commits, with as few branches as the lone thread can do with.
                    const uint32_t full_bar = full0 + 8u * (uint32_t)stage;
                    if (!mbar_wait_warp(full_bar, parity, &sh->abort_flag, lane)) {
                        give_up(sh, u.status, 3);
                        break;
                    }
                    if (elect_one()) {
                        uint32_t a_lo = a_lo0 + (uint32_t)stage * stage_step, b_lo = sb;
                        umma_slot<4>(d_tmem, a_lo, b_lo, desc_hi32, u.idesc, 0u);
                        for (int e = 1; e < k_iters; ++e) {
                            a_lo += slot_step;
                            b_lo += b_step;
                            umma_slot<4>(d_tmem, a_lo, b_lo, desc_hi32, u.idesc, 1u);
                        }
                        umma_commit(empty0 + 8u * (uint32_t)stage);
                        umma_commit(smem_u32(&sh->tmem_full[buf]));
                    }
                    const bool wrap = ++stage == u.stages;
                    stage = wrap ? 0 : stage;
                    parity ^= wrap ? 1u : 0u;
                    continue;
                }
                if (simple) {
                    // The long reductions (one 128-byte k-iteration per stage, B riding in the stage):
                    // a round per stage of nothing but the wait, four MMAs and the commit.  Every
                    // taken branch of this lone thread costs tens of cycles that the tensor pipe's
                    // short queue does not cover, and here there are 6 to 36 rounds per tile.  A fused
                    // projection's iterations come first, into the second accumulator tile.
                    IssueRing ring;
                    ring.stage = stage; ring.parity = parity;
                    ring.a_lo = a_lo0 + (uint32_t)stage * stage_step;
                    ring.full_bar = full0 + 8u * (uint32_t)stage; ring.empty_bar = empty0 + 8u * (uint32_t)stage;
                    if (EPI == EPI_PROJ && u.p_iters) {
                        ok = issue_rounds<PAIR>(ring, d_tmem + (uint32_t)u.block_n, u.idesc_p, u.p_iters, u.stages, a_lo0, stage_step, slot_a_step,
                                                desc_hi32, full0, empty0, &sh->abort_flag);
                        if (ok) ok = issue_rounds<PAIR>(ring, d_tmem, u.idesc, k_iters - u.p_iters, u.stages, a_lo0, stage_step, slot_a_step,
                                                        desc_hi32, full0, empty0, &sh->abort_flag);
                    } else {
                        ok = issue_rounds<PAIR>(ring, d_tmem, u.idesc, k_iters, u.stages, a_lo0, stage_step, slot_a_step, desc_hi32, full0, empty0,
                                                &sh->abort_flag);
                    }
                    stage = ring.stage; parity = ring.parity;
                    if (!ok) give_up(sh, u.status, 3);
                    else if (elect_one()) { if (PAIR) umma_commit_pair(smem_u32(&sh->tmem_full[buf])); else umma_commit(smem_u32(&sh->tmem_full[buf])); }
                    continue;
                }
                for (int ki = 0; ISSUE == 0 && ki < k_iters;) {
                    if (!mbar_wait_warp(smem_u32(&sh->full[stage]), parity, &sh->abort_flag, lane)) {
                        give_up(sh, u.status, 3);
                        ok = false;
                        break;
                    }
                    // low descriptor halves: start address in 16-byte units, bit 16 = the (ignored) leading offset
                    uint32_t a_lo = a_lo0 + (uint32_t)stage * stage_step;
                    uint32_t b_lo = u.resident_b ? sb : a_lo + slot_a_step;
                    const int in_stage = min(u.kg, k_iters - ki);
                    if (elect_one()) {
                        if (kj == 4) umma_stage<4>(d_tmem, (uint32_t)u.block_n, a_lo, b_lo, slot_step, b_step, desc_hi32, u.idesc, u.idesc_p, ki, in_stage, EPI == EPI_PROJ ? u.p_iters : 0);
                        else if (kj == 2) umma_stage<2>(d_tmem, (uint32_t)u.block_n, a_lo, b_lo, slot_step, b_step, desc_hi32, u.idesc, u.idesc_p, ki, in_stage, EPI == EPI_PROJ ? u.p_iters : 0);
                        else umma_stage<1>(d_tmem, (uint32_t)u.block_n, a_lo, b_lo, slot_step, b_step, desc_hi32, u.idesc, u.idesc_p, ki, in_stage, EPI == EPI_PROJ ? u.p_iters : 0);
                        umma_commit(smem_u32(&sh->empty[stage]));   // frees the stage when these MMAs are done
                    }
                    ki += in_stage;
                    if (u.resident_b) sb = b_lo + (uint32_t)in_stage * b_step;
                    if (++stage == u.stages) { stage = 0; parity ^= 1u; }
                }
                if (ok && elect_one()) umma_commit(smem_u32(&sh->tmem_full[buf]));
            }
        }
        __syncwarp();
    } else if (warp >= EPI_WARP0 && warp < EPI_WARP0 + u.epi_warps) {
        // ---------------------------------------------------------------- epilogue
        // warp % 4 fixes the TMEM lane quadrant (32 output pixels) a warp may read.  The warps
        // of a quadrant form `cs * bi` slots: `cs` slots split a tile's columns, `bi` groups
        // of them take alternate tiles (each on its own accumulator buffer).  A warp works
        // alone: it prefetches its own part of an 8-bit skip tensor by TMA, stages its
        // outputs in its own two swizzled shared-memory pieces and writes them with its own
        // TMA stores (which also clip the ragged last tile and the channels beyond c_out), so
        // no cross-warp barrier exists that a warp which gave up could strand.
        grid_dep_wait();                            // the skip operand may come from the kernel before this one
        const int ew = warp - EPI_WARP0;
        const int quad = warp & 3;
        const int slot = ew >> 2;
        const int part = slot % u.cs;
        const int turn = slot / u.cs;
        const int col_lo = part * u.part_n;
        const int ncols = min(u.block_n - col_lo, u.part_n);
        constexpr int esz = (EPI == EPI_RAW) ? 4 : 1;
        const int esz_rt = (EPI == EPI_WIDE && a.out_dtype == ICONV_I32) ? 4 : esz;
        const int pb = u.piece_bytes;
        const int pcols = pb / esz_rt;                                // columns per staged piece
        const int piece_smem = 32 * pb;
        const uint32_t obuf = smem_u32(epi_smem + (size_t)ew * u.epi_warp_bytes);   // two output pieces of 32 rows x piece_bytes
        const uint32_t sbuf = obuf + 2u * (uint32_t)piece_smem;                      // ring of SKIP_RING skip pieces (8-bit skip variants)
        const uint32_t skip_bar0 = smem_u32(&sh->skip_full[ew][0]);
        const int swz_shift = pb == 128 ? 0 : (pb == 64 ? 1 : 2);
        const unsigned row_off = (unsigned)lane * (unsigned)pb;
        const unsigned row_swz16 = pb >= 32 ? ((((unsigned)lane >> swz_shift) & (unsigned)(pb / 16 - 1)) << 4) : 0u;   // XOR mask of the row's 16-byte chunks
        const int tile_step = u.bi * tile_stride;
        const EpiScalars es = epi_scalars(a, u);
        int pieces = 0;
        bool ok = true;

        // The 8-bit skip operand arrives by TMA, piece by piece (32 pixels x piece_bytes), into a ring of
        // SKIP_RING buffers: the load of a piece is issued when the piece SKIP_RING places before it has
        // been consumed, i.e. two pieces of epilogue work ahead of its use, which covers the DRAM latency.
        // (pf_tile, pf_pc): the next piece to request; lane 0 only.
        int pf_tile = tile0 + turn * tile_stride, pf_pc = 0;
        auto request_skip_piece = [&](int ring_slot) {
            if (pf_tile >= num_tiles) return;
            const int mt = (int)fast_div((unsigned)pf_tile, u.div_nt_mul, u.div_nt_shr);
            const uint32_t bar = skip_bar0 + 8u * (uint32_t)ring_slot;
            mbar_expect_tx(bar, (uint32_t)piece_smem);
            tma_load_2d(sbuf + (uint32_t)(ring_slot * piece_smem), &tmap_skip, bar, (pf_tile - mt * u.n_tiles) * u.block_n + col_lo + pf_pc,
                        (PAIR ? 2 * mt + (int)rank : mt) * BLOCK_M + quad * 32);
            ++skip_issued;
            pf_pc += pcols;
            if (pf_pc >= ncols) { pf_pc = 0; pf_tile += tile_step; }
        };
        const int skip_ring = u.skip_ring;
        if (SKIP8 && lane == 0)
            for (int r = 0; r < skip_ring; ++r) request_skip_piece(r);
        int ring = 0;
        uint32_t ring_parity = 0;

        for (int t = turn, tile = tile0 + turn * tile_stride; tile < num_tiles && ok; t += u.bi, tile += tile_step) {
            const int m_unit = (int)fast_div((unsigned)tile, u.div_nt_mul, u.div_nt_shr);
            const int n_tile = tile - m_unit * u.n_tiles;
            const int m_tile = PAIR ? 2 * m_unit + (int)rank : m_unit;
            const int buf = t & (u.nbuf - 1);
            const int n0 = n_tile * u.block_n + col_lo;                // first channel of this warp
            if (!mbar_wait_warp(smem_u32(&sh->tmem_full[buf]), (uint32_t)((t >> u.lg_nbuf) & 1), &sh->abort_flag, lane)) {
                give_up(sh, u.status, 4);
                break;
            }
            tc_fence_after();
            const long long m = (long long)m_tile * BLOCK_M + quad * 32 + lane;
            const bool row_ok = m < u.m_total;
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * u.acc_cols + col_lo);
            int acc[16], accp[16];
            uint4 o_prev = make_uint4(0, 0, 0, 0);       // the packed outputs of the group before: the reload of acc is ordered after them

            for (int pc = 0; pc < ncols && ok; pc += pcols, ++pieces) {
                const uint32_t ob = obuf + (uint32_t)((pieces & 1) * piece_smem);
                const uint32_t ob_row = ob + row_off;                                              // this lane's staged output row
                const uint32_t sk_row = sbuf + (uint32_t)(ring * piece_smem) + row_off;            // and its staged skip row
                const int4 *cap = (const int4 *)(u.c_a + n0 + pc);
                const uint32_t t_piece = t_row + (uint32_t)pc;
                // the store issued two pieces ago must have finished reading this buffer
                if (pieces >= 2) {
                    if (elect_one()) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
                }
                if (SKIP8) {
                    if (!mbar_wait_warp(skip_bar0 + 8u * (uint32_t)ring, ring_parity, &sh->abort_flag, lane)) {
                        give_up(sh, u.status, 5);
                        ok = false;
                        break;
                    }
                    if (lane == 0) ++skip_taken;
                }
                // 16 columns at a time: the group's constants and skip bytes are requested, then the
                // accumulators are read (load and wait together), worked on and staged.  The usual piece
                // (four groups) is straight-line code.
                auto group = [&](int gcur) {
                    const int cc = gcur << 4;
                    const int co0 = n0 + pc + cc;
                    const uint32_t goff = (uint32_t)cc ^ row_swz16;                 // swizzled 16-byte chunk of the row (8-bit rows)
                    int4 ca[4];
#pragma unroll
                    for (int g = 0; g < 4; ++g) ca[g] = __ldg(cap + 4 * gcur + g);
                    uint4 sk = make_uint4(0, 0, 0, 0);
                    if (SKIP8) sk = lds128(sk_row + goff);
                    if (EPI == EPI_PROJ) tmem_ld16(t_piece + (uint32_t)(u.block_n + cc), accp);
                    tmem_ld16_sync(t_piece + (uint32_t)cc, acc, o_prev);
                    int V[16];
                    epilogue16<EPI>(acc, accp, V, ca, co0, m, row_ok, sk, es, a, u);
                    if (esz_rt == 4) {
#pragma unroll
                        for (int g = 0; g < 4; ++g)      // 4 columns = 16 bytes; 128-byte rows
                            sts128(ob_row + ((uint32_t)((cc << 2) + (g << 4)) ^ row_swz16), make_uint4((unsigned)V[4 * g], (unsigned)V[4 * g + 1], (unsigned)V[4 * g + 2], (unsigned)V[4 * g + 3]));
                    } else {
                        uint4 o;
                        if (EPI == EPI_FAST || EPI == EPI_FAST_SKIP8 || es.out_dtype == ICONV_U8) {
                            o.x = pack4_sat<false>(V[0], V[1], V[2], V[3]); o.y = pack4_sat<false>(V[4], V[5], V[6], V[7]);
                            o.z = pack4_sat<false>(V[8], V[9], V[10], V[11]); o.w = pack4_sat<false>(V[12], V[13], V[14], V[15]);
                        } else {
                            o.x = pack4_sat<true>(V[0], V[1], V[2], V[3]); o.y = pack4_sat<true>(V[4], V[5], V[6], V[7]);
                            o.z = pack4_sat<true>(V[8], V[9], V[10], V[11]); o.w = pack4_sat<true>(V[12], V[13], V[14], V[15]);
                        }
                        sts128(ob_row + goff, o);
                        o_prev = o;
                    }
                };
                const int ngroups = pcols >> 4;
                if (ngroups == 4) {
                    group(0); group(1); group(2); group(3);
                } else if (ngroups == 2) {
                    group(0); group(1);
                } else {
                    for (int gi = 0; gi < ngroups; ++gi) group(gi);
                }
                // hand the staged piece to the TMA unit (the store clips rows beyond the last
                // pixel and columns beyond c_out); the skip piece just consumed makes room for the
                // one SKIP_RING places on
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (elect_one()) {
                    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                 ::"l"(&tmap_out), "r"(ob), "r"(n0 + pc), "r"(m_tile * BLOCK_M + quad * 32)
                                 : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    if (SKIP8) request_skip_piece(ring);
                }
                if (SKIP8 && ++ring == skip_ring) { ring = 0; ring_parity ^= 1u; }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { if (PAIR) mbar_arrive_leader(smem_u32(&sh->tmem_empty[buf])); else mbar_arrive(smem_u32(&sh->tmem_empty[buf])); }
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
        if (warp < NUM_PRODUCERS && lane == 0) {
            if (b_issued) mbar_wait(smem_u32(&sh->b_full), 0, &never);
            // this warp's loads that can still be in flight: wait for the phase of the last one (it
            // may lack another producer's arrival, hence the bound), then for longer than any load
            // already handed to the TMA unit can take
            if (last_stage >= 0) mbar_wait(smem_u32(&sh->full[last_stage]), last_parity, &never);
            const long long t0 = clock64();
            while (clock64() - t0 < 2000000) {}
        }
        if (warp == MMA_WARP && lane == 0 && (!PAIR || rank == 0)) {
            if (PAIR) umma_commit_pair(smem_u32(&sh->drain)); else umma_commit(smem_u32(&sh->drain));
            mbar_wait(smem_u32(&sh->drain), 0, &never);
        }
        if (warp >= EPI_WARP0 && warp < EPI_WARP0 + u.epi_warps && lane == 0)
            for (int j = skip_taken; j < skip_issued; ++j)      // skip pieces requested and not yet waited for (at most the ring)
                mbar_wait(smem_u32(&sh->skip_full[warp - EPI_WARP0][j % u.skip_ring]), (uint32_t)((j / u.skip_ring) & 1), &never);
        __syncthreads();
    }
    // pairs: neither CTA may leave (or give back its TMEM) while the other can still reach its shared memory
    // or have MMAs in flight that write its TMEM
    if (PAIR) cluster_sync_all();
    if (warp == MMA_WARP) {
        tc_fence_after();
        if (PAIR) tmem_dealloc_pair(tmem_base, (uint32_t)u.tmem_cols);
        else tmem_dealloc(tmem_base, (uint32_t)u.tmem_cols);
    }
}

// Window-mode epilogue of one warp and tile: groups of 16 columns from TMEM (one register block,
// load and wait in one step: a second block with the next group in flight measured no faster),
// each through the layer's epilogue and out with one 16-byte store per pixel.  NG: the number of groups when known at compile time (0: `ngroups`).
// GU: per-channel parameters that are uniform per group (fetched group by group).
template <int EPI, int NG, bool GU>
__device__ __forceinline__ void window_groups(uint32_t t_row, const int4 *cap, uint8_t *ocol, const uint8_t *scol, bool valid, int col_lo,
                                              int ngroups, int *accA, const EpiScalars &es, const ConvArgs &a, const UmmaArgs &u)
{
    constexpr bool SKIP8 = (EPI == EPI_FAST_SKIP8 || EPI == EPI_SAFE_SKIP8);    // scol: this pixel's 8-bit skip row, read directly
    const int ng = NG ? NG : ngroups;
    const bool wide = (((uintptr_t)ocol) & 31u) == 0;      // this pixel's columns start on a 32-byte boundary
    uint4 o_even = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int gi = 0; gi < (NG ? NG : 16); gi += 2) {
        if (!NG && gi >= ng) break;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const int gcur = gi + hf;
            if (gcur >= ng) break;
            const int co0 = col_lo + (gcur << 4);
            int4 ca[4];
#pragma unroll
            for (int g = 0; g < 4; ++g) ca[g] = __ldg(cap + 4 * gcur + g);
            uint4 sk = make_uint4(0, 0, 0, 0);
            if (SKIP8 && valid && co0 < a.c_out) sk = __ldg((const uint4 *)(scol + (gcur << 4)));
            tmem_ld16_sync(t_row + (uint32_t)(gcur << 4), accA);
            int V[16];
            if (GU) epilogue16<EPI>(accA, accA, V, ca, co0, 0, false, sk, group_scalars(es, u, co0), a, u);
            else epilogue16<EPI>(accA, accA, V, ca, co0, 0, false, sk, es, a, u);
            uint4 o;
            if (EPI == EPI_FAST || EPI == EPI_FAST_SKIP8 || a.out_dtype == ICONV_U8) {
                o.x = pack4_sat<false>(V[0], V[1], V[2], V[3]); o.y = pack4_sat<false>(V[4], V[5], V[6], V[7]);
                o.z = pack4_sat<false>(V[8], V[9], V[10], V[11]); o.w = pack4_sat<false>(V[12], V[13], V[14], V[15]);
            } else {
                o.x = pack4_sat<true>(V[0], V[1], V[2], V[3]); o.y = pack4_sat<true>(V[4], V[5], V[6], V[7]);
                o.z = pack4_sat<true>(V[8], V[9], V[10], V[11]); o.w = pack4_sat<true>(V[12], V[13], V[14], V[15]);
            }
            // Two groups of a pixel are 32 contiguous bytes: one 32-byte store writes a whole sector where two
            // 16-byte stores wrote it in halves (with few MMAs per tile the epilogue's stores are the critical path:
            // every 16-byte-per-lane store is 32 half-written sectors to the load/store unit).
            if (hf == 0) {
                o_even = o;
                if ((!wide || gcur + 1 >= ng) && valid && co0 < a.c_out) *(uint4 *)(ocol + (gcur << 4)) = o;
            } else if (!wide) {
                if (valid && co0 < a.c_out) *(uint4 *)(ocol + (gcur << 4)) = o;
            } else if (valid && co0 < a.c_out) {
                st_global_32(ocol + ((gcur - 1) << 4), o_even, o);
            } else if (valid && co0 - 16 < a.c_out) {
                *(uint4 *)(ocol + ((gcur - 1) << 4)) = o_even;
            }
        }
    }
}

// ---------------------------------------------------------------- window mode
// Stride-1 filters wider than one tap re-read every input pixel kh * kw times in the im2col
// form, and what a CTA can pull through the TMA unit is about its share of the HBM rate.  Here a
// tile's whole input patch (its rows plus the halo, the full padded width or a 128 + kw - 1
// wide strip of it) arrives with ONE tiled load, zero-filled outside the image, as consecutive
// pixel rows of KC bytes.  Output pixels are numbered along "virtual rows" of win_vw pixels
// (the padded width, or the width rounded up to 128), 128 consecutive numbers per tile, so that
// for tap (r, s) the A operand is simply the 128 patch rows starting r * win_bw + s further on:
// a descriptor whose start address moves by whole rows (the swizzle is a function of the
// absolute shared-memory address, so any start row reads what TMA wrote).  Virtual pixels
// beyond the real width are computed and dropped.  The filter bank is resident, the epilogue
// stores straight from registers (a tile is not a contiguous run of real pixels).
// KH, KW, KJ: filter size and MMAs per tap when known at compile time (0: read from the
// arguments).  The issuing thread runs alone: every branch it takes costs it a resolution
// latency nothing hides, so the common filters get straight-line issue code.
template <int EPI, int KH, int KW, int KJ>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_window_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                   const __grid_constant__ ConvArgs a, const __grid_constant__ UmmaArgs u)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *b_res = tiles + (size_t)u.stages * u.stage_bytes;
    Shared *sh = (Shared *)(b_res + (size_t)u.b_tile_bytes * u.taps);
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);    // the same value in every lane, and known to the compiler as such: per-warp addresses and coordinates live in uniform registers
    const int lane = threadIdx.x & 31;
    const int num_tiles = u.m_tiles;

    if (threadIdx.x == 32) {
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_w);
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < u.stages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < u.nbuf; ++b) {
            mbar_init(smem_u32(&sh->tmem_full[b]), 1);
            mbar_init(smem_u32(&sh->tmem_empty[b]), (uint32_t)(4 * u.cs));
        }
        mbar_init(smem_u32(&sh->b_full), 1);
        mbar_init(smem_u32(&sh->drain), WIN_ISSUERS);          // one arrival per MMA issuer
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        grid_dep_launch();
    }
    if (warp == MMA_WARP) tmem_alloc(smem_u32(&sh->tmem_base), (uint32_t)u.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    int last_stage = -1, b_issued = 0;
    uint32_t last_parity = 0;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0 && (int)blockIdx.x < num_tiles) {
            const uint32_t bf = smem_u32(&sh->b_full);
            mbar_expect_tx(bf, (uint32_t)(u.block_n * u.kc * u.taps));
            for (int tap = 0; tap < u.taps; ++tap)
                tma_load_2d(smem_u32(b_res + (size_t)tap * u.b_tile_bytes), &tmap_w, bf, tap * u.kc, 0);
            b_issued = 1;
            grid_dep_wait();                        // the activations may come from the kernel before this one
            int stage = 0;
            uint32_t parity = 0;
            const uint32_t tx = (uint32_t)(u.kc * u.win_bw * u.win_bh);
            for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
                const int img = (int)fast_div((unsigned)tile, u.div_tpi_mul, u.div_tpi_shr);
                const unsigned rem = (unsigned)(tile - img * u.win_tpi);
                int cx, cy;                                   // first output pixel of the tile
                if (u.win_blocks) {
                    const int by = (int)fast_div(rem, u.div_vw_mul, u.div_vw_shr);
                    cx = ((int)rem - by * u.win_vw) * 8;
                    cy = by * 16;
                } else {
                    const unsigned i0 = rem * BLOCK_M;
                    cy = (int)fast_div(i0, u.div_vw_mul, u.div_vw_shr);
                    cx = u.win_full_width ? 0 : (int)i0 - cy * u.win_vw;
                }
                if (!mbar_wait(smem_u32(&sh->empty[stage]), parity ^ 1u, &sh->abort_flag)) {
                    give_up(sh, u.status, 1);
                    break;
                }
                const uint32_t full = smem_u32(&sh->full[stage]);
                mbar_expect_tx(full, tx);
                tma_load_tile_4d(smem_u32(tiles + (size_t)stage * u.stage_bytes), &tmap_x, full, 0,
                                 cx - a.pad, cy - a.pad, img);
                last_stage = stage;
                last_parity = parity;
                if (++stage == u.stages) { stage = 0; parity ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == MMA_WARP || warp == MMA_WARP2 || warp == MMA_WARP3) {
        // ---------------------------------------------------------------- MMA issuers
        // Three warps issue the tiles in turn.  Between two tiles an issuer spends several hundred
        // cycles on its barrier round (two commits, two waits), longer than the tensor pipe's
        // queue covers; one issuer's round hides behind the others' MMAs.
        // Tiles are independent (own accumulator buffer, own patch), so no order is needed
        // between the instruction streams, and each issuer's commits cover its own MMAs.
        // The whole warp walks the tiles and waits (warp-uniform control flow: addresses and descriptors
        // are then computed in uniform registers, which is where the MMA instruction takes them from);
        // one elected lane issues.  With the loop inside a single-lane branch every operand of every MMA
        // had to be moved over from a vector register, and the lone thread could not keep the pipe fed.
        // A stage's fills all go through the same issuer (the number of issuers divides the number of
        // stages): a parity wait tells a phase only from its neighbours, so the thread that waits for a
        // stage's next fill must be the one that consumed the fill before.
        const int which = warp == MMA_WARP ? 0 : warp == MMA_WARP2 ? 1 : 2;
        if (which < u.win_issuers && (int)blockIdx.x + which * (int)gridDim.x < num_tiles) {
            int t = which, stage = which % u.stages;
            uint32_t parity = (uint32_t)((which / u.stages) & 1);
            bool ok = mbar_wait_warp(smem_u32(&sh->b_full), 0, &sh->abort_flag, lane);
            if (!ok) give_up(sh, u.status, 6);
            const int kj = u.kc >> 5;
            const uint32_t desc_hi32 = (uint32_t)(u.desc_hi >> 32);
            const uint32_t a_hi32 = u.win_blocks ? u.desc_hi_a : desc_hi32;
            const uint32_t a_lo0 = ((smem_u32(tiles) & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t b_lo0 = ((smem_u32(b_res) & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t stage_step = (uint32_t)u.stage_bytes >> 4, row_step = (uint32_t)u.kc >> 4;
            const uint32_t b_step = (uint32_t)u.b_tile_bytes >> 4;
            const uint32_t line_step = (uint32_t)u.win_bw * row_step;
            const uint32_t tap_step = (uint32_t)u.win_tap_step * row_step;
            for (int tile = blockIdx.x + which * gridDim.x; tile < num_tiles && ok; tile += u.win_issuers * gridDim.x, t += u.win_issuers) {
                const int buf = t & (u.nbuf - 1);
                uint32_t off0 = 0;
                if (u.win_full_width) {
                    const int img = (int)fast_div((unsigned)tile, u.div_tpi_mul, u.div_tpi_shr);
                    const unsigned i0 = (unsigned)(tile - img * u.win_tpi) * BLOCK_M;
                    off0 = i0 - fast_div(i0, u.div_vw_mul, u.div_vw_shr) * (unsigned)u.win_vw;
                }
                if (!mbar_wait_warp(smem_u32(&sh->tmem_empty[buf]), (uint32_t)(((t >> u.lg_nbuf) & 1) ^ 1), &sh->abort_flag, lane)) {
                    give_up(sh, u.status, 2);
                    break;
                }
                tc_fence_after();
                if (!mbar_wait_warp(smem_u32(&sh->full[stage]), parity, &sh->abort_flag, lane)) {
                    give_up(sh, u.status, 3);
                    break;
                }
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * u.block_n);
                uint32_t a_line = a_lo0 + (uint32_t)stage * stage_step + off0 * row_step;
                uint32_t b_lo = b_lo0;
                if (!elect_one()) {
                } else if (KH) {
#pragma unroll
                    for (int r = 0; r < (KH ? KH : 1); ++r) {
#pragma unroll
                        for (int sx = 0; sx < (KW ? KW : 1); ++sx)
                            umma_slot2<KJ ? KJ : 1>(d_tmem, a_line + (uint32_t)sx * tap_step, a_hi32, b_lo + (uint32_t)(r * KW + sx) * b_step, desc_hi32,
                                                   u.idesc, (uint32_t)((r | sx) != 0));
                        a_line += line_step;
                    }
                } else {
                    uint32_t acc = 0;
                    for (int r = 0; r < a.kh; ++r) {
                        uint32_t a_lo = a_line;
                        for (int sx = 0; sx < a.kw; ++sx) {
                            if (kj == 4) umma_slot2<4>(d_tmem, a_lo, a_hi32, b_lo, desc_hi32, u.idesc, acc);
                            else if (kj == 2) umma_slot2<2>(d_tmem, a_lo, a_hi32, b_lo, desc_hi32, u.idesc, acc);
                            else umma_slot2<1>(d_tmem, a_lo, a_hi32, b_lo, desc_hi32, u.idesc, acc);
                            acc = 1;
                            a_lo += row_step;
                            b_lo += b_step;
                        }
                        a_line += line_step;
                    }
                }
                if (elect_one()) {
                    umma_commit(smem_u32(&sh->empty[stage]));
                    umma_commit(smem_u32(&sh->tmem_full[buf]));
                }
                stage += u.win_issuers;
                if (stage >= u.stages) { stage -= u.stages; parity ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp >= EPI_WARP0 && warp < EPI_WARP0 + u.epi_warps) {
        // ---------------------------------------------------------------- epilogue
        grid_dep_wait();                            // the skip operand may come from the kernel before this one
        const int ew = warp - EPI_WARP0;
        const int quad = warp & 3;
        const int slot = ew >> 2;
        const int part = slot % u.cs;
        const int turn = slot / u.cs;
        const int col_lo = part * u.part_n;
        const int ncols = min(u.block_n - col_lo, u.part_n);
        const int tile_step = u.bi * (int)gridDim.x;
        const EpiScalars es = epi_scalars(a, u);
        for (int t = turn, tile = blockIdx.x + turn * gridDim.x; tile < num_tiles; t += u.bi, tile += tile_step) {
            const int buf = t & (u.nbuf - 1);
            const int img = (int)fast_div((unsigned)tile, u.div_tpi_mul, u.div_tpi_shr);
            const unsigned rem = (unsigned)(tile - img * u.win_tpi);
            int y, xq;                                        // this lane's (virtual) output pixel
            if (u.win_blocks) {
                const int by = (int)fast_div(rem, u.div_vw_mul, u.div_vw_shr);
                const int mm = quad * 32 + lane;
                y = by * 16 + (mm >> 3);
                xq = ((int)rem - by * u.win_vw) * 8 + (mm & 7);
            } else {
                const unsigned i = rem * BLOCK_M + (unsigned)(quad * 32 + lane);
                y = (int)fast_div(i, u.div_vw_mul, u.div_vw_shr);
                xq = (int)i - y * u.win_vw;
            }
            const bool valid = xq < a.w_out && y < a.h_out;
            uint8_t *orow = (uint8_t *)a.out + (((long long)img * a.h_out + y) * a.w_out + xq) * a.out_c_total + a.out_c_offset;
            if (!mbar_wait_warp(smem_u32(&sh->tmem_full[buf]), (uint32_t)((t >> u.lg_nbuf) & 1), &sh->abort_flag, lane)) {
                give_up(sh, u.status, 4);
                break;
            }
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * u.block_n + col_lo);
            const int ngroups = ncols >> 4;
            int accA[16];
            if (EPI == EPI_NARROW) {
                tmem_ld16(t_row, accA);
                // a handful of channels per pixel (the regression networks' last layer): the general
                // 64-bit epilogue channel by channel, the skip read and the output written byte-wise
                const long long mpix = ((long long)img * a.h_out + y) * a.w_out + xq;
                for (int g0 = 0; g0 < ngroups; ++g0) {
                    if (g0) tmem_ld16(t_row + (uint32_t)(g0 << 4), accA);
                    tmem_ld_wait();
                    const int co0 = col_lo + (g0 << 4);
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const int co = co0 + k;
                        if (valid && co < a.c_out) {
                            const int pc = a.per_channel ? co : 0;
                            long long Y = (long long)accA[k] + __ldg(u.c_a + co);
                            if (a.skip_dtype >= 0)
                                Y += round_shift64((long long)load_skip(a.skip, mpix * a.skip_c_total + a.skip_c_offset + co, a.skip_dtype) * a.skip_mul,
                                                   a.skip_shift);
                            const int v = requant_tail(Y, a.brelu, __ldg(u.c_h + pc), __ldg(u.c_mul + pc), __ldg(u.c_shift + pc), a.out_zero,
                                                       a.out_lo, a.out_hi);
                            orow[co] = (uint8_t)v;
                        }
                    }
                }
            }
            if (EPI != EPI_NARROW) {
                const int4 *cap = (const int4 *)(u.c_a + col_lo);
                uint8_t *ocol = orow + col_lo;
                const uint8_t *scol = nullptr;
                if (EPI == EPI_FAST_SKIP8 || EPI == EPI_SAFE_SKIP8)
                    scol = (const uint8_t *)a.skip + (((long long)img * a.h_out + y) * a.w_out + xq) * a.skip_c_total + a.skip_c_offset + col_lo;
                // the usual widths get straight-line code: every offset an immediate, no loop control
                if (es.group_uniform) window_groups<EPI, 0, true>(t_row, cap, ocol, scol, valid, col_lo, ngroups, accA, es, a, u);
                else if (ngroups == 4) window_groups<EPI, 4, false>(t_row, cap, ocol, scol, valid, col_lo, ngroups, accA, es, a, u);
                else if (ngroups == 3) window_groups<EPI, 3, false>(t_row, cap, ocol, scol, valid, col_lo, ngroups, accA, es, a, u);
                else if (ngroups == 2) window_groups<EPI, 2, false>(t_row, cap, ocol, scol, valid, col_lo, ngroups, accA, es, a, u);
                else if (ngroups == 1) window_groups<EPI, 1, false>(t_row, cap, ocol, scol, valid, col_lo, ngroups, accA, es, a, u);
                else window_groups<EPI, 0, false>(t_row, cap, ocol, scol, valid, col_lo, ngroups, accA, es, a, u);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty[buf]));
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (sh->abort_flag) {
        volatile int never = 0;
        if (warp == 0 && lane == 0) {
            if (b_issued) mbar_wait(smem_u32(&sh->b_full), 0, &never);
            if (last_stage >= 0) mbar_wait(smem_u32(&sh->full[last_stage]), last_parity, &never);
            const long long t0 = clock64();
            while (clock64() - t0 < 2000000) {}
        }
        if ((warp == MMA_WARP || warp == MMA_WARP2 || warp == MMA_WARP3) && lane == 0) {
            umma_commit(smem_u32(&sh->drain));
            mbar_wait(smem_u32(&sh->drain), 0, &never);
        }
        __syncthreads();
    }
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)u.tmem_cols);
    }
}

}  // namespace iconv
