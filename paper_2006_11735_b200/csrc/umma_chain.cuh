// Two layers in one kernel: a block-closing 1x1 convolution with its 8-bit identity skip (Section
// 4.1) and the 1x1 convolution that opens the next block (Section 3.1: the output V_i of a layer
// is the input of the next).  The closing layer's 8-bit output tile is staged in shared memory for
// its TMA store anyway; staged as a K-major operand it is also the A operand of the next layer,
// whose filter bank (at most 64 KB) stays resident.  The wide tensor is then written once and
// never read back by the next layer, and one launch goes.
//
//   GEMM 1   128 pixels x 128 channels per tile (N tiles of 128, all N tiles of a pixel tile in
//            turn on the same CTA; the pixel tile's A operand is loaded once), int32 in TMEM,
//            two accumulator buffers.
//   epilogue 1  sixteen warps (lane quadrant x 32-column part): bias, rescaled skip, Eq. 4, u8
//            saturation in the clamp-free 32-bit form the plan proved, 16-byte swizzled stores into
//            the staging tile [4 parts][128 pixels][32 bytes], one TMA store per warp.
//   GEMM 2   the staged tile (four K = 32 chunks) x the next layer's weights for those 128 input
//            channels, accumulated over the N tiles of the pixel tile into a second accumulator
//            (c2 = 64 or 128 columns, two buffers).
//   epilogue 2  the same warps, c2 / 4 columns each: Eq. 4 in the clamp-free form, 16-byte stores.
//
// Integer sums in another order: both outputs are bit-identical to the two layers run apart.
// All waits are bounded as in the other kernels.
#pragma once

#include "umma_device.cuh"

namespace iconv {

constexpr int CHAIN_STAGES_MAX = 3;

struct ChainArgs {
    long long m_total;
    int m_tiles, n_tiles;           // pixel tiles; N tiles (of 128 channels) of the first layer
    int k1;                         // input channels of the first layer = its whole reduction (64 or 128)
    int c2;                         // output channels of the second layer (64 or 128)
    int stages;                     // A-operand stages (one per pixel tile in flight)
    int skip_ring;                  // staged skip pieces per warp (2 or 3)
    unsigned idesc1, idesc2;
    unsigned desc_hi1;              // upper descriptor word of the k1-byte rows (A1, W1)
    // first layer's epilogue (clamp-free form with an 8-bit skip)
    int q_mul, q_shift, q_half, skip_mul;
    unsigned skip_xor;
    const int32_t *c_a;             // [c1] (b << 8) + 2^7 - z * skip_mul
    // second layer's epilogue (clamp-free form)
    int q2_mul, q2_shift;
    const int32_t *c_a2;            // [c2] b * mul + 2^(shift-1)
    uint8_t *out2;                  // second layer's output tensor
    int out2_c_total, out2_c_offset;
    int *status;
};

struct ChainShared {
    unsigned long long skip_full[EPI_WARPS_MAX][SKIP_RING];
    unsigned long long a1_full[CHAIN_STAGES_MAX], a1_empty[CHAIN_STAGES_MAX];
    unsigned long long acc1_full[2];
    unsigned long long a2_full[2], a2_empty[2];
    unsigned long long d2_full[2], d2_empty[2];
    unsigned long long w_full, drain;
    uint32_t tmem_base;
    volatile int abort_flag;
};

__device__ __forceinline__ void chain_give_up(ChainShared *sh, int *status, int code)
{
    sh->abort_flag = 1;
    atomicCAS(status, 0, code);
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_chain_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w1,
                  const __grid_constant__ CUtensorMap tmap_w2, const __grid_constant__ CUtensorMap tmap_out,
                  const __grid_constant__ CUtensorMap tmap_skip, const __grid_constant__ ChainArgs c)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int a1_bytes = BLOCK_M * c.k1;                    // 8 or 16 KB
    const int w1_tile = 128 * c.k1;                         // one N tile of the first filter bank
    const int w2_tile = c.c2 * 128;                         // the second bank's rows for 128 input channels
    uint8_t *a1 = base;                                     // [stages][128][k1]
    uint8_t *w1 = a1 + (size_t)c.stages * a1_bytes;         // [n_tiles][128][k1]
    uint8_t *w2 = w1 + (size_t)c.n_tiles * w1_tile;         // [n_tiles][c2][128]
    uint8_t *a2 = w2 + (size_t)c.n_tiles * w2_tile;         // [2][4 parts][4 quadrants][32 pixels][32 bytes]
    uint8_t *skp = a2 + 2 * 16384;                          // [16 warps][ring][32 pixels][32 bytes]
    ChainShared *sh = (ChainShared *)(skp + (size_t)EPI_WARPS_MAX * c.skip_ring * 1024);

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);    // the same value in every lane, and known to the compiler as such: per-warp addresses and coordinates live in uniform registers
    const int lane = threadIdx.x & 31;
    const int n_super = (int)blockIdx.x < c.m_tiles ? (c.m_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int T = n_super * c.n_tiles;                      // tiles of this CTA

    if (threadIdx.x == 32) {
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_w1);
        prefetch_tensormap(&tmap_w2);
        prefetch_tensormap(&tmap_out);
        prefetch_tensormap(&tmap_skip);
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < CHAIN_STAGES_MAX; ++s) {
            mbar_init(smem_u32(&sh->a1_full[s]), 1);
            mbar_init(smem_u32(&sh->a1_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh->acc1_full[b]), 1);
            mbar_init(smem_u32(&sh->a2_full[b]), EPI_WARPS_MAX);
            mbar_init(smem_u32(&sh->a2_empty[b]), 1);
            mbar_init(smem_u32(&sh->d2_full[b]), 1);
            mbar_init(smem_u32(&sh->d2_empty[b]), EPI_WARPS_MAX);
        }
        for (int w = 0; w < EPI_WARPS_MAX * SKIP_RING; ++w) mbar_init(smem_u32(&sh->skip_full[0][0]) + 8u * (uint32_t)w, 1);
        mbar_init(smem_u32(&sh->w_full), 1);
        mbar_init(smem_u32(&sh->drain), 1);
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        grid_dep_launch();
    }
    if (warp == MMA_WARP) tmem_alloc(smem_u32(&sh->tmem_base), 512u);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    int w_issued = 0, a1_last = -1;
    int skip_issued = 0, skip_taken = 0;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0 && T > 0) {
            const uint32_t wf = smem_u32(&sh->w_full);
            mbar_expect_tx(wf, (uint32_t)(c.n_tiles * (w1_tile + w2_tile)));
            for (int nt = 0; nt < c.n_tiles; ++nt) {
                tma_load_2d(smem_u32(w1 + (size_t)nt * w1_tile), &tmap_w1, wf, 0, nt * 128);
                tma_load_2d(smem_u32(w2 + (size_t)nt * w2_tile), &tmap_w2, wf, nt * 128, 0);
            }
            w_issued = 1;
            grid_dep_wait();                        // the activations may come from the kernel before this one
            for (int s = 0; s < n_super; ++s) {
                const int st = s % c.stages;
                if (!mbar_wait(smem_u32(&sh->a1_empty[st]), (uint32_t)(((s / c.stages) & 1) ^ 1), &sh->abort_flag)) {
                    chain_give_up(sh, c.status, 1);
                    break;
                }
                const uint32_t full = smem_u32(&sh->a1_full[st]);
                mbar_expect_tx(full, (uint32_t)a1_bytes);
                tma_load_2d(smem_u32(a1 + (size_t)st * a1_bytes), &tmap_x, full, 0, ((int)blockIdx.x + s * (int)gridDim.x) * BLOCK_M);
                a1_last = s;
            }
        }
        __syncwarp();
    } else if (warp == MMA_WARP) {
        // ---------------------------------------------------------------- MMA issuer
        // (the whole warp walks the tiles and waits, so that addresses and descriptors are computed in uniform
        // registers, where the MMA instruction takes them from; one elected lane issues)
        if (T > 0) {
            bool ok = mbar_wait_warp(smem_u32(&sh->w_full), 0, &sh->abort_flag, lane);
            if (!ok) chain_give_up(sh, c.status, 6);
            const int kj1 = c.k1 >> 5;
            const uint32_t a1_lo0 = ((smem_u32(a1) & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t w1_lo0 = ((smem_u32(w1) & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t w2_lo0 = ((smem_u32(w2) & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t a2_lo0 = ((smem_u32(a2) & 0x3FFFFu) >> 4) | (1u << 16);
            // staged tile: rows of 32 bytes, 32-byte swizzle, 8-row groups 256 bytes apart; second bank: rows of
            // 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart
            const uint32_t a2_hi = (uint32_t)(((unsigned long long)(256 >> 4) << 32 | (1ull << 46) | (6ull << 61)) >> 32);
            const uint32_t w2_hi = (uint32_t)(((unsigned long long)(1024 >> 4) << 32 | (1ull << 46) | (2ull << 61)) >> 32);
            // GEMM 2 of tile tt: four K = 32 chunks of the staged tile against the second bank's rows for
            // the tile's 128 input channels, into the accumulator of the tile's pixel tile
            int ps = 0, pn = 0;                      // pixel tile and N tile of the tile before the current one
            auto second = [&](int tt, int ss, int nn) -> bool {
                if (!mbar_wait_warp(smem_u32(&sh->a2_full[tt & 1]), (uint32_t)((tt >> 1) & 1), &sh->abort_flag, lane)) { chain_give_up(sh, c.status, 3); return false; }
                if (nn == 0 && !mbar_wait_warp(smem_u32(&sh->d2_empty[ss & 1]), (uint32_t)(((ss >> 1) & 1) ^ 1), &sh->abort_flag, lane)) {
                    chain_give_up(sh, c.status, 2);
                    return false;
                }
                tc_fence_after();
                const uint32_t d2 = tmem_base + 256u + (uint32_t)((ss & 1) * 128);
                const uint32_t a_lo = a2_lo0 + (uint32_t)((tt & 1) * (16384 >> 4));
                const uint32_t b_lo = w2_lo0 + (uint32_t)(nn * (w2_tile >> 4));
                if (elect_one()) {
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch)
                        umma_i8_split2(d2, a_lo + (uint32_t)(ch * (4096 >> 4)), a2_hi, b_lo + 2u * (uint32_t)ch, w2_hi, c.idesc2, (uint32_t)(nn != 0 || ch != 0));
                    umma_commit(smem_u32(&sh->a2_empty[tt & 1]));
                    if (nn == c.n_tiles - 1) umma_commit(smem_u32(&sh->d2_full[ss & 1]));
                }
                return true;
            };
            int s = 0, nt = 0, st = 0;
            uint32_t a1_parity = 0;
            for (int t = 0; t < T && ok; ++t) {
                // (accumulator buffer t & 1 is free: the second GEMM of tile t - 2, issued in the round before this
                // one, waited until every epilogue warp had staged that tile, i.e. had read the buffer)
                if (nt == 0 && !mbar_wait_warp(smem_u32(&sh->a1_full[st]), a1_parity, &sh->abort_flag, lane)) {
                    chain_give_up(sh, c.status, 3);
                    break;
                }
                tc_fence_after();
                const uint32_t d1 = tmem_base + (uint32_t)((t & 1) * 128);
                const uint32_t a_lo = a1_lo0 + (uint32_t)(st * (a1_bytes >> 4)), b_lo = w1_lo0 + (uint32_t)(nt * (w1_tile >> 4));
                if (elect_one()) {
                    for (int j = 0; j < kj1; ++j) umma_i8_split(d1, a_lo + 2u * (uint32_t)j, b_lo + 2u * (uint32_t)j, c.desc_hi1, c.idesc1, (uint32_t)(j != 0));
                    umma_commit(smem_u32(&sh->acc1_full[t & 1]));
                    if (nt == c.n_tiles - 1) umma_commit(smem_u32(&sh->a1_empty[st]));
                }
                if (t > 0) ok = second(t - 1, ps, pn);
                ps = s; pn = nt;
                if (++nt == c.n_tiles) { nt = 0; ++s; if (++st == c.stages) { st = 0; a1_parity ^= 1u; } }
            }
            if (ok && T > 0) second(T - 1, ps, pn);
        }
        __syncwarp();
    } else if (warp >= EPI_WARP0) {
        // ---------------------------------------------------------------- epilogue
        grid_dep_wait();                            // the skip operand may come from the kernel before this one
        const int ew = warp - EPI_WARP0;
        const int quad = warp & 3, part = ew >> 2;  // TMEM lane quadrant (32 pixels); 32-column part of the tile
        const uint32_t skip_bar0 = smem_u32(&sh->skip_full[ew][0]);
        const uint32_t sbuf = smem_u32(skp + (size_t)ew * c.skip_ring * 1024);
        const unsigned row_off = (unsigned)lane * 32u;
        const unsigned row_swz16 = (((unsigned)lane >> 2) & 1u) << 4;
        const int q_mul = c.q_mul, q_shift = c.q_shift, skip_mul = c.skip_mul;
        const unsigned skip_xor = c.skip_xor;
        int q_half;                                 // pinned in a vector register (see epi_scalars)
        asm volatile("mov.b32 %0, %1;" : "=r"(q_half) : "r"(c.q_half));
        const int c2w = c.c2 >> 2;                  // second layer's columns per warp: 16 or 32
        bool ok = true;

        // skip pieces (32 pixels x 32 bytes) through a ring, requested `ring - 1` tiles ahead
        // (no divisions in the per-tile paths: pixel-tile and N-tile counters advance by themselves)
        int pf = 0, pf_nt = 0, pf_m = (int)blockIdx.x * BLOCK_M + quad * 32;      // next tile to request: index, N tile, first pixel row
        const int m_step = (int)gridDim.x * BLOCK_M, col0 = part * 32;
        auto request_skip = [&](int ring_slot) {
            if (pf >= T) return;
            const uint32_t bar = skip_bar0 + 8u * (uint32_t)ring_slot;
            mbar_expect_tx(bar, 1024u);
            tma_load_2d(sbuf + (uint32_t)(ring_slot * 1024), &tmap_skip, bar, pf_nt * 128 + col0, pf_m);
            ++skip_issued;
            ++pf;
            if (++pf_nt == c.n_tiles) { pf_nt = 0; pf_m += m_step; }
        };
        if (lane == 0)
            for (int r = 0; r < c.skip_ring; ++r) request_skip(r);
        int ring = 0;
        uint32_t ring_parity = 0;

        // second epilogue of pixel tile ss: this warp's c2 / 4 columns
        auto second = [&](int ss) -> bool {
            if (!mbar_wait_warp(smem_u32(&sh->d2_full[ss & 1]), (uint32_t)((ss >> 1) & 1), &sh->abort_flag, lane)) { chain_give_up(sh, c.status, 4); return false; }
            tc_fence_after();
            const long long m = (long long)((int)blockIdx.x + ss * (int)gridDim.x) * BLOCK_M + quad * 32 + lane;
            uint8_t *orow = c.out2 + m * c.out2_c_total + c.out2_c_offset + part * c2w;
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + 256u + (uint32_t)((ss & 1) * 128 + part * c2w);
            for (int g = 0; g < (c2w >> 4); ++g) {
                const int4 *cap = (const int4 *)(c.c_a2 + part * c2w + (g << 4));
                int4 ca[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) ca[k] = __ldg(cap + k);
                int acc[16];
                tmem_ld16_sync(t_row + (uint32_t)(g << 4), acc);
                const int cav[16] = {ca[0].x, ca[0].y, ca[0].z, ca[0].w, ca[1].x, ca[1].y, ca[1].z, ca[1].w,
                                     ca[2].x, ca[2].y, ca[2].z, ca[2].w, ca[3].x, ca[3].y, ca[3].z, ca[3].w};
                int V[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) V[k] = (acc[k] * c.q2_mul + cav[k]) >> c.q2_shift;
                uint4 o;
                o.x = pack4_sat<false>(V[0], V[1], V[2], V[3]); o.y = pack4_sat<false>(V[4], V[5], V[6], V[7]);
                o.z = pack4_sat<false>(V[8], V[9], V[10], V[11]); o.w = pack4_sat<false>(V[12], V[13], V[14], V[15]);
                if (m < c.m_total) *(uint4 *)(orow + (g << 4)) = o;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->d2_empty[ss & 1]));
            return true;
        };

        int s = 0, nt = 0, m0 = (int)blockIdx.x * BLOCK_M + quad * 32;
        const uint32_t acc1_full0 = smem_u32(&sh->acc1_full[0]), a2_full0 = smem_u32(&sh->a2_full[0]), a2_empty0 = smem_u32(&sh->a2_empty[0]);
        const uint32_t a2_base = smem_u32(a2) + (uint32_t)(part * 4096 + quad * 1024);
        const uint32_t t_base = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(part * 32);
        for (int t = 0; t < T && ok; ++t) {
            const uint32_t par = (uint32_t)(t & 1), par8 = par << 3, phase = (uint32_t)((t >> 1) & 1);
            if (!mbar_wait_warp(acc1_full0 + par8, phase, &sh->abort_flag, lane)) {
                chain_give_up(sh, c.status, 4);
                break;
            }
            tc_fence_after();
            // the staging buffer: GEMM 2 of the tile two back has read it, and so has this warp's own store
            if (!mbar_wait_warp(a2_empty0 + par8, phase ^ 1u, &sh->abort_flag, lane)) {
                chain_give_up(sh, c.status, 4);
                break;
            }
            if (t >= 2) {
                if (elect_one()) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                __syncwarp();
            }
            if (!mbar_wait_warp(skip_bar0 + 8u * (uint32_t)ring, ring_parity, &sh->abort_flag, lane)) {
                chain_give_up(sh, c.status, 5);
                break;
            }
            if (lane == 0) ++skip_taken;
            const uint32_t ob = a2_base + par * 16384u;
            const uint32_t ob_row = ob + row_off, sk_row = sbuf + (uint32_t)(ring * 1024) + row_off;
            const uint32_t t_row = t_base + par * 128u;
            const int n0 = nt * 128 + col0;
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                const uint32_t goff = (uint32_t)(g << 4) ^ row_swz16;
                const int4 *cap = (const int4 *)(c.c_a + n0 + (g << 4));
                int4 ca[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) ca[k] = __ldg(cap + k);
                const uint4 sk = lds128(sk_row + goff);
                int acc[16], V[16];
                tmem_ld16_sync(t_row + (uint32_t)(g << 4), acc);
                // Y = U + ((s * skip_mul + C) >> 8), C = (b << 8) + 2^7 - z * skip_mul; V = (Y * mul + half) >> shift
                const int cav[16] = {ca[0].x, ca[0].y, ca[0].z, ca[0].w, ca[1].x, ca[1].y, ca[1].z, ca[1].w,
                                     ca[2].x, ca[2].y, ca[2].z, ca[2].w, ca[3].x, ca[3].y, ca[3].z, ca[3].w};
                const unsigned w4[4] = {sk.x ^ skip_xor, sk.y ^ skip_xor, sk.z ^ skip_xor, sk.w ^ skip_xor};
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    const int sv = (int)__byte_perm(w4[k >> 2], 0, 0x4440 + (k & 3));
                    const int y = acc[k] + ((sv * skip_mul + cav[k]) >> FAST_SKIP_SHIFT);
                    V[k] = (y * q_mul + q_half) >> q_shift;
                }
                uint4 o;
                o.x = pack4_sat<false>(V[0], V[1], V[2], V[3]); o.y = pack4_sat<false>(V[4], V[5], V[6], V[7]);
                o.z = pack4_sat<false>(V[8], V[9], V[10], V[11]); o.w = pack4_sat<false>(V[12], V[13], V[14], V[15]);
                sts128(ob_row + goff, o);
            }
            // the accumulator buffer is free; the staged piece goes to the TMA unit and counts towards GEMM 2
            tc_fence_before();
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (elect_one()) {
                mbar_arrive(a2_full0 + par8);      // also tells the issuer that this warp has read the accumulator buffer
                asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                             ::"l"(&tmap_out), "r"(ob), "r"(n0), "r"(m0)
                             : "memory");
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                request_skip(ring);
            }
            if (++ring == c.skip_ring) { ring = 0; ring_parity ^= 1u; }
            // the second layer's outputs of the pixel tile before this one: its last GEMM 2 was issued
            // behind this tile's GEMM 1
            if (nt == 0 && s > 0) ok = second(s - 1);
            if (++nt == c.n_tiles) { nt = 0; ++s; m0 += m_step; }
        }
        if (ok && n_super > 0) second(n_super - 1);
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        __syncwarp();
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (sh->abort_flag) {
        volatile int never = 0;
        if (warp == 0 && lane == 0) {
            if (w_issued) mbar_wait(smem_u32(&sh->w_full), 0, &never);
            if (a1_last >= 0) mbar_wait(smem_u32(&sh->a1_full[a1_last % c.stages]), (uint32_t)((a1_last / c.stages) & 1), &never);
            const long long t0 = clock64();
            while (clock64() - t0 < 2000000) {}
        }
        if (warp == MMA_WARP && lane == 0) {
            umma_commit(smem_u32(&sh->drain));
            mbar_wait(smem_u32(&sh->drain), 0, &never);
        }
        if (warp >= EPI_WARP0 && lane == 0)
            for (int j = skip_taken; j < skip_issued; ++j)
                mbar_wait(smem_u32(&sh->skip_full[warp - EPI_WARP0][j % c.skip_ring]), (uint32_t)((j / c.skip_ring) & 1), &never);
        __syncthreads();
    }
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512u);
    }
}

}  // namespace iconv
