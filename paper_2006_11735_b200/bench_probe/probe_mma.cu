// Issue-rate probe of tcgen05.mma kind::i8: what the tensor pipe of this GPU sustains when
// nothing but the instruction stream limits it (operands resident in shared memory, one
// issuing thread per SM, every instruction accumulating into the same TMEM tile).  A
// measurement aid of the benchmark, built into a library of its own (libiconv_probe.so): the
// convolution kernel's achieved TOP/s is reported against this figure as well as against the
// nominal one.  Not part of the layer's C ABI.
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <vector>

namespace iconv_probe {

namespace {

__device__ __forceinline__ uint32_t probe_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

struct ProbeResult {
    long long cycles;
    int timed_out;
    int pad;
};

__global__ void __launch_bounds__(128, 1) mma_rate_kernel(int n, int row_bytes, int a_group_stride, int iters, ProbeResult *res)
{
    extern __shared__ uint8_t probe_raw[];
    uint8_t *tiles = (uint8_t *)(((uintptr_t)probe_raw + 1023) & ~(uintptr_t)1023);   // A: 16 KB, B: 32 KB
    __shared__ unsigned long long bar;
    __shared__ uint32_t tmem_base;
    for (int i = threadIdx.x; i < (16384 + 32768) / 4; i += blockDim.x) ((uint32_t *)tiles)[i] = 0x01010101u;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(probe_smem_u32(&bar)), "r"(1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(probe_smem_u32(&tmem_base)), "r"(256) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tb = tmem_base;
    if (threadIdx.x == 0) {
        // K-major tiles with rows of row_bytes (128, 64 or 32) and the swizzle of that width, as the
        // convolution kernels stage them; A's 8-row groups a_group_stride bytes apart (8 * row_bytes for
        // a dense tile, a patch line in the window kernel's block tiling)
        const unsigned long long layout = row_bytes == 128 ? 2ull : (row_bytes == 64 ? 4ull : 6ull);
        const unsigned long long hi_a = ((unsigned long long)(a_group_stride >> 4) << 32) | (1ull << 46) | (layout << 61);
        const unsigned long long hi_b = ((unsigned long long)((8 * row_bytes) >> 4) << 32) | (1ull << 46) | (layout << 61);
        const unsigned long long da = hi_a | (unsigned long long)((probe_smem_u32(tiles) & 0x3FFFFu) >> 4) | (1ull << 16);
        const unsigned long long db = hi_b | (unsigned long long)((probe_smem_u32(tiles + 16384) & 0x3FFFFu) >> 4) | (1ull << 16);
        const uint32_t idesc = (2u << 4) | (1u << 10) | ((unsigned)(n >> 3) << 17) | ((128u >> 4) << 24);   // u8 x s8 -> s32
        const unsigned slices = (unsigned)(row_bytes >> 5);
        // four instructions per loop round, their K-slice offsets fixed before the loop: whatever the issuing
        // thread executes between two instructions shows in the rate once the pipe's queue runs empty
        unsigned long long koff[4];
        for (int j = 0; j < 4; ++j) koff[j] = 2ull * ((unsigned)j & (slices - 1));    // walk the 32-byte K slices of a row
        const long long t0 = clock64();
        for (int i = 0; i < iters; i += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                asm volatile(
                    "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                    "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                    ::"r"(tb), "l"(da + koff[j]), "l"(db + koff[j]), "r"(idesc), "r"(i + j) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(probe_smem_u32(&bar)) : "memory");
        int timed_out = 1;
        for (long long spin = 0; spin < 200000000ll; ++spin) {     // bounded wait for the last MMA
            uint32_t ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(probe_smem_u32(&bar)), "r"(0) : "memory");
            if (ok) { timed_out = 0; break; }
        }
        res[blockIdx.x].cycles = clock64() - t0;
        res[blockIdx.x].timed_out = timed_out;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tb), "r"(256) : "memory");
    }
}

}  // namespace

}  // namespace iconv_probe

using namespace iconv_probe;

// How fast this GPU's tensor pipe retires tcgen05.mma kind::i8 (M = 128, N = block_n, K = 32,
// u8 x s8 -> s32) when only the instruction stream limits it: one thread per SM issues `iters`
// dependent instructions on operands in shared memory.  Writes whole-GPU TOP/s (2 * MACs / event
// time of the launch) and the slowest SM's cycles per instruction to the HOST pointers.
// `iters` is a multiple of 4 (the issue loop is unrolled four times).
// Synchronous; allocates a few KB on the current device.  Returns 0, -1 (bad argument),
// -6 (a CUDA call failed) or -7 (the bounded wait for the last instruction ran out).
//
// probe_mma_rate_rows: the same with operand rows of row_bytes (32, 64 or 128: the swizzle width) and
// A's 8-row groups a_group_stride bytes apart (a multiple of 16, at least 8 * row_bytes, the 16 groups
// within 16 KB), the forms the convolution kernels use for narrow layers and for block tiling.
static int probe_run(int32_t block_n, int32_t row_bytes, int32_t a_group_stride, int32_t iters, double *tops, double *cycles_per_mma);

extern "C" __attribute__((visibility("default"))) int probe_mma_rate(int32_t block_n, int32_t iters, double *tops, double *cycles_per_mma)
{
    return probe_run(block_n, 128, 1024, iters, tops, cycles_per_mma);
}

extern "C" __attribute__((visibility("default"))) int probe_mma_rate_rows(int32_t block_n, int32_t row_bytes, int32_t a_group_stride, int32_t iters,
                                                                          double *tops, double *cycles_per_mma)
{
    if ((row_bytes != 32 && row_bytes != 64 && row_bytes != 128) || a_group_stride % 16 || a_group_stride < 8 * row_bytes ||
        15 * a_group_stride + 8 * row_bytes > 16384)
        return -1;
    return probe_run(block_n, row_bytes, a_group_stride, iters, tops, cycles_per_mma);
}

static int probe_run(int32_t block_n, int32_t row_bytes, int32_t a_group_stride, int32_t iters, double *tops, double *cycles_per_mma)
{
    if (!tops || !cycles_per_mma || iters < 4 || iters % 4 || iters > (1 << 22) || block_n < 16 || block_n > 256 || block_n % 16) return -1;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -6;
    const size_t smem = 16384 + 32768 + 1024;
    if (cudaFuncSetAttribute(mma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return -6;
    ProbeResult *d_res = nullptr;
    if (cudaMalloc((void **)&d_res, sizeof(ProbeResult) * sms) != cudaSuccess) return -6;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    float ms = 0.f;
    cudaError_t err = cudaEventCreate(&e0);
    if (err == cudaSuccess) err = cudaEventCreate(&e1);
    for (int rep = 0; rep < 2 && err == cudaSuccess; ++rep) {      // the first launch warms up
        if (err == cudaSuccess) err = cudaEventRecord(e0, 0);
        mma_rate_kernel<<<sms, 128, smem, 0>>>(block_n, row_bytes, a_group_stride, iters, d_res);
        if (err == cudaSuccess) err = cudaGetLastError();
        if (err == cudaSuccess) err = cudaEventRecord(e1, 0);
        if (err == cudaSuccess) err = cudaEventSynchronize(e1);
    }
    if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, e0, e1);
    std::vector<ProbeResult> h((size_t)sms);
    if (err == cudaSuccess) err = cudaMemcpy(h.data(), d_res, sizeof(ProbeResult) * sms, cudaMemcpyDeviceToHost);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(d_res);
    if (err != cudaSuccess) return -6;
    long long worst = 0;
    for (const ProbeResult &r : h) {
        if (r.timed_out) return -7;
        worst = std::max(worst, r.cycles);
    }
    *cycles_per_mma = (double)worst / iters;
    *tops = 2.0 * (double)sms * iters * 128.0 * block_n * 32.0 / (ms * 1e-3) / 1e12;
    return 0;
}
