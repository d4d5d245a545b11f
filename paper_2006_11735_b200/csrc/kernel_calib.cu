// The n-sigma bound of Section 3.2.2 on the GPU: the smallest value among the largest
// `fraction` of an int32 feature map Y, i.e. its k-th largest element with
// k = max(1, ceil(count * fraction)), clamped to at least 1 (a BReLU bound is positive).
// It is the step right before the hot path: the bound h_ri it returns feeds Eq. 9-13
// (`iq_brelu_params`), which give the layer's mul, shift and h_i.
//
// Exact selection without sorting: a most-significant-digit radix select over the
// order-preserving key y ^ 0x80000000.  Four passes, one per byte from the top; a pass
// histograms the next byte of every key that still matches the prefix found so far (a
// 256-bin histogram per block in shared memory, merged with one atomic per non-empty bin),
// and a one-thread step walks the bins from the top until it has passed k elements, appending
// that bin to the prefix.  The prefix, the remaining k and the histograms stay on the
// device, so the four passes run back to back on the stream; each pass reads Y once
// (count * 4 bytes, HBM-bound for tensors beyond L2).
#include "plan.h"

namespace iconv {

namespace {

struct SelectState {
    unsigned long long hist[256];
    unsigned long long k;          // rank (from the top, 1-based) still to find inside the prefix
    unsigned prefix, mask;         // key bits fixed so far
    int result;
    int pad;
};

constexpr int CALIB_THREADS = 512;

__global__ void select_init_kernel(SelectState *st, unsigned long long k)
{
    const int t = threadIdx.x;
    if (t < 256) st->hist[t] = 0;
    if (t == 0) { st->k = k; st->prefix = 0; st->mask = 0; st->result = 0; }
}

// Counts one key into the block's histogram if it lies under the prefix.  A feature map's keys
// crowd into a few bins of the upper bytes, so a thread keeps the count of its current bin
// in a register and touches shared memory only when the bin changes.
__device__ __forceinline__ void tally(unsigned key, unsigned prefix, unsigned mask, int shift, unsigned *sh, unsigned &cur, unsigned &cnt)
{
    if ((key & mask) != prefix) return;
    const unsigned bin = (key >> shift) & 255u;
    if (bin == cur) { ++cnt; return; }
    if (cnt) atomicAdd(&sh[cur], cnt);
    cur = bin;
    cnt = 1;
}

// One pass: the byte at `shift` of every key under the current prefix.
__global__ void __launch_bounds__(CALIB_THREADS) select_hist_kernel(const int32_t *__restrict__ y, long long count, int shift, SelectState *st)
{
    __shared__ unsigned sh[256];
    if (threadIdx.x < 256) sh[threadIdx.x] = 0;
    __syncthreads();
    const unsigned prefix = st->prefix, mask = st->mask;
    unsigned cur = 0, cnt = 0;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long step = (long long)gridDim.x * blockDim.x;
    // 16-byte loads over the aligned middle, scalar loads at the ragged ends
    const long long head = min(count, (long long)((16 - ((uintptr_t)y & 15)) & 15) / 4);
    const long long vecs = (count - head) / 4;
    const int4 *yv = (const int4 *)(y + head);
    for (long long i = tid; i < vecs; i += step) {
        const int4 v = __ldg(yv + i);
        tally((unsigned)v.x ^ 0x80000000u, prefix, mask, shift, sh, cur, cnt);
        tally((unsigned)v.y ^ 0x80000000u, prefix, mask, shift, sh, cur, cnt);
        tally((unsigned)v.z ^ 0x80000000u, prefix, mask, shift, sh, cur, cnt);
        tally((unsigned)v.w ^ 0x80000000u, prefix, mask, shift, sh, cur, cnt);
    }
    for (long long e = tid; e < head; e += step) tally((unsigned)y[e] ^ 0x80000000u, prefix, mask, shift, sh, cur, cnt);
    for (long long e = head + vecs * 4 + tid; e < count; e += step) tally((unsigned)y[e] ^ 0x80000000u, prefix, mask, shift, sh, cur, cnt);
    if (cnt) atomicAdd(&sh[cur], cnt);
    __syncthreads();
    if (threadIdx.x < 256 && sh[threadIdx.x]) atomicAdd(&st->hist[threadIdx.x], (unsigned long long)sh[threadIdx.x]);
}

// Picks the bin that holds the k-th largest key, fixes it in the prefix, clears the histogram.
__global__ void select_step_kernel(SelectState *st, int shift, int last)
{
    if (threadIdx.x == 0) {
        unsigned long long k = st->k, above = 0;
        int b = 255;
        for (; b > 0; --b) {
            if (above + st->hist[b] >= k) break;
            above += st->hist[b];
        }
        st->k = k - above;
        st->prefix |= (unsigned)b << shift;
        st->mask |= 255u << shift;
        if (last) {
            const int v = (int)(st->prefix ^ 0x80000000u);
            st->result = v < 1 ? 1 : v;
        }
    }
    __syncthreads();
    if (threadIdx.x < 256) st->hist[threadIdx.x] = 0;
}

SelectState *g_state[16] = {nullptr};

int state_for_device(SelectState **out)
{
    int dev = 0;
    ICONV_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 16) { set_error("iq_sigma_bound: device index beyond 15"); return ICONV_ERR_ARG; }
    if (!g_state[dev]) ICONV_CUDA_TRY(cudaMalloc((void **)&g_state[dev], sizeof(SelectState)));
    *out = g_state[dev];
    return ICONV_OK;
}

}  // namespace

}  // namespace iconv

using namespace iconv;

extern "C" int iq_sigma_bound(const int32_t *y, int64_t count, double fraction, int32_t *bound, void *cuda_stream)
{
    if (!bound || count < 0 || !(fraction > 0.0) || fraction > 1.0 || (count > 0 && !y)) {
        set_error("iq_sigma_bound: needs a device tensor, 0 < fraction <= 1 and a place for the result");
        return ICONV_ERR_ARG;
    }
    if ((uintptr_t)y % 4) { set_error("iq_sigma_bound: the tensor must be 4-byte aligned"); return ICONV_ERR_ALIGN; }
    if (count == 0) { *bound = 1; return ICONV_OK; }       // an empty map bounds nothing: the smallest legal bound
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    SelectState *st = nullptr;
    int rc = state_for_device(&st);
    if (rc != ICONV_OK) return rc;
    double kd = ceil((double)count * fraction);
    unsigned long long k = kd < 1.0 ? 1ull : (unsigned long long)kd;
    if (k > (unsigned long long)count) k = (unsigned long long)count;
    long long blocks = (count / 4 + CALIB_THREADS - 1) / CALIB_THREADS;
    if (blocks < 1) blocks = 1;
    if (blocks > 148ll * 4) blocks = 148ll * 4;
    select_init_kernel<<<1, 256, 0, stream>>>(st, k);
    for (int pass = 3; pass >= 0; --pass) {
        select_hist_kernel<<<(unsigned)blocks, CALIB_THREADS, 0, stream>>>(y, (long long)count, 8 * pass, st);
        select_step_kernel<<<1, 256, 0, stream>>>(st, 8 * pass, pass == 0);
    }
    ICONV_CUDA_TRY(cudaGetLastError());
    int result = 0;
    ICONV_CUDA_TRY(cudaMemcpyAsync(&result, &st->result, sizeof(int), cudaMemcpyDeviceToHost, stream));
    ICONV_CUDA_TRY(cudaStreamSynchronize(stream));
    *bound = result;
    return ICONV_OK;
}
