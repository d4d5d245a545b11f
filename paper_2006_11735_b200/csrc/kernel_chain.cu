// Host side of the two-layer kernel (umma_chain.cuh): which pairs of layers it takes, its plan
// (two ordinary layer plans hold the packed weights and the epilogue constants; the pair adds
// tensor maps over them with its own tile shapes), the launch.
#include <cuda.h>

#include <atomic>
#include <cstring>
#include <new>

#include "umma_chain.cuh"
#include "umma_inst.h"

struct iconv_chain_s {
    iconv_plan_t *p1 = nullptr, *p2 = nullptr;
    CUtensorMap tmap_w1, tmap_w2;
    int k1 = 0, c1 = 0, c2 = 0, n_tiles = 0, stages = 0, skip_ring = 0;
    size_t smem = 0;
};

namespace iconv {

namespace {

const char *chain_refusal(const iconv_desc &a, const iconv_desc &b)
{
    if (a.kh != 1 || a.kw != 1 || a.stride != 1 || a.pad != 0 || b.kh != 1 || b.kw != 1 || b.stride != 1 || b.pad != 0) return "both layers must be 1x1, stride 1, unpadded";
    if (a.n != b.n || a.h != b.h || a.w != b.w) return "the layers' pixel grids differ";
    if (a.c_in != 64 && a.c_in != 128) return "the first layer's reduction must be 64 or 128 channels";
    if (a.in_dtype != ICONV_U8 || b.in_dtype != ICONV_U8 || a.out_dtype != ICONV_U8 || b.out_dtype != ICONV_U8) return "8-bit unsigned activations only";
    if (a.c_out % 128 || a.c_out > 512) return "the first layer's output channels must be 128, 256, 384 or 512";
    if (b.c_in != a.c_out || b.in_c_total != a.out_c_total || b.in_c_offset != a.out_c_offset) return "the second layer must read exactly the first layer's output slice";
    if (b.c_out != 64 && b.c_out != 128) return "the second layer's output channels must be 64 or 128";
    if (a.proj_weights || b.proj_weights || b.skip_dtype >= 0) return "no fused projection, no skip on the second layer";
    if (a.skip_dtype != ICONV_U8 && a.skip_dtype != ICONV_S8 && a.skip_dtype != ICONV_U8_RAW128) return "the first layer needs an 8-bit skip";
    if (a.per_channel || b.per_channel) return "per-layer mul / shift / h_i only";
    if (a.in_c_total % 16 || a.in_c_offset % 16 || a.out_c_total % 16 || a.out_c_offset % 16 || a.skip_c_total % 16 || a.skip_c_offset % 16 ||
        b.out_c_total % 16 || b.out_c_offset % 16)
        return "channel strides and offsets must be multiples of 16";
    return nullptr;
}

}  // namespace

}  // namespace iconv

using namespace iconv;

extern "C" int iconv_chain_destroy(iconv_chain_t *c)
{
    if (!c) return ICONV_OK;
    iconv_plan_destroy(c->p1);
    iconv_plan_destroy(c->p2);
    delete c;
    return ICONV_OK;
}

extern "C" int iconv_plan_chain(const iconv_desc *first, const iconv_desc *second, iconv_chain_t **chain_out)
{
    if (!first || !second || !chain_out) { set_error("iconv_plan_chain: null argument"); return ICONV_ERR_ARG; }
    *chain_out = nullptr;
    if (const char *why = chain_refusal(*first, *second)) { set_error("iconv_plan_chain: %s", why); return ICONV_ERR_UNSUPPORTED; }
    iconv_chain_t *c = new (std::nothrow) iconv_chain_s();
    if (!c) { set_error("iconv_plan_chain: out of host memory"); return ICONV_ERR_ARG; }
    iconv_desc d1 = *first, d2 = *second;
    d1.kernel = ICONV_KERNEL_UMMA_IM2COL;
    d2.kernel = ICONV_KERNEL_UMMA_IM2COL;
    int rc = iconv_plan(&d1, &c->p1);               // validates, packs the weights, proves and fills the epilogue constants
    if (rc == ICONV_OK) rc = iconv_plan(&d2, &c->p2);
    if (rc == ICONV_OK && (c->p1->epi != EPI_FAST_SKIP8 || c->p2->epi != EPI_FAST)) {
        set_error("iconv_plan_chain: the clamp-free 32-bit epilogue forms are not provable for these layers (variants %d, %d)", c->p1->epi, c->p2->epi);
        rc = ICONV_ERR_UNSUPPORTED;
    }
    if (rc == ICONV_OK && (c->p1->c_in_pad != first->c_in || c->p1->kc != first->c_in || c->p2->c_in_pad != second->c_in || c->p2->c_out_pad != second->c_out ||
                           c->p1->c_out_pad != first->c_out)) {
        set_error("iconv_plan_chain: unexpected packing of the layers' weights");
        rc = ICONV_ERR_UNSUPPORTED;
    }
    if (rc == ICONV_OK) {
        c->k1 = first->c_in; c->c1 = first->c_out; c->c2 = second->c_out; c->n_tiles = first->c_out / 128;
        // shared memory: A stages, both filter banks, the staging tile (two buffers), the skip ring
        const size_t fixed = 1024 + sizeof(ChainShared) + (size_t)c->n_tiles * (128 * c->k1 + c->c2 * 128) + 2 * 16384;
        c->stages = 0;
        for (int ring = SKIP_RING; ring >= 2 && !c->stages; --ring)
            for (int st = CHAIN_STAGES_MAX; st >= 2 && !c->stages; --st) {
                const size_t need = fixed + (size_t)EPI_WARPS_MAX * ring * 1024 + (size_t)st * BLOCK_M * c->k1;
                if (need <= (size_t)MAX_SMEM) { c->stages = st; c->skip_ring = ring; c->smem = need; }
            }
        if (!c->stages) { set_error("iconv_plan_chain: the two filter banks do not fit shared memory"); rc = ICONV_ERR_UNSUPPORTED; }
    }
    if (rc == ICONV_OK) rc = umma_encode_2d(&c->tmap_w1, c->p1->w_packed, c->k1, c->c1, c->k1, c->k1, 128, c->k1);
    if (rc == ICONV_OK) rc = umma_encode_2d(&c->tmap_w2, c->p2->w_packed, c->c1, c->c2, c->c1, 128, c->c2, 128);
    if (rc == ICONV_OK) rc = umma_chain_opt_in();
    if (rc != ICONV_OK) { iconv_chain_destroy(c); return rc; }
    *chain_out = c;
    return ICONV_OK;
}

extern "C" int iconv_forward_chain(const iconv_chain_t *c, const void *x, const void *skip, void *out, void *out2, void *cuda_stream)
{
    if (!c) { set_error("iconv_forward_chain: null plan"); return ICONV_ERR_ARG; }
    const iconv_desc &d1 = c->p1->d, &d2 = c->p2->d;
    if (d1.n == 0) return ICONV_OK;
    if (!x || !skip || !out || !out2) { set_error("iconv_forward_chain: null tensor pointer"); return ICONV_ERR_ARG; }
    if (((uintptr_t)x % 16) || ((uintptr_t)skip % 16) || ((uintptr_t)out % 16) || ((uintptr_t)out2 % 16)) {
        set_error("iconv_forward_chain: tensor pointers must be 16-byte aligned");
        return ICONV_ERR_ALIGN;
    }
    int rc = umma_chain_opt_in();
    if (rc != ICONV_OK) return rc;
    const long long m_total = (long long)d1.n * d1.h * d1.w;
    CUtensorMap tmap_x, tmap_out, tmap_skip;
    rc = umma_encode_2d(&tmap_x, (const uint8_t *)x + d1.in_c_offset, d1.c_in, m_total, d1.in_c_total, c->k1, BLOCK_M, c->k1);
    if (rc == ICONV_OK) rc = umma_encode_2d(&tmap_out, (uint8_t *)out + d1.out_c_offset, d1.c_out, m_total, d1.out_c_total, 32, 32, 32);
    if (rc == ICONV_OK) rc = umma_encode_2d(&tmap_skip, (const uint8_t *)skip + d1.skip_c_offset, d1.c_out, m_total, d1.skip_c_total, 32, 32, 32);
    if (rc != ICONV_OK) return rc;
    ChainArgs a;
    memset(&a, 0, sizeof(a));
    a.m_total = m_total;
    a.m_tiles = (int)((m_total + BLOCK_M - 1) / BLOCK_M);
    a.n_tiles = c->n_tiles; a.k1 = c->k1; a.c2 = c->c2; a.stages = c->stages; a.skip_ring = c->skip_ring;
    a.idesc1 = (2u << 4) | (1u << 10) | ((unsigned)(128 >> 3) << 17) | ((unsigned)(BLOCK_M >> 4) << 24);
    a.idesc2 = (2u << 4) | (1u << 10) | ((unsigned)(c->c2 >> 3) << 17) | ((unsigned)(BLOCK_M >> 4) << 24);
    const unsigned long long layout = c->k1 == 128 ? 2ull : 4ull;
    a.desc_hi1 = (unsigned)((((unsigned long long)((8 * c->k1) >> 4) << 32) | (1ull << 46) | (layout << 61)) >> 32);
    a.q_mul = c->p1->q_mul; a.q_shift = c->p1->q_shift; a.q_half = (int)(1u << (c->p1->q_shift - 1)); a.skip_mul = d1.skip_mul;
    a.skip_xor = d1.skip_dtype == ICONV_S8 ? 0x80808080u : 0u;
    a.c_a = c->p1->params_packed;
    a.q2_mul = c->p2->q_mul; a.q2_shift = c->p2->q_shift;
    a.c_a2 = c->p2->params_packed;
    a.out2 = (uint8_t *)out2; a.out2_c_total = d2.out_c_total; a.out2_c_offset = d2.out_c_offset;
    a.status = device_status_ptr();
    if (!a.status) { set_error("device status word not available"); return ICONV_ERR_CUDA; }
    const int sms = umma_device_ready(current_device_slot());
    if (sms < 1) { set_error("iconv_forward_chain: device not initialised"); return ICONV_ERR_CUDA; }
    UmmaLaunch l;
    memset(&l, 0, sizeof(l));
    l.grid = (unsigned)(a.m_tiles < sms ? a.m_tiles : sms);
    l.smem = c->smem;
    l.stream = (cudaStream_t)cuda_stream;
    l.cluster = 1;
    ICONV_CUDA_TRY(umma_launch_pdl(umma_chain_kernel, l, tmap_x, c->tmap_w1, c->tmap_w2, tmap_out, tmap_skip, a));
    return ICONV_OK;
}

namespace iconv {

// Shared-memory opt-in of the two-layer kernel on the current device (once per device), after the
// other kernels' (which also fills the device's table entry).
int umma_chain_opt_in()
{
    static std::atomic<int> done[MAX_DEVICES];
    int rc = umma_init_once();
    if (rc != ICONV_OK) return rc;
    const int dev = current_device_slot();
    if (dev < 0) return ICONV_ERR_UNSUPPORTED;
    if (!done[dev].load(std::memory_order_acquire)) {
        ICONV_CUDA_TRY(cudaFuncSetAttribute(umma_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM));
        done[dev].store(1, std::memory_order_release);
    }
    return ICONV_OK;
}

}  // namespace iconv
