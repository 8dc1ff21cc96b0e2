// Host side of the GEMV kernel (small M): table of instantiations and the launch.
#include "../../include/kx.h"
#include "kx_internal.h"
#include "kx_gemv.cuh"

#include <cstring>

namespace kx {
namespace {

struct GemvVariant {
    int mr, rw;
    const void* fn;
};
#define KX_GEMV(MR, RW) \
    GemvVariant { MR, RW, reinterpret_cast<const void*>(&kx_gemv_kernel<MR, RW>) }
const GemvVariant kGemvVariants[] = {
    KX_GEMV(1, 1), KX_GEMV(2, 1), KX_GEMV(4, 1), KX_GEMV(1, 2), KX_GEMV(2, 2), KX_GEMV(4, 2),
    KX_GEMV(1, 4), KX_GEMV(2, 4), KX_GEMV(4, 4),
};

const GemvVariant* find_gemv(int mr, int rw) {
    for (const auto& v : kGemvVariants)
        if (v.mr == mr && v.rw == rw) return &v;
    return nullptr;
}

struct SkinnyVariant {
    int mb, fr, smem;
    const void* fn;
};
#define KX_SKINNY(MB, FR) \
    SkinnyVariant { MB, FR, kSkinnyWarps * 8 * MB * 16 * FR * 4, reinterpret_cast<const void*>(&kx_skinny_kernel<MB, FR>) }
const SkinnyVariant kSkinnyVariants[] = {
    KX_SKINNY(1, 1), KX_SKINNY(2, 1), KX_SKINNY(3, 1), KX_SKINNY(4, 1),
    KX_SKINNY(1, 2), KX_SKINNY(2, 2), KX_SKINNY(3, 2), KX_SKINNY(4, 2),
};
const SkinnyVariant* find_skinny(int mb, int fr) {
    for (const auto& v : kSkinnyVariants)
        if (v.mb == mb && v.fr == fr) return &v;
    return nullptr;
}

}  // namespace

int skinny_setup() {
    for (const auto& v : kSkinnyVariants)
        if (cudaFuncSetAttribute(v.fn, cudaFuncAttributeMaxDynamicSharedMemorySize, v.smem) != cudaSuccess) {
            cudaGetLastError();
            return KX_ERR_CUDA;
        }
    return KX_OK;
}

bool skinny_variant_exists(int rows_per_cta) { return rows_per_cta == 16 || rows_per_cta == 32; }

int launch_skinny(const GemvLaunch& a, cudaStream_t stream) {
    if (a.M < 1 || a.M > kSkinnyMaxM || (a.K % 8) != 0 || (a.N % 2) != 0) return KX_ERR_PLAN;
    const SkinnyVariant* v = find_skinny(static_cast<int>((a.M + 7) / 8), a.rows_per_cta / 16);
    if (!v || (a.rows_per_cta != 16 && a.rows_per_cta != 32)) return KX_ERR_PLAN;
    GemvParams p;
    p.X = static_cast<const uint16_t*>(a.X);
    p.W = static_cast<const uint16_t*>(a.W);
    p.bias = static_cast<const uint16_t*>(a.bias);
    p.R = static_cast<const uint16_t*>(a.R);
    p.Y = static_cast<uint16_t*>(a.Y);
    p.M = static_cast<int>(a.M);
    p.N = static_cast<int>(a.N);
    p.K = static_cast<int>(a.K);
    p.ldx = a.ldx;
    p.ldw = a.ldw;
    p.ldr = a.ldr;
    p.ldy = a.ldy;
    p.pf_bytes = a.pf_bytes;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>((a.N + a.rows_per_cta - 1) / a.rows_per_cta), 1, 1);
    cfg.blockDim = dim3(kSkinnyWarps * 32, 1, 1);
    cfg.dynamicSmemBytes = v->smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    int nattr = 0;
    if (a.pdl) {
        attr[nattr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[nattr].val.programmaticStreamSerializationAllowed = 1;
        ++nattr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = nattr;
    void* args[] = {&p};
    if (cudaLaunchKernelExC(&cfg, v->fn, args) != cudaSuccess) {
        cudaGetLastError();
        return KX_ERR_CUDA;
    }
    return KX_OK;
}

bool gemv_variant_exists(int rows_per_cta, int warps) {
    return find_gemv(1, rows_per_cta) != nullptr && warps >= 1 && warps <= kGemvMaxWarps;
}

int launch_gemv(const GemvLaunch& a, cudaStream_t stream) {
    if (a.M < 1 || a.M > kGemvMaxM || (a.K % 8) != 0 || a.rows_per_cta < 1 || (a.N % a.rows_per_cta) != 0)
        return KX_ERR_PLAN;
    const int mr = a.M == 1 ? 1 : a.M == 2 ? 2 : 4;
    const GemvVariant* v = find_gemv(mr, a.rows_per_cta);
    if (!v || a.warps < 1 || a.warps > kGemvMaxWarps) return KX_ERR_PLAN;
    GemvParams p;
    p.X = static_cast<const uint16_t*>(a.X);
    p.W = static_cast<const uint16_t*>(a.W);
    p.bias = static_cast<const uint16_t*>(a.bias);
    p.R = static_cast<const uint16_t*>(a.R);
    p.Y = static_cast<uint16_t*>(a.Y);
    p.M = static_cast<int>(a.M);
    p.N = static_cast<int>(a.N);
    p.K = static_cast<int>(a.K);
    p.ldx = a.ldx;
    p.ldw = a.ldw;
    p.ldr = a.ldr;
    p.ldy = a.ldy;
    p.pf_bytes = a.pf_bytes;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(a.N / a.rows_per_cta), 1, 1);
    cfg.blockDim = dim3(a.warps * 32, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    int nattr = 0;
    if (a.pdl) {
        attr[nattr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[nattr].val.programmaticStreamSerializationAllowed = 1;
        ++nattr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = nattr;
    void* args[] = {&p};
    if (cudaLaunchKernelExC(&cfg, v->fn, args) != cudaSuccess) {
        cudaGetLastError();
        return KX_ERR_CUDA;
    }
    return KX_OK;
}

}  // namespace kx
