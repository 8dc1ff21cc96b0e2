// Host side of kx_rowcode_kernel (rows of at most 8192 elements; plain code books up to 16384): instantiation
// table and launch.
#include "../../include/kx.h"
#include "kx_internal.h"
#include "kx_rowcode.cuh"

#include <algorithm>
#include <mutex>
#include <cstdlib>
#include <cstring>

namespace kx {
namespace {

template <int G, int NV>
const void* rowcode_fn(bool norm, int fmt, bool full) {
#define KX_RC(NORM, FMT) \
    (full ? reinterpret_cast<const void*>(&kx_rowcode_kernel<G, NV, NORM, FMT, true>) \
          : reinterpret_cast<const void*>(&kx_rowcode_kernel<G, NV, NORM, FMT, false>))
    switch (fmt) {
        case 0: return norm ? KX_RC(true, 0) : KX_RC(false, 0);
        case 1: return norm ? KX_RC(true, 1) : KX_RC(false, 1);
        case 2: return norm ? KX_RC(true, 2) : KX_RC(false, 2);
        case 3: return norm ? KX_RC(true, 3) : KX_RC(false, 3);
        case 4: return norm ? KX_RC(true, 4) : nullptr;
        default: return nullptr;
    }
#undef KX_RC
}

// the plain code books of longer rows (up to 16384 elements: 256 threads, 5..8 vectors per thread); no normalised
// forms, whose gamma and widened row would not fit the register file
template <int NV>
const void* rowcode_long_fn(int fmt, bool full) {
#define KX_RC(FMT) \
    (full ? reinterpret_cast<const void*>(&kx_rowcode_kernel<256, NV, false, FMT, true>) \
          : reinterpret_cast<const void*>(&kx_rowcode_kernel<256, NV, false, FMT, false>))
    switch (fmt) {
        case 0: return KX_RC(0);
        case 1: return KX_RC(1);
        case 2: return KX_RC(2);
        case 3: return KX_RC(3);
        default: return nullptr;
    }
#undef KX_RC
}

}  // namespace

namespace {
constexpr int ring_bytes(int nv) { return kRowDepth * nv * kRowThreads * 16; }

// CTAs of one instantiation that fit on an SM (asked once per kernel; 1..8)
int ctas_per_sm(const void* fn, int smem) {
    static std::mutex mu;
    static const void* fns[192];
    static int counts[192];
    static int used = 0;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < used; ++i)
        if (fns[i] == fn) return counts[i];
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fn, kRowThreads, smem) != cudaSuccess) {
        cudaGetLastError();
        n = 2;
    }
    n = std::max(1, std::min(n, 8));
    if (used < 192) {
        fns[used] = fn;
        counts[used] = n;
        ++used;
    }
    return n;
}

}  // namespace

int rowcode_setup() {
    const bool tf[2] = {false, true};
    for (bool norm : tf)
        for (int fmt = 0; fmt <= 4; ++fmt) {
            const void* fns[12] = {rowcode_fn<128, 1>(norm, fmt, false), rowcode_fn<128, 2>(norm, fmt, false),
                                   rowcode_fn<128, 3>(norm, fmt, false), rowcode_fn<128, 4>(norm, fmt, false),
                                   rowcode_fn<256, 3>(norm, fmt, false), rowcode_fn<256, 4>(norm, fmt, false),
                                   rowcode_fn<128, 1>(norm, fmt, true),  rowcode_fn<128, 2>(norm, fmt, true),
                                   rowcode_fn<128, 3>(norm, fmt, true),  rowcode_fn<128, 4>(norm, fmt, true),
                                   rowcode_fn<256, 3>(norm, fmt, true),  rowcode_fn<256, 4>(norm, fmt, true)};
            const int nvs[12] = {1, 2, 3, 4, 3, 4, 1, 2, 3, 4, 3, 4};
            if (!norm && fmt < 4) {
                const void* lf[8] = {rowcode_long_fn<5>(fmt, false), rowcode_long_fn<6>(fmt, false), rowcode_long_fn<7>(fmt, false),
                                     rowcode_long_fn<8>(fmt, false), rowcode_long_fn<5>(fmt, true),  rowcode_long_fn<6>(fmt, true),
                                     rowcode_long_fn<7>(fmt, true),  rowcode_long_fn<8>(fmt, true)};
                const int lnv[8] = {5, 6, 7, 8, 5, 6, 7, 8};
                for (int i = 0; i < 8; ++i)
                    if (cudaFuncSetAttribute(lf[i], cudaFuncAttributeMaxDynamicSharedMemorySize, ring_bytes(lnv[i])) != cudaSuccess) {
                        cudaGetLastError();
                        return KX_ERR_CUDA;
                    }
            }
            for (int i = 0; i < 12; ++i)
                if (fns[i] &&
                    cudaFuncSetAttribute(fns[i], cudaFuncAttributeMaxDynamicSharedMemorySize, ring_bytes(nvs[i])) != cudaSuccess) {
                    cudaGetLastError();
                    return KX_ERR_CUDA;
                }
        }
    return KX_OK;
}

int launch_rowcode(const QuantParams& qp, bool norm, int fmt, cudaStream_t stream, int sm_count) {
    if (qp.N < 8 || qp.N > (norm ? kRowCodeMaxN : kRowCodeMaxPlainN) || (qp.N % 8) != 0 || qp.M < 1) return KX_ERR_PLAN;
    const int nvec = qp.N / 8;
    // the fewest vectors per thread that cover the row with 128 threads; 256 threads for the longest rows
    const void* fn = nullptr;
    int rows_per_cta = 2, nv = 4;
    if (nvec <= 128) { fn = rowcode_fn<128, 1>(norm, fmt, nvec == 128); nv = 1; }
    else if (nvec <= 256) { fn = rowcode_fn<128, 2>(norm, fmt, nvec == 256); nv = 2; }
    else if (nvec <= 384) { fn = rowcode_fn<128, 3>(norm, fmt, nvec == 384); nv = 3; }
    else if (nvec <= 512) fn = rowcode_fn<128, 4>(norm, fmt, nvec == 512);
    else if (nvec <= 768) { fn = rowcode_fn<256, 3>(norm, fmt, nvec == 768); nv = 3; rows_per_cta = 1; }
    else if (nvec <= 1024) { fn = rowcode_fn<256, 4>(norm, fmt, nvec == 1024); rows_per_cta = 1; }
    else {
        rows_per_cta = 1;
        if (nvec <= 1280) { fn = rowcode_long_fn<5>(fmt, nvec == 1280); nv = 5; }
        else if (nvec <= 1536) { fn = rowcode_long_fn<6>(fmt, nvec == 1536); nv = 6; }
        else if (nvec <= 1792) { fn = rowcode_long_fn<7>(fmt, nvec == 1792); nv = 7; }
        else { fn = rowcode_long_fn<8>(fmt, nvec == 2048); nv = 8; }
    }
    if (!fn) return KX_ERR_PLAN;
    const int smem = ring_bytes(nv);
    const long long steps = (qp.M + rows_per_cta - 1) / rows_per_cta;
    // The fused kernels (normalisation + code book) are bound by instruction issue: one persistent CTA per slot,
    // which pays for gamma and the first loads once.  The plain ones (normalisation only, code book only) are
    // HBM-bound, and under a saturated memory system SMs progress at different rates: they get about 3.5 steps per
    // CTA (at most 8 CTAs per slot), so that the hardware's block scheduler evens the SMs out.
    const long long resident = static_cast<long long>(ctas_per_sm(fn, smem)) * sm_count;
    long long mult = 1;
    if (!norm || fmt == 4) mult = std::max(1ll, std::min(8ll, (2 * steps) / (7 * resident)));
#ifdef KX_TRACE
    if (const char* e = std::getenv("KX_DEV_ROW_GRID_MULT")) mult = std::max(1, std::atoi(e));
#endif
    const long long grid = std::min(steps, resident * mult);
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kRowThreads, 1, 1);
    cfg.dynamicSmemBytes = static_cast<size_t>(smem);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    QuantParams p = qp;
    void* args[] = {&p};
    if (cudaLaunchKernelExC(&cfg, fn, args) != cudaSuccess) {
        cudaGetLastError();
        return KX_ERR_CUDA;
    }
    return KX_OK;
}

}  // namespace kx
