// Host side of kx_rowcode_kernel (rows of at most 8192 elements): instantiation table and launch.
#include "../../include/kx.h"
#include "kx_internal.h"
#include "kx_rowcode.cuh"

#include <algorithm>
#include <mutex>
#include <cstring>

namespace kx {
namespace {

template <int G, int NV>
const void* rowcode_fn(bool norm, int fmt) {
#define KX_RC(NORM, FMT) reinterpret_cast<const void*>(&kx_rowcode_kernel<G, NV, NORM, FMT>)
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

// CTAs of one instantiation that fit on an SM (asked once per kernel; 1..8)
int ctas_per_sm(const void* fn) {
    static std::mutex mu;
    static const void* fns[64];
    static int counts[64];
    static int used = 0;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < used; ++i)
        if (fns[i] == fn) return counts[i];
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fn, kRowThreads, 0) != cudaSuccess) {
        cudaGetLastError();
        n = 2;
    }
    n = std::max(1, std::min(n, 8));
    if (used < 64) {
        fns[used] = fn;
        counts[used] = n;
        ++used;
    }
    return n;
}

}  // namespace

int launch_rowcode(const QuantParams& qp, bool norm, int fmt, cudaStream_t stream, int sm_count) {
    if (qp.N < 8 || qp.N > kRowCodeMaxN || (qp.N % 8) != 0 || qp.M < 1) return KX_ERR_PLAN;
    const int nvec = qp.N / 8;
    // the fewest vectors per thread that cover the row with 128 threads; 256 threads for the longest rows
    const void* fn = nullptr;
    int rows_per_cta = 2;
    if (nvec <= 128) fn = rowcode_fn<128, 1>(norm, fmt);
    else if (nvec <= 256) fn = rowcode_fn<128, 2>(norm, fmt);
    else if (nvec <= 512) fn = rowcode_fn<128, 4>(norm, fmt);
    else { fn = rowcode_fn<256, 4>(norm, fmt); rows_per_cta = 1; }
    if (!fn) return KX_ERR_PLAN;
    const long long steps = (qp.M + rows_per_cta - 1) / rows_per_cta;
    // persistent over row steps: as many CTAs as fit on the device at once, fewer when there is less work
    const long long resident = static_cast<long long>(ctas_per_sm(fn)) * sm_count;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(std::min(steps, resident)), 1, 1);
    cfg.blockDim = dim3(kRowThreads, 1, 1);
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
