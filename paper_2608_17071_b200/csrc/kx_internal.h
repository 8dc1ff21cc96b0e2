// Declarations shared by the translation units of libkx.so (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace kx {

// Arguments of one launch of the GEMV kernel (small M); see kx_gemv.cuh.
struct GemvLaunch {
    const void* X;
    const void* W;
    const void* bias;
    const void* R;
    void* Y;
    long long M, N, K;
    long long ldx, ldw, ldr, ldy;
    int rows_per_cta;      // rows of W per CTA: 1, 2 or 4 (must divide N)
    int warps;             // warps per CTA that share the K range: 1..16
    int pf_bytes;          // L2 request per W row ahead of the dependency wait
    bool pdl;              // programmatic stream serialization
};
constexpr int kGemvMaxM = 4;
constexpr int kSkinnyMaxM = 32;
// true if a kernel instantiation exists for this combination
bool gemv_variant_exists(int rows_per_cta, int warps);
// Enqueues the kernel; returns a kx_status value.
int launch_gemv(const GemvLaunch& a, cudaStream_t stream);
// The warp-level tensor-core kernel for 5..32 rows (kx_skinny_kernel): same arguments; rows_per_cta is 16 or
// 32 and `warps` is ignored.  skinny_setup raises the kernels' shared-memory limit once per device.
int skinny_setup();
bool skinny_variant_exists(int rows_per_cta);
int launch_skinny(const GemvLaunch& a, cudaStream_t stream);

}  // namespace kx
