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

// Arguments of the row kernels (RMSNorm, code books; see kx_kernels.cuh and kx_rowcode.cuh).
struct QuantParams {
    const uint16_t* A0;
    const uint16_t* A1;
    const uint16_t* gamma;
    int8_t* Q0;
    int8_t* Q1;
    float* S0;
    float* S1;
    uint8_t* SF0;          // FMT 2: chunked scale bytes
    long long rows0, M;
    int N;
    int kchunks;           // FMT 2: ceil(N / 128); FMT 3: ceil(N / 64)
    float eps;
    float gs;              // FMT 3: tensor scale (> 0)
};
// The kernels for rows of at most kRowCodeMaxN elements (kx_rowcode.cuh).  fmt: 0 INT8 / 1 E4M3 codes with one
// scale per row, 2 / 3 the block-scaled 8-bit / 4-bit formats, 4 the BF16 RMSNorm itself (qp.Q0 = output).
constexpr int kRowCodeMaxN = 8192;
constexpr int kRowCodeMaxPlainN = 16384;   // code books without normalisation
// rowcode_setup raises the kernels' shared-memory limit once per device.
int rowcode_setup();
int launch_rowcode(const QuantParams& qp, bool norm, int fmt, cudaStream_t stream, int sm_count);

}  // namespace kx
