// kx_gemv_kernel: Y = X W^T (+ bias) (+ R) for a handful of rows of X (M <= 4), the
// decode-like end of the per-M specialisation of Appendix A, Algorithm 3, and the
// memory-scheduling strategy of Table 1: the job is to read W [N, K] from HBM exactly once at
// the full memory rate; the arithmetic (2 M flops per weight element) is far below the FP32 rate of
// the CUDA cores, so no tensor core, no tensor memory and no shared-memory pipeline are used.
//
// One CTA owns RW consecutive rows of W (= RW output columns) over the whole K range.  The K range is cut
// into 16-byte chunks (8 BF16); chunk c belongs to thread c % T (T = threads of the CTA, chosen by the host
// so that a thread's chunks of a row fit in one batch of loads), so one pass of the CTA over a row reads
// 16 T contiguous bytes.  Every thread keeps U x RW independent 16-byte loads of W in flight
// (non-coherent path, no L1 allocation), multiplies them with the matching chunks of the MR rows of X
// (read through L1: X is a few KB and is shared by every CTA of the SM) and accumulates in FP32 in chunk
// order.  Partial sums are combined by a shuffle tree inside each warp and then across the warps in warp
// order, so the summation order is fixed (deterministic run to run); bias and residual are added once,
// in FP32, before the single rounding to BF16.  R may alias Y: the one thread that writes an output
// element is the one that read its residual value.
//
// Before waiting for the previous kernel of the stream (programmatic dependent launch) the CTA only asks
// for its W rows to be brought into L2 (a hint: no data is consumed before the wait).
#pragma once
#include "kx_ptx.cuh"

namespace kx {

struct GemvParams {
    const uint16_t* X;
    const uint16_t* W;
    const uint16_t* bias;      // or null
    const uint16_t* R;         // or null; may alias Y
    uint16_t* Y;
    int M, N, K;               // 1 <= M <= MR, N % RW == 0, K % 8 == 0
    long long ldx, ldw, ldr, ldy;   // row pitches in elements
    int pf_bytes;              // bytes of each W row to request into L2 before the dependency wait (0 = none)
};

__device__ __forceinline__ uint4 ld_stream_u4(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::256B.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
// Ask for `bytes` (a multiple of 16, 16-byte aligned start) to be brought into L2; no completion to wait for.
__device__ __forceinline__ void prefetch_l2_bulk(const void* p, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

constexpr int kGemvMaxWarps = 16;

template <int MR, int RW>
__global__ void __launch_bounds__(kGemvMaxWarps * 32)
kx_gemv_kernel(const GemvParams p) {
    constexpr int U = (RW >= 4) ? 2 : 4;       // U * RW 16-byte loads of W in flight per thread
    __shared__ float s_red[kGemvMaxWarps][RW * MR];
    const int T = blockDim.x, WARPS = T >> 5;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long n0 = static_cast<long long>(blockIdx.x) * RW;
    const int nch = p.K >> 3;

    if (p.pf_bytes > 0 && tid < RW)
        prefetch_l2_bulk(p.W + (n0 + tid) * p.ldw, static_cast<uint32_t>(p.pf_bytes));
    pdl_wait_prior();
    pdl_launch_dependents();

    const uint4* wrow[RW];
#pragma unroll
    for (int r = 0; r < RW; ++r) wrow[r] = reinterpret_cast<const uint4*>(p.W + (n0 + r) * p.ldw);
    const uint4* xrow[MR];
#pragma unroll
    for (int m = 0; m < MR; ++m)
        xrow[m] = reinterpret_cast<const uint4*>(p.X + static_cast<long long>(m < p.M ? m : p.M - 1) * p.ldx);

    float acc[RW][MR];
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
        for (int m = 0; m < MR; ++m) acc[r][m] = 0.f;

#pragma unroll 1
    for (int c0 = tid; c0 < nch; c0 += T * U) {
        uint4 w[U][RW];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = c0 + u * T;
#pragma unroll
            for (int r = 0; r < RW; ++r) w[u][r] = (c < nch) ? ld_stream_u4(wrow[r] + c) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = c0 + u * T;
            if (c < nch) {
                float xf[MR][8];
#pragma unroll
                for (int m = 0; m < MR; ++m) {
                    const uint4 x = __ldg(xrow[m] + c);
                    xf[m][0] = bf16_lo(x.x); xf[m][1] = bf16_hi(x.x); xf[m][2] = bf16_lo(x.y); xf[m][3] = bf16_hi(x.y);
                    xf[m][4] = bf16_lo(x.z); xf[m][5] = bf16_hi(x.z); xf[m][6] = bf16_lo(x.w); xf[m][7] = bf16_hi(x.w);
                }
#pragma unroll
                for (int r = 0; r < RW; ++r) {
                    const uint4 v = w[u][r];
                    const float wf[8] = {bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y),
                                         bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w)};
#pragma unroll
                    for (int m = 0; m < MR; ++m)
#pragma unroll
                        for (int i = 0; i < 8; ++i) acc[r][m] = fmaf(wf[i], xf[m][i], acc[r][m]);
                }
            }
        }
    }

#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
        for (int m = 0; m < MR; ++m) {
            float v = acc[r][m];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) s_red[warp][r * MR + m] = v;
        }
    __syncthreads();
    if (tid < RW * MR) {
        const int r = tid / MR, m = tid - r * MR;
        if (m < p.M) {
            float v = 0.f;
            for (int w = 0; w < WARPS; ++w) v += s_red[w][tid];
            const long long n = n0 + r;
            if (p.bias) v += __uint_as_float(static_cast<uint32_t>(__ldg(p.bias + n)) << 16);
            if (p.R) v += __uint_as_float(static_cast<uint32_t>(p.R[m * p.ldr + n]) << 16);
            p.Y[m * p.ldy + n] = static_cast<uint16_t>(pack_bf16x2(v, 0.f) & 0xFFFFu);
        }
    }
}


// kx_skinny_kernel: the same job for up to 32 rows of X, where 2 M flops per weight element are too many for
// the CUDA cores but the problem is still bound by reading W once (Table 1, memory strategy; the per-M
// specialisation of Algorithm 3).  Warp-level tensor-core instructions (mma.sync m16n8k16, BF16 x BF16 ->
// FP32) are fed straight from registers, so there is no shared-memory pipeline, no tensor-memory accumulator
// to hand over and no split-K across CTAs: the whole chain behind the last load is one reduction over the
// warps of the CTA in shared memory.
//
// One CTA owns 16 FR consecutive rows of W over the whole K range; its 16 warps take the 32-element steps
// of K in turn (warp w takes steps w, w + 16, ...).  In a step, lane (g, t) (g = lane / 4, t = lane % 4)
// loads 16 bytes = 8 consecutive K elements, starting at element 8 t of the step, of W rows g and g + 8 of
// every 16-row fragment (non-coherent path, no L1 allocation) and of X rows g, g + 8, ... (read-only path
// through L1 / L2).  The tensor-core instruction sums over 16 K slots; which element of K sits in which
// slot does not matter as long as both operands agree, so the 8 elements a lane holds serve two
// instructions (elements 0..3 and 4..7 of every lane) and no data is exchanged between lanes.  The warps'
// partial tiles are added in warp order (fixed summation order), bias and residual are added once, in
// FP32, before the single rounding to BF16; the thread that writes an output element is the one that read
// its residual value, so R may alias Y.
constexpr int kSkinnyWarps = 16;

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// MB = groups of 8 rows of X (M <= 8 MB), FR = 16-row fragments of W per CTA.
template <int MB, int FR>
__global__ void __launch_bounds__(kSkinnyWarps * 32)
kx_skinny_kernel(const GemvParams p) {
    constexpr int ROWS = 16 * FR, MR = 8 * MB, UNR = 2;
    extern __shared__ float s_part[];                       // [warp][m][n]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const long long n0 = static_cast<long long>(blockIdx.x) * ROWS;
    const int nch = p.K >> 3;                               // 16-byte chunks per row
    const int nit = (p.K + 31) >> 5;                        // steps of 32 K elements

    if (p.pf_bytes > 0 && tid < ROWS && n0 + tid < p.N)
        prefetch_l2_bulk(p.W + (n0 + tid) * p.ldw, static_cast<uint32_t>(p.pf_bytes));
    pdl_wait_prior();
    pdl_launch_dependents();

    const uint4* wp[2 * FR];
#pragma unroll
    for (int i = 0; i < 2 * FR; ++i) {
        long long r = n0 + 8 * i + g;                       // fragment i / 2, rows g and g + 8
        if (r >= p.N) r = p.N - 1;                          // rows past the end: loaded again, never stored
        wp[i] = reinterpret_cast<const uint4*>(p.W + r * p.ldw);
    }
    const uint4* xp[MB];
#pragma unroll
    for (int j = 0; j < MB; ++j) {
        const int m = 8 * j + g;
        xp[j] = reinterpret_cast<const uint4*>(p.X + static_cast<long long>(m < p.M ? m : p.M - 1) * p.ldx);
    }
    float acc[FR][MB][4];
#pragma unroll
    for (int f = 0; f < FR; ++f)
#pragma unroll
        for (int j = 0; j < MB; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[f][j][e] = 0.f;

#pragma unroll 1
    for (int it0 = warp; it0 < nit; it0 += kSkinnyWarps * UNR) {
        uint4 w[UNR][2 * FR], x[UNR][MB];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int c = (it0 + u * kSkinnyWarps) * 4 + t;
            const bool ok = c < nch;                        // also false for steps past the end
#pragma unroll
            for (int i = 0; i < 2 * FR; ++i) w[u][i] = ok ? ld_stream_u4(wp[i] + c) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int j = 0; j < MB; ++j) x[u][j] = ok ? __ldg(xp[j] + c) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u)
#pragma unroll
            for (int f = 0; f < FR; ++f)
#pragma unroll
                for (int j = 0; j < MB; ++j) {
                    mma_bf16_16816(acc[f][j], w[u][2 * f].x, w[u][2 * f + 1].x, w[u][2 * f].y, w[u][2 * f + 1].y,
                                   x[u][j].x, x[u][j].y);
                    mma_bf16_16816(acc[f][j], w[u][2 * f].z, w[u][2 * f + 1].z, w[u][2 * f].w, w[u][2 * f + 1].w,
                                   x[u][j].z, x[u][j].w);
                }
    }

    // accumulator element e of fragment (f, j): W row 16 f + g + 8 (e / 2), X row 8 j + 2 t + (e % 2)
    float* mine = s_part + warp * (MR * ROWS);
#pragma unroll
    for (int f = 0; f < FR; ++f)
#pragma unroll
        for (int j = 0; j < MB; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                mine[(8 * j + 2 * t + (e & 1)) * ROWS + 16 * f + g + 8 * (e >> 1)] = acc[f][j][e];
    __syncthreads();
    for (int o = tid; o < MR * ROWS / 2; o += kSkinnyWarps * 32) {
        const int m = o / (ROWS / 2), nn = (o - m * (ROWS / 2)) * 2;
        const long long n = n0 + nn;
        if (m < p.M && n < p.N) {                           // N is even: n + 1 < N as well
            float v0 = 0.f, v1 = 0.f;
#pragma unroll
            for (int wv = 0; wv < kSkinnyWarps; ++wv) {
                const float2 q = *reinterpret_cast<const float2*>(s_part + wv * (MR * ROWS) + m * ROWS + nn);
                v0 += q.x;
                v1 += q.y;
            }
            if (p.bias) {
                const uint32_t bb = __ldg(reinterpret_cast<const uint32_t*>(p.bias + n));
                v0 += bf16_lo(bb);
                v1 += bf16_hi(bb);
            }
            if (p.R) {
                const uint32_t rr = *reinterpret_cast<const uint32_t*>(p.R + m * p.ldr + n);
                v0 += bf16_lo(rr);
                v1 += bf16_hi(rr);
            }
            *reinterpret_cast<uint32_t*>(p.Y + m * p.ldy + n) = pack_bf16x2(v0, v1);
        }
    }
}

}  // namespace kx
