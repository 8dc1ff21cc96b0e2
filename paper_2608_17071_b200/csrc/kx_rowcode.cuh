// kx_rowcode_kernel: the row kernels of Appendix A, Algorithm 7 for rows of at most 8192 elements (plain code
// books: 16384, with up to eight vectors per thread) -
// RMSNorm ("add + RMSNorm" after the projection), the per-row and per-block code books ("activation
// quantization", "quantize gate/up weights") and the two fused ("fused add + RMSNorm + activation
// quantization").  Same arithmetic, element by element, as kx_rmsnorm_kernel / kx_rowquant_kernel
// (which keep the longer rows); what differs is how the work is laid out, because at these row
// lengths the older kernels are bound by instruction issue, not by HBM:
//
//   * G = 128 or 256 threads share a row and a thread owns NV <= 4 (plain code books: 8) 16-byte vectors of it (32 elements
//     when the row has 4096), so the fixed per-row work of a thread (two shuffle trees, two group
//     barriers, the divisions) is spread over twice as many elements; a CTA of 256 threads works on
//     256 / G neighbouring rows at once, each group with a named barrier of its own;
//   * the FP32 arithmetic runs two elements per instruction (mul / fma .f32x2: the same IEEE results as
//     the scalar forms), the maxima are taken on packed BF16 pairs (exact: a maximum rounds nothing),
//     and gamma is widened to FP32 once per thread and kept in registers across rows;
//   * a thread copies its own vectors of the next three row steps into private slots of shared memory
//     with cp.async while it works on the current one, so the HBM latency of a row is not paid between
//     its barriers; nothing but the issuing thread ever reads a slot, hence no barrier guards it.
//
// Summation order of the sum of squares (fixed, so runs are reproducible and kx_rmsnorm and the fused
// kernels give the same bits): per thread two chains (even / odd elements of its vectors, in vector
// order), added; a shuffle tree inside each warp; the warps of the group in order.
// HBM-bound by design: 2 N bytes read per row; N + 4 (8-bit codes), N + N/32, N/2 + N/16 or 2 N written.
#pragma once
#include "kx_internal.h"
#include "kx_ptx.cuh"

namespace kx {

constexpr int kRowThreads = 256;
constexpr int kRowDepth = 3;          // row steps a thread has in flight or in use: enough bytes on their way per SM
                                      // to keep HBM busy when reads compete with the previous kernel's write-back

// ---- two binary32 values in one 64-bit register (sm_100: one instruction for both lanes)
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// a BF16 pair widened (exact): low element in the low lane
__device__ __forceinline__ uint64_t f2_from_bf16x2(uint32_t w) { return f2_pack(bf16_lo(w), bf16_hi(w)); }
__device__ __forceinline__ uint32_t bf16x2_from_f2(uint64_t v) {
    float lo, hi;
    f2_unpack(v, lo, hi);
    return pack_bf16x2(lo, hi);
}
// max(acc, |w|) on both BF16 lanes (a NaN lane is ignored, as fmaxf does)
__device__ __forceinline__ uint32_t bf16x2_absmax(uint32_t acc, uint32_t w) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(acc), "r"(w & 0x7FFF7FFFu));
    return d;
}
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory");
}
__device__ __forceinline__ void group_barrier(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// FMT 0 INT8 / 1 E4M3 codes with one FP32 scale per row; 2 E4M3 codes with one E8M0 scale per 32 elements;
// 3 E2M1 codes with one E4M3 scale per 16 elements and a tensor scale; 4 BF16 (the RMSNorm itself, NORM only:
// Q0 is then the BF16 output, which may be the input).  The formats' definitions are those of
// kx_rowquant_kernel.  G * NV * 8 >= N; FULL: equal (every vector of every thread lies inside the row).
template <int G, int NV, bool NORM, int FMT, bool FULL>
#ifndef KX_ROW_MINB
#define KX_ROW_MINB 2
#endif
__global__ void __launch_bounds__(kRowThreads, KX_ROW_MINB)
kx_rowcode_kernel(const QuantParams p) {
    static_assert(G == 128 || G == 256, "threads per row");
    static_assert(FMT != 4 || NORM, "format 4 is the normalised row");
    constexpr int RPC = kRowThreads / G;                 // rows per CTA and step
    constexpr int WG = G / 32;                           // warps per row
    constexpr float kTop = (FMT == 1) ? 448.0f : 127.0f;
    extern __shared__ uint4 s_ring[];                    // [kRowDepth][NV][kRowThreads]
    __shared__ __align__(16) float s_sum[2][RPC][WG];
    __shared__ __align__(16) float s_max[2][RPC][WG];
    const int tid = threadIdx.x, lane = tid & 31;
    const int gi = tid / G, g = tid - gi * G, wg = g >> 5;
    const int N = p.N, nvec = N / 8;
    const long long steps = (p.M + RPC - 1) / RPC;

    bool valid[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) valid[i] = FULL || g + i * G < nvec;
    const float inv_n = 1.0f / static_cast<float>(N);
    uint64_t gam[NORM ? NV : 1][4];                      // gamma, widened once (weights: not produced by the previous kernel)
    if constexpr (NORM) {
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            uint4 gv = make_uint4(0u, 0u, 0u, 0u);
            if (valid[i]) gv = __ldg(reinterpret_cast<const uint4*>(p.gamma) + g + i * G);
            gam[i][0] = f2_from_bf16x2(gv.x);
            gam[i][1] = f2_from_bf16x2(gv.y);
            gam[i][2] = f2_from_bf16x2(gv.z);
            gam[i][3] = f2_from_bf16x2(gv.w);
        }
    }
    pdl_wait_prior();
    pdl_launch_dependents();

    // the row of this thread's group at a step, and where it starts
    auto row_of = [&](long long step) { return step * RPC + gi; };
    auto src_of = [&](long long m) -> const uint4* {
        const bool second = m >= p.rows0;
        return reinterpret_cast<const uint4*>((second ? p.A1 : p.A0) + (second ? m - p.rows0 : m) * N);
    };
    auto fetch = [&](long long step, int slot) {
        const long long m = row_of(step);
        if (step < steps && m < p.M) {
            const uint4* src = src_of(m);
#pragma unroll
            for (int i = 0; i < NV; ++i)
                if (valid[i]) cp_async16(smem_u32(&s_ring[(slot * NV + i) * kRowThreads + tid]), src + g + i * G);
        }
        cp_async_commit();
    };
#pragma unroll
    for (int d = 0; d < kRowDepth; ++d) fetch(blockIdx.x + static_cast<long long>(d) * gridDim.x, d);

    int slot = 0, par = 0;
    for (long long step = blockIdx.x; step < steps; step += gridDim.x, slot = (slot + 1 == kRowDepth) ? 0 : slot + 1, par ^= 1) {
        const long long m = row_of(step);
        const bool live = m < p.M;                       // the last step of an odd row count has an idle group
        const bool second = m >= p.rows0;
        const long long r = second ? m - p.rows0 : m;
        cp_async_wait<kRowDepth - 1>();
        uint4 v[NV];
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            // a group without a row (last step of an odd row count) computes on whatever the slot holds and stores nothing
            if (FULL) v[i] = s_ring[(slot * NV + i) * kRowThreads + tid];
            else v[i] = (valid[i] && live) ? s_ring[(slot * NV + i) * kRowThreads + tid] : make_uint4(0u, 0u, 0u, 0u);
        }

        if constexpr (NORM) {
            uint64_t h2[NV][4];
            uint64_t ss2 = 0ull;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const uint32_t w4[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    h2[i][k] = f2_from_bf16x2(w4[k]);
                    ss2 = f2_fma(h2[i][k], h2[i][k], ss2);
                }
            }
            // the slot's contents are in registers (the sums above used them): refill it
            fetch(step + static_cast<long long>(kRowDepth) * gridDim.x, slot);
            float se, so;
            f2_unpack(ss2, se, so);
            float ss = se + so;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
            if (lane == 0) s_sum[par][gi][wg] = ss;
            group_barrier(1 + gi, G);
            float t = 0.f;
            {
                float part[WG];
#pragma unroll
                for (int w = 0; w < WG; w += 4)
                    *reinterpret_cast<float4*>(&part[w]) = *reinterpret_cast<const float4*>(&s_sum[par][gi][w]);
#pragma unroll
                for (int w = 0; w < WG; ++w) t += part[w];
            }
            const float inv = rsqrtf(t * inv_n + p.eps);
            const uint64_t inv2 = f2_pack(inv, inv);
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                uint32_t o4[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) o4[k] = bf16x2_from_f2(f2_mul(f2_mul(h2[i][k], inv2), gam[i][k]));
                v[i] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
            }
        }

        if constexpr (FMT == 4) {
            if (live) {
                uint4* zrow = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(p.Q0) + m * N);
#pragma unroll
                for (int i = 0; i < NV; ++i)
                    if (valid[i]) zrow[g + i * G] = v[i];
            }
        } else if constexpr (FMT == 2) {
            uint2* qrow = reinterpret_cast<uint2*>(p.Q0 + r * N);
            uint8_t* const sfrow = p.SF0 + (r >> 7) * p.kchunks * 512 + (r & 31) * 16 + ((r & 127) >> 5) * 4;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const int idx = g + i * G;
                const bool ok = valid[i] && live;
                const uint32_t w4[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
                uint32_t mx = 0u;
#pragma unroll
                for (int k = 0; k < 4; ++k) mx = bf16x2_absmax(mx, w4[k]);
                float bmax = fmaxf(bf16_lo(mx), bf16_hi(mx));
                // N % 32 == 0: the four threads of a block are all valid or all invalid, and sit in one warp
                bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 1));
                bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 2));
                uint32_t e = 127u;                           // lanes past the row end carry the padding value
                if (ok) {
                    const int field = static_cast<int>(__float_as_uint(bmax) >> 23);
                    e = (bmax > 0.f) ? static_cast<uint32_t>(max(field - 8, 0)) : 127u;
                    const float mult = __uint_as_float((254u - e) << 23);   // 2^(127 - e), e <= 247
                    const uint64_t mult2 = f2_pack(mult, mult);
                    float z[8];
#pragma unroll
                    for (int k = 0; k < 4; ++k) f2_unpack(f2_mul(f2_from_bf16x2(w4[k]), mult2), z[2 * k], z[2 * k + 1]);
                    qrow[idx] = make_uint2(pack_e4m3x4(z[0], z[1], z[2], z[3]), pack_e4m3x4(z[4], z[5], z[6], z[7]));
                }
                // one byte per block, stored by the block's first lane; lanes past the row end but inside the row's
                // last chunk write that chunk's padding entries
                if (live && (g & 3) == 0 && (idx >> 4) < p.kchunks) sfrow[(idx >> 4) * 512 + ((idx >> 2) & 3)] = static_cast<uint8_t>(e);
            }
            if (live && r == p.M - 1) {                      // rows up to the next multiple of 128
                const long long pad_rows = ((p.M + 127) & ~127ll) - p.M;
                const int per_row = p.kchunks * 4;
                for (long long t = g; t < pad_rows * per_row; t += G) {
                    const long long rr = p.M + t / per_row;
                    const int jj = static_cast<int>(t % per_row);
                    p.SF0[((rr >> 7) * p.kchunks + (jj >> 2)) * 512 + (rr & 31) * 16 + ((rr & 127) >> 5) * 4 + (jj & 3)] = 127;
                }
            }
        } else if constexpr (FMT == 3) {
            uint32_t* qrow = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(p.Q0) + r * (N / 2));
            uint8_t* const sfrow = p.SF0 + (r >> 7) * p.kchunks * 512 + (r & 31) * 16 + ((r & 127) >> 5) * 4;
            const float d6 = __fmul_rn(6.0f, p.gs);
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const int idx = g + i * G;
                const bool ok = valid[i] && live;
                const uint32_t w4[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
                uint32_t mx = 0u;
#pragma unroll
                for (int k = 0; k < 4; ++k) mx = bf16x2_absmax(mx, w4[k]);
                float bmax = fmaxf(bf16_lo(mx), bf16_hi(mx));
                // N % 16 == 0: the two threads of a block are both valid or both invalid
                bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 1));
                uint32_t sb = 0u;                            // lanes past the row end carry the padding value
                if (ok) {
                    sb = pack_e4m3x4(__fdiv_rn(bmax, d6), 0.f, 0.f, 0.f) & 0xFFu;
                    const float dq = __fmul_rn(e4m3_to_f32(sb), p.gs);
                    const float rcp = (dq > 0.f) ? __fdiv_rn(1.0f, dq) : 0.f;
                    const uint64_t rcp2 = f2_pack(rcp, rcp);
                    float z[8];
#pragma unroll
                    for (int k = 0; k < 4; ++k) f2_unpack(f2_mul(f2_from_bf16x2(w4[k]), rcp2), z[2 * k], z[2 * k + 1]);
                    qrow[idx] = (dq > 0.f) ? pack_e2m1x8(z) : 0u;
                }
                // one byte per block, stored by the block's first lane, the padding entries of the row's last chunk included
                if (live && (g & 1) == 0 && (idx >> 3) < p.kchunks) sfrow[(idx >> 3) * 512 + ((idx >> 1) & 3)] = static_cast<uint8_t>(sb);
            }
            if (live && r == p.M - 1) {
                const long long pad_rows = ((p.M + 127) & ~127ll) - p.M;
                const int per_row = p.kchunks * 4;
                for (long long t = g; t < pad_rows * per_row; t += G) {
                    const long long rr = p.M + t / per_row;
                    const int jj = static_cast<int>(t % per_row);
                    p.SF0[((rr >> 7) * p.kchunks + (jj >> 2)) * 512 + (rr & 31) * 16 + ((rr & 127) >> 5) * 4 + (jj & 3)] = 0;
                }
            }
        } else {
            // row maximum of |z| (exact: BF16 values)
            uint32_t mx = 0u;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                mx = bf16x2_absmax(mx, v[i].x);
                mx = bf16x2_absmax(mx, v[i].y);
                mx = bf16x2_absmax(mx, v[i].z);
                mx = bf16x2_absmax(mx, v[i].w);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = bf16x2_max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            if (lane == 0) s_max[par][gi][wg] = fmaxf(bf16_lo(mx), bf16_hi(mx));
            group_barrier(1 + gi, G);
            float a = 0.f;
            {
                float part[WG];
#pragma unroll
                for (int w = 0; w < WG; w += 4)
                    *reinterpret_cast<float4*>(&part[w]) = *reinterpret_cast<const float4*>(&s_max[par][gi][w]);
#pragma unroll
                for (int w = 0; w < WG; ++w) a = fmaxf(a, part[w]);
            }
            if (wg == 0) {                                   // one warp of the group pays for the scale's division
                if (g == 0 && live) (second ? p.S1 : p.S0)[r] = (a > 0.f) ? __fdiv_rn(a, kTop) : 1.0f;
            }
            const float rcp = (a > 0.f) ? __fdiv_rn(kTop, a) : 0.f;
            const uint64_t rcp2 = f2_pack(rcp, rcp);
            if (live) {
                uint2* qrow = reinterpret_cast<uint2*>((second ? p.Q1 : p.Q0) + r * N);
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    if (!valid[i]) continue;
                    const uint32_t w4[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
                    // |z| <= a and rcp = fl(top / a) keep |z * rcp| below top + 1/2, so the INT8 codes are already
                    // within -127..127; the packing instruction saturates anyway
                    float t[8];
#pragma unroll
                    for (int k = 0; k < 4; ++k) f2_unpack(f2_mul(f2_from_bf16x2(w4[k]), rcp2), t[2 * k], t[2 * k + 1]);
                    if constexpr (FMT == 1) {
                        qrow[g + i * G] = make_uint2(pack_e4m3x4(t[0], t[1], t[2], t[3]), pack_e4m3x4(t[4], t[5], t[6], t[7]));
                    } else {
                        int q[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) q[k] = __float2int_rn(t[k]);
                        qrow[g + i * G] = make_uint2(pack_s8x4_sat(q[0], q[1], q[2], q[3]), pack_s8x4_sat(q[4], q[5], q[6], q[7]));
                    }
                }
            }
        }
        // without the normalisation the slot is refilled only here, after everything that read v has run
        if constexpr (!NORM) fetch(step + static_cast<long long>(kRowDepth) * gridDim.x, slot);
    }
    cp_async_wait<0>();
}

}  // namespace kx
