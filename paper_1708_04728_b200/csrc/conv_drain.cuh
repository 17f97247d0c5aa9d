// Epilogues that drain one thread's accumulator row from tensor memory (thread = TMEM lane = GEMM row) and store it:
// shared by the TMA convolution kernels.
#pragma once
#include "conv_common.cuh"
#include "umma_ptx.cuh"

namespace dr {
using namespace ptx;

// Drain `ncols` accumulator columns of this thread's TMEM lane and run the direct epilogue.
__device__ __forceinline__ void drain_direct(const ConvParams& p, uint32_t taddr, int ncols, long long m, bool row_ok, int n0) {
    for (int c = 0; c < ncols; c += 32) {
        uint32_t r[32];
        if (ncols - c >= 32) {
            tmem_ld_x32(taddr + c, r);
            tmem_ld_wait();
            if (row_ok) epilogue_direct<32>(p, m, n0 + c, reinterpret_cast<float*>(r));
        } else {
            tmem_ld_x16(taddr + c, r);
            tmem_ld_wait();
            if (row_ok) epilogue_direct<16>(p, m, n0 + c, reinterpret_cast<float*>(r));
        }
    }
}

// Lean epilogue of the common case (bias and/or ReLU only, bf16 out, Cout a multiple of 16, aligned
// slice): bias comes from a shared-memory copy as float4, the ReLU choice is a template argument, and
// a thread stores its 64 bytes per 32-column chunk with four 16-byte stores.
// MODE 0: +bias;  1: +bias, ReLU;  2: +bias, +residual;  3: +bias, +residual, ReLU.
template <int MODE>
__device__ __forceinline__ void drain_fast(const ConvParams& p, uint32_t taddr, int ncols, long long m, bool row_ok, int n0,
                                           const float* bias_s) {
    constexpr bool RELU = (MODE & 1) != 0, RES = (MODE & 2) != 0;
    uint4* y = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.y) + m * p.ldc + p.coff + n0);
    const uint4* res = reinterpret_cast<const uint4*>(p.residual + (RES && row_ok ? m * p.Cout + n0 : 0));
    const float4* b4 = reinterpret_cast<const float4*>(bias_s + n0);
    int c = 0;
    for (; c + 32 <= ncols; c += 32) {
        uint32_t r[32];
        tmem_ld_x32(taddr + c, r);
        tmem_ld_wait();
        uint32_t o[16];
        uint32_t rr[16];
        if (RES && row_ok) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint4 u = __ldg(res + (c >> 3) + q);
                rr[4 * q] = u.x; rr[4 * q + 1] = u.y; rr[4 * q + 2] = u.z; rr[4 * q + 3] = u.w;
            }
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 b = b4[(c >> 2) + q];
            float v0 = __uint_as_float(r[4 * q]) + b.x, v1 = __uint_as_float(r[4 * q + 1]) + b.y;
            float v2 = __uint_as_float(r[4 * q + 2]) + b.z, v3 = __uint_as_float(r[4 * q + 3]) + b.w;
            if (RES && row_ok) { v0 += bf16_lo(rr[2 * q]); v1 += bf16_hi(rr[2 * q]); v2 += bf16_lo(rr[2 * q + 1]); v3 += bf16_hi(rr[2 * q + 1]); }
            if (RELU) { v0 = fmaxf(v0, 0.f); v1 = fmaxf(v1, 0.f); v2 = fmaxf(v2, 0.f); v3 = fmaxf(v3, 0.f); }
            o[2 * q] = pack_bf16(v0, v1);
            o[2 * q + 1] = pack_bf16(v2, v3);
        }
        if (row_ok) {
#pragma unroll
            for (int q = 0; q < 4; ++q) y[(c >> 3) + q] = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
        }
    }
    if (c < ncols) {   // 16-column tail
        uint32_t r[16];
        tmem_ld_x16(taddr + c, r);
        tmem_ld_wait();
        uint32_t o[8];
        uint32_t rr[8];
        if (RES && row_ok) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const uint4 u = __ldg(res + (c >> 3) + q);
                rr[4 * q] = u.x; rr[4 * q + 1] = u.y; rr[4 * q + 2] = u.z; rr[4 * q + 3] = u.w;
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 b = b4[(c >> 2) + q];
            float v0 = __uint_as_float(r[4 * q]) + b.x, v1 = __uint_as_float(r[4 * q + 1]) + b.y;
            float v2 = __uint_as_float(r[4 * q + 2]) + b.z, v3 = __uint_as_float(r[4 * q + 3]) + b.w;
            if (RES && row_ok) { v0 += bf16_lo(rr[2 * q]); v1 += bf16_hi(rr[2 * q]); v2 += bf16_lo(rr[2 * q + 1]); v3 += bf16_hi(rr[2 * q + 1]); }
            if (RELU) { v0 = fmaxf(v0, 0.f); v1 = fmaxf(v1, 0.f); v2 = fmaxf(v2, 0.f); v3 = fmaxf(v3, 0.f); }
            o[2 * q] = pack_bf16(v0, v1);
            o[2 * q + 1] = pack_bf16(v2, v3);
        }
        if (row_ok) {
            y[(c >> 3)] = make_uint4(o[0], o[1], o[2], o[3]);
            y[(c >> 3) + 1] = make_uint4(o[4], o[5], o[6], o[7]);
        }
    }
}

}  // namespace dr
