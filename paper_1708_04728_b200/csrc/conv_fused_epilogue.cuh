// Fused pooling / LRN epilogue of the patch-tiled convolution kernels (conv_patch.cu).
//
// A tile is a (2*PH+1) x (2*PW+1) patch of convolution outputs (GEMM row = i*(2*PW+1) + j) whose
// accumulators sit in tensor memory, one row per TMEM lane.  Four warps (thread = row) drain them:
//   LRN first (ReLU -> LRN -> pool):  the thread owns all channels of its pixel, so the LRN window is a
//       register sliding window over 32-column TMEM chunks; the result goes to shared memory as
//       bf16 (max-pooling commutes with the monotone bf16 rounding, so rounding before the max gives
//       the same stored value as rounding after it), then 3x3/2 max over rows.
//   pool first (ReLU -> pool [-> LRN]): the raw float32 accumulators are staged and the 3x3/2 max is
//       taken on them; bias and ReLU are applied to the pooled values only (adding a per-channel
//       constant and clamping are monotone, so they commute with the max: 4-5x fewer evaluations),
//       then LRN (if any) on the pooled float32 values, then the single bf16 rounding.
// Rows of the patch that fall outside the convolution plane are staged as -inf, so the max needs no
// masks ("padding never wins"; every window holds at least one real pixel).
//
// LRN scale s^(-beta), s = k + (alpha/n) * sum x^2: when the normalised excess u = (s-k)/k is below
// 1/32 for a whole 32-channel chunk of the warp, (1+u)^(-beta) is evaluated by its binomial series
// to the u^4 term (truncation error < 2e-8 relative, below float32 resolution); otherwise the chunk
// takes the exp2/log2 route.  The special-function unit would otherwise bound the layer.
#pragma once
#include "conv_common.cuh"
#include "umma_ptx.cuh"

namespace dr {

constexpr int FE_THREADS = 128;          // epilogue threads (4 warps)

__device__ __forceinline__ void fe_bar(int id) { asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(FE_THREADS) : "memory"); }

__host__ __device__ inline bool fe_lrn_first(const ConvParams& p) { return (p.flags & DR_LRN) && (p.flags & DR_LRN_BEFORE_POOL); }
// bytes of one staged row: bf16 after LRN-first, float32 raw accumulators otherwise (+16 B: 16-byte
// row-wise stores of a warp then fall on distinct banks)
// With the positions of the maxima asked for (argmax), every staged value is float32: the decision is taken on the
// unrounded values, as the layer sequence the slim layer stands for would take it.
__host__ __device__ inline int fe_stage_pitch(const ConvParams& p) { return (fe_lrn_first(p) && !p.argmax) ? (p.Cout * 2 + 16) : (p.Cout * 4 + 16); }
__host__ __device__ inline int fe_smem_bytes(const ConvParams& p) {
    int b = TILE_M * fe_stage_pitch(p) + 256 * 4;                       // stage + bias copy
    if ((p.flags & DR_LRN) && !fe_lrn_first(p)) b += p.PH * p.PW * (p.Cout + 8) * 4;   // pooled float32 values, 4 floats of halo each side
    return (b + 1023) & ~1023;
}
inline bool fe_supports(const ConvParams& p) {
    if (!(p.flags & DR_POOL)) return false;                      // LRN-only layers: the TMA / gather kernels
    if (p.Cout % 32 || p.Cout > 256) return false;
    if ((p.flags & DR_LRN) && (p.lrn_half != 2 || p.lrn_k <= 0.f || p.lrn_alpha_n < 0.f)) return false;
    if (p.flags & (DR_RESIDUAL | DR_OUT_F32)) return false;
    if ((p.ldc & 7) || (p.coff & 7)) return false;
    return true;
}
// the kernels call this once (all threads) before the first tile
__device__ __forceinline__ void fe_init(const ConvParams& p, uint8_t* stage, int tid, int nthreads) {
    float* bias_s = reinterpret_cast<float*>(stage + TILE_M * fe_stage_pitch(p));
    for (int i = tid; i < 256; i += nthreads) bias_s[i] = ((p.flags & DR_BIAS) && i < p.Cout) ? p.bias[i] : 0.f;
}

// LRN scale factors for N window sums at once; the series/exact choice is uniform over the warp.
template <int N>
__device__ __forceinline__ void fe_lrn_scale(const ConvParams& p, const float* ss, float* scale) {
    float smax = 0.f;
#pragma unroll
    for (int j = 0; j < N; ++j) smax = fmaxf(smax, ss[j]);
    if (__all_sync(0xffffffffu, smax < p.lrn_ss_max2)) {     // series in ss, k^(-beta) folded into the coefficients; two terms suffice
#pragma unroll
        for (int j = 0; j < N; ++j) scale[j] = fmaf(ss[j], fmaf(ss[j], p.lrn_s2, p.lrn_s1), p.lrn_kpow);
    } else if (__all_sync(0xffffffffu, smax < p.lrn_ss_max)) {
#pragma unroll
        for (int j = 0; j < N; ++j) scale[j] = fmaf(ss[j], fmaf(ss[j], fmaf(ss[j], fmaf(ss[j], p.lrn_s4, p.lrn_s3), p.lrn_s2), p.lrn_s1), p.lrn_kpow);
    } else {
#pragma unroll
        for (int j = 0; j < N; ++j) scale[j] = __powf(fmaf(p.lrn_alpha_n, ss[j], p.lrn_k), -p.lrn_beta);
    }
}

// 32 accumulator columns starting at column c (+ bias, ReLU) into x; zeros when the chunk lies past the last channel.
__device__ __forceinline__ void fe_load_chunk(uint32_t taddr, const float* bias_s, int c, bool present, bool relu, float* x) {
    if (present) {
        uint32_t r[32];
        ptx::tmem_ld_x32(taddr + c, r);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 b4 = *reinterpret_cast<const float4*>(bias_s + c + 4 * q);
            const float bb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float v = __uint_as_float(r[4 * q + k]) + bb[k];
                x[4 * q + k] = relu ? fmaxf(v, 0.f) : v;
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) x[j] = 0.f;
    }
}

// The registers of a TMEM load that has just been waited for, passed through an empty volatile statement: what reads them
// stays behind the wait in program order.
__device__ __forceinline__ void fe_pin32(uint32_t* r) {
#pragma unroll
    for (int j = 0; j < 32; j += 8)
        asm volatile("" : "+r"(r[j]), "+r"(r[j + 1]), "+r"(r[j + 2]), "+r"(r[j + 3]), "+r"(r[j + 4]), "+r"(r[j + 5]), "+r"(r[j + 6]), "+r"(r[j + 7]));
}
// raw accumulators of 32 columns starting at channel c -> + bias, ReLU
__device__ __forceinline__ void fe_convert_chunk(const uint32_t* r, const float* bias_s, int c, bool relu, float* x) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const float4 b4 = *reinterpret_cast<const float4*>(bias_s + c + 4 * q);
        const float bb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float v = __uint_as_float(r[4 * q + k]) + bb[k];
            x[4 * q + k] = relu ? fmaxf(v, 0.f) : v;
        }
    }
}

// LRN (window of five) of the 32 channels in cur, given the two channels before (pm2, pm1) and the chunk after;
// the result goes to dst as bfloat16 (-inf for rows outside the convolution plane).  The window sum slides:
// ss[j] = ss[j-1] + x[j+2]^2 - x[j-3]^2, restarted from its five terms every 8 channels (a sum that cancels to a few
// ulps below zero is harmless: the scale is k + (alpha/n) ss with k > 0).  The scale is the series in ss with k^(-beta)
// folded in while the sum of all squares of the warp's chunk is below lrn_ss_max; exp2/log2 otherwise.
template <bool F32OUT>
__device__ __forceinline__ void fe_lrn_chunk(const ConvParams& p, const float* cur, const float* nxt, float& pm2, float& pm1, uint8_t* dst,
                                             bool valid) {
    float sq[36];                                  // squares of x[c0-2 .. c0+33]
    sq[0] = pm2 * pm2; sq[1] = pm1 * pm1;
#pragma unroll
    for (int j = 0; j < 32; ++j) sq[2 + j] = cur[j] * cur[j];
    sq[34] = nxt[0] * nxt[0]; sq[35] = nxt[1] * nxt[1];
    float ss[32], sc[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if ((j & 7) == 0) ss[j] = (sq[j] + sq[j + 1]) + (sq[j + 2] + sq[j + 3]) + sq[j + 4];
        else ss[j] = (ss[j - 1] - sq[j - 1]) + sq[j + 4];
    }
    // every window sum is at most the sum of all squares = seven disjoint windows + the last square
    const float total = ((ss[0] + ss[5]) + (ss[10] + ss[15])) + ((ss[20] + ss[25]) + (ss[30] + sq[35]));
    if (__all_sync(0xffffffffu, total < p.lrn_ss_max2)) {   // the usual case (alpha = 1e-4): two terms are exact to float32 resolution
#pragma unroll
        for (int j = 0; j < 32; ++j) sc[j] = fmaf(ss[j], fmaf(ss[j], p.lrn_s2, p.lrn_s1), p.lrn_kpow);
    } else if (__all_sync(0xffffffffu, total < p.lrn_ss_max)) {
#pragma unroll
        for (int j = 0; j < 32; ++j) sc[j] = fmaf(ss[j], fmaf(ss[j], fmaf(ss[j], fmaf(ss[j], p.lrn_s4, p.lrn_s3), p.lrn_s2), p.lrn_s1), p.lrn_kpow);
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) sc[j] = __powf(fmaf(p.lrn_alpha_n, ss[j], p.lrn_k), -p.lrn_beta);
    }
    if (F32OUT) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            float4 v;
            if (valid) v = make_float4(cur[4 * q] * sc[4 * q], cur[4 * q + 1] * sc[4 * q + 1], cur[4 * q + 2] * sc[4 * q + 2], cur[4 * q + 3] * sc[4 * q + 3]);
            else v.x = v.y = v.z = v.w = __uint_as_float(0xff800000u);
            *reinterpret_cast<float4*>(dst + 16 * q) = v;
        }
        pm2 = cur[30];
        pm1 = cur[31];
        return;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint4 v;
        if (valid) {
            v.x = pack_bf16(cur[8 * q + 0] * sc[8 * q + 0], cur[8 * q + 1] * sc[8 * q + 1]);
            v.y = pack_bf16(cur[8 * q + 2] * sc[8 * q + 2], cur[8 * q + 3] * sc[8 * q + 3]);
            v.z = pack_bf16(cur[8 * q + 4] * sc[8 * q + 4], cur[8 * q + 5] * sc[8 * q + 5]);
            v.w = pack_bf16(cur[8 * q + 6] * sc[8 * q + 6], cur[8 * q + 7] * sc[8 * q + 7]);
        } else {
            v.x = v.y = v.z = v.w = 0xFF80FF80u;     // -inf, -inf
        }
        *reinterpret_cast<uint4*>(dst + 16 * q) = v;
    }
    pm2 = cur[30];
    pm1 = cur[31];
}

// taddr: TMEM address of this thread's lane, column 0 of the accumulator.  row = 0..127.
// Called by the 4 warps of one epilogue group together (a kernel may run two groups on alternate tiles,
// each with its own stage buffer and named barrier); `release` is invoked by each warp once its TMEM
// reads are done.
// PREFETCH (kernels that give the epilogue warps registers for it): the TMEM load of the next 32-channel chunk is in
// flight while the LRN of the current one is computed.
template <bool PREFETCH, class Release>
__device__ __forceinline__ void fused_epilogue(const ConvParams& p, int tile, uint32_t taddr, uint8_t* stage, int row, int bar_id,
                                               Release release) {
    const int C = p.Cout;
    const bool lrn = p.flags & DR_LRN;
    const bool lrn_first = fe_lrn_first(p);
    const bool relu = p.flags & DR_RELU;
    const bool am = p.argmax != nullptr;
    const int pitch = fe_stage_pitch(p);
    const float* bias_s = reinterpret_cast<const float*>(stage + TILE_M * pitch);
    const int pwc = 2 * p.PW + 1, phc = 2 * p.PH + 1;
    const int per = p.tiles_h * p.tiles_w;
    const int n = tile / per, t = tile - n * per;
    const int th = t / p.tiles_w, tw = t - th * p.tiles_w;
    const int pi = row / pwc, pj = row - pi * pwc;
    const int ho = 2 * th * p.PH - 1 + pi, wo = 2 * tw * p.PW - 1 + pj;
    const bool valid = pi < phc && ho >= 0 && ho < p.Ho && wo >= 0 && wo < p.Wo;
    uint8_t* srow = stage + (size_t)row * pitch;

    // ---- drain TMEM (+ bias, ReLU, LRN when LRN comes first), stage
    if (lrn_first && PREFETCH && !am) {
        // as below, with the raw accumulators of the chunk after the next one requested before the LRN of the current one
        float xa[32], xb[32];
        uint32_t raw[32];
        float pm2 = 0.f, pm1 = 0.f;
        fe_load_chunk(taddr, bias_s, 0, true, relu, xa);
        if (32 < C) ptx::tmem_ld_x32(taddr + 32, raw);
        for (int c0 = 0; c0 < C; c0 += 64) {
            const bool has_b = c0 + 32 < C;
            if (has_b) { ptx::tmem_ld_wait(); fe_pin32(raw); fe_convert_chunk(raw, bias_s, c0 + 32, relu, xb); }
            else {
#pragma unroll
                for (int j = 0; j < 32; ++j) xb[j] = 0.f;
            }
            if (c0 + 64 < C) ptx::tmem_ld_x32(taddr + c0 + 64, raw);
            fe_lrn_chunk<false>(p, xa, xb, pm2, pm1, srow + c0 * 2, valid);
            if (has_b) {
                const bool has_a = c0 + 64 < C;
                if (has_a) { ptx::tmem_ld_wait(); fe_pin32(raw); fe_convert_chunk(raw, bias_s, c0 + 64, relu, xa); }
                else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) xa[j] = 0.f;
                }
                if (c0 + 96 < C) ptx::tmem_ld_x32(taddr + c0 + 96, raw);
                fe_lrn_chunk<false>(p, xb, xa, pm2, pm1, srow + (c0 + 32) * 2, valid);
            }
        }
    } else if (lrn_first) {
        // two register chunks used alternately as "current" and "next" (no copy between them)
        float xa[32], xb[32];
        float pm2 = 0.f, pm1 = 0.f;                      // x[c-2], x[c-1] of the chunk before
        fe_load_chunk(taddr, bias_s, 0, true, relu, xa);
        for (int c0 = 0; c0 < C; c0 += 64) {
            fe_load_chunk(taddr, bias_s, c0 + 32, c0 + 32 < C, relu, xb);
            if (am) fe_lrn_chunk<true>(p, xa, xb, pm2, pm1, srow + c0 * 4, valid);
            else fe_lrn_chunk<false>(p, xa, xb, pm2, pm1, srow + c0 * 2, valid);
            if (c0 + 32 < C) {
                fe_load_chunk(taddr, bias_s, c0 + 64, c0 + 64 < C, relu, xa);
                if (am) fe_lrn_chunk<true>(p, xb, xa, pm2, pm1, srow + (c0 + 32) * 4, valid);
                else fe_lrn_chunk<false>(p, xb, xa, pm2, pm1, srow + (c0 + 32) * 2, valid);
            }
        }
    } else {
        for (int c0 = 0; c0 < C; c0 += 32) {
            uint32_t r[32];
            ptx::tmem_ld_x32(taddr + c0, r);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                uint4 v = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
                if (!valid) v.x = v.y = v.z = v.w = 0xff800000u;   // -inf
                *reinterpret_cast<uint4*>(srow + (c0 + 4 * q) * 4) = v;
            }
        }
    }
    ptx::tc_fence_before();
    release();                                            // this warp no longer needs the accumulator
    fe_bar(bar_id);

    // ---- 3x3 / 2 max over the staged patch
    __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(p.y);
    const int npp = p.PH * p.PW;
    if (am) {
        // Positions wanted: the maximum is taken on float32 values that have been through everything the layer applies
        // before pooling (bias and ReLU here if LRN did not come first), window positions in row-major order, a later one
        // wins only if strictly greater: the first maximum, as the pooling layer defines it.  Rows outside the
        // convolution plane hold -inf and never win; the first window position inside the plane always does over them.
        float* pooled = reinterpret_cast<float*>(stage + (size_t)TILE_M * pitch + 256 * 4);
        const int ldp = C + 8;
        const bool lrn_after = lrn && !lrn_first;
        const float NEG = __uint_as_float(0xff800000u);
        const int C4 = C >> 2;
        for (int item = row; item < npp * C4; item += FE_THREADS) {
            const int pp = item / C4, c = (item - pp * C4) << 2;
            const int ppi = pp / p.PW, ppj = pp - ppi * p.PW;
            const int ph = th * p.PH + ppi, pw = tw * p.PW + ppj;
            const uint8_t* base = stage + (size_t)((2 * ppi) * pwc + 2 * ppj) * pitch + c * 4;
            const float4 b4 = *reinterpret_cast<const float4*>(bias_s + c);
            float m[4] = {NEG, NEG, NEG, NEG};
            int w[4] = {-1, -1, -1, -1};
#pragma unroll
            for (int d = 0; d < 9; ++d) {
                const float4 u = *reinterpret_cast<const float4*>(base + (size_t)((d / 3) * pwc + (d % 3)) * pitch);
                float v[4] = {u.x, u.y, u.z, u.w};
                const int hh = 2 * ph - 1 + d / 3, ww = 2 * pw - 1 + d % 3;
                const int pos = hh * p.Wo + ww;
                if (!lrn_first) {
                    const float bb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (v[k] != NEG) { v[k] += bb[k]; if (relu) v[k] = fmaxf(v[k], 0.f); }
                }
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (v[k] > m[k]) { m[k] = v[k]; w[k] = pos; }
            }
            if (lrn_after) {
                *reinterpret_cast<float4*>(pooled + pp * ldp + 4 + c) = make_float4(m[0], m[1], m[2], m[3]);
                if (c == 0) { pooled[pp * ldp + 2] = 0.f; pooled[pp * ldp + 3] = 0.f; pooled[pp * ldp + C + 4] = 0.f; pooled[pp * ldp + C + 5] = 0.f; }
            }
            if (ph < p.Hy && pw < p.Wy) {
                const long long q = ((long long)n * p.Hy + ph) * p.Wy + pw;
                *reinterpret_cast<int4*>(p.argmax + q * C + c) = make_int4(w[0], w[1], w[2], w[3]);
                if (!lrn_after) {
                    uint2 o;
                    o.x = pack_bf16(m[0], m[1]); o.y = pack_bf16(m[2], m[3]);
                    *reinterpret_cast<uint2*>(y + q * p.ldc + p.coff + c) = o;
                }
            }
        }
        if (lrn_after) {
            fe_bar(bar_id);
            for (int item = row; item < ((npp * C + FE_THREADS - 1) / FE_THREADS) * FE_THREADS; item += FE_THREADS) {
                const bool active = item < npp * C;
                const int it2 = active ? item : npp * C - 1;
                const int pp = it2 / C, c = it2 - pp * C;
                const int ppi = pp / p.PW, ppj = pp - ppi * p.PW;
                const int ph = th * p.PH + ppi, pw = tw * p.PW + ppj;
                const float* s5 = pooled + pp * ldp + 4 + c;               // two zeros of halo on either side of the row
                float ss[1] = {(s5[-2] * s5[-2] + s5[-1] * s5[-1]) + (s5[0] * s5[0] + s5[1] * s5[1]) + s5[2] * s5[2]}, sc[1];
                fe_lrn_scale<1>(p, ss, sc);
                if (active && ph < p.Hy && pw < p.Wy) {
                    const long long q = ((long long)n * p.Hy + ph) * p.Wy + pw;
                    y[q * p.ldc + p.coff + c] = __float2bfloat16_rn(s5[0] * sc[0]);
                }
            }
        }
    } else if (lrn_first) {
        const int C8 = C >> 3;
        const int dpp = FE_THREADS / C8, dc8 = FE_THREADS - dpp * C8;      // step of the (pp, c8) item index per pass
        int pp = row / C8, c8 = row - pp * C8;
        while (pp < npp) {
            const int ppi = pp / p.PW, ppj = pp - ppi * p.PW;
            const int ph = th * p.PH + ppi, pw = tw * p.PW + ppj;
            if (ph < p.Hy && pw < p.Wy) {
                const uint8_t* base = stage + (size_t)((2 * ppi) * pwc + 2 * ppj) * pitch + c8 * 16;
                uint4 m = *reinterpret_cast<const uint4*>(base);
                __nv_bfloat162* mm = reinterpret_cast<__nv_bfloat162*>(&m);
#pragma unroll
                for (int d = 1; d < 9; ++d) {
                    const uint4 u = *reinterpret_cast<const uint4*>(base + (size_t)((d / 3) * pwc + (d % 3)) * pitch);
                    const __nv_bfloat162* uu = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
                    for (int k = 0; k < 4; ++k) mm[k] = __hmax2(mm[k], uu[k]);
                }
                const long long q = ((long long)n * p.Hy + ph) * p.Wy + pw;
                *reinterpret_cast<uint4*>(y + q * p.ldc + p.coff + c8 * 8) = m;
            }
            pp += dpp; c8 += dc8;
            if (c8 >= C8) { c8 -= C8; ++pp; }
        }
    } else {
        float* pooled = reinterpret_cast<float*>(stage + (size_t)TILE_M * pitch + 256 * 4);   // [pp][4 halo | C | 4 halo]
        const int ldp = C + 8;
        const int C4 = C >> 2;
        const int dpp = FE_THREADS / C4, dc4 = FE_THREADS - dpp * C4;
        int pp = row / C4, c4 = row - pp * C4;
        while (pp < npp) {
            const int ppi = pp / p.PW, ppj = pp - ppi * p.PW;
            const int ph = th * p.PH + ppi, pw = tw * p.PW + ppj;
            const int c = c4 << 2;
            const uint8_t* base = stage + (size_t)((2 * ppi) * pwc + 2 * ppj) * pitch + c * 4;
            float4 m = *reinterpret_cast<const float4*>(base);
#pragma unroll
            for (int d = 1; d < 9; ++d) {
                const float4 u = *reinterpret_cast<const float4*>(base + (size_t)((d / 3) * pwc + (d % 3)) * pitch);
                m.x = fmaxf(m.x, u.x); m.y = fmaxf(m.y, u.y); m.z = fmaxf(m.z, u.z); m.w = fmaxf(m.w, u.w);
            }
            const float4 b4 = *reinterpret_cast<const float4*>(bias_s + c);
            m.x += b4.x; m.y += b4.y; m.z += b4.z; m.w += b4.w;
            if (relu) { m.x = fmaxf(m.x, 0.f); m.y = fmaxf(m.y, 0.f); m.z = fmaxf(m.z, 0.f); m.w = fmaxf(m.w, 0.f); }
            if (lrn) {
                *reinterpret_cast<float4*>(pooled + pp * ldp + 4 + c) = m;
                if (c == 0) { pooled[pp * ldp + 2] = 0.f; pooled[pp * ldp + 3] = 0.f; pooled[pp * ldp + C + 4] = 0.f; pooled[pp * ldp + C + 5] = 0.f; }
            } else if (ph < p.Hy && pw < p.Wy) {
                const long long q = ((long long)n * p.Hy + ph) * p.Wy + pw;
                uint2 o;
                o.x = pack_bf16(m.x, m.y); o.y = pack_bf16(m.z, m.w);
                *reinterpret_cast<uint2*>(y + q * p.ldc + p.coff + c) = o;
            }
            pp += dpp; c4 += dc4;
            if (c4 >= C4) { c4 -= C4; ++pp; }
        }
        if (lrn) {
            fe_bar(bar_id);
            // LRN on the pooled float32 values, 8 channels per thread
            const int C8 = C >> 3;
            const int dpp8 = FE_THREADS / C8, dc8 = FE_THREADS - dpp8 * C8;
            int pq = row / C8, c8 = row - pq * C8;
            const int iters = (npp * C8 + FE_THREADS - 1) / FE_THREADS;   // same trip count for every lane: the
            for (int itn = 0; itn < iters; ++itn) {                         // series/exact vote below is warp-wide
                const bool active = pq < npp;
                const int pr = active ? pq : npp - 1;
                const int ppi = pr / p.PW, ppj = pr - ppi * p.PW;
                const int ph = th * p.PH + ppi, pw = tw * p.PW + ppj;
                const float4* s4 = reinterpret_cast<const float4*>(pooled + pr * ldp + (c8 << 3));   // x[c-4 .. c+11]
                float w16[16];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float4 f = s4[j];
                    w16[4 * j] = f.x; w16[4 * j + 1] = f.y; w16[4 * j + 2] = f.z; w16[4 * j + 3] = f.w;
                }
                float v[12], sq[12], ss[8], sc[8];
#pragma unroll
                for (int j = 0; j < 12; ++j) { v[j] = w16[j + 2]; sq[j] = v[j] * v[j]; }          // v[0] = x[c-2]
#pragma unroll
                for (int j = 0; j < 8; ++j) ss[j] = (sq[j] + sq[j + 1]) + (sq[j + 2] + sq[j + 3]) + sq[j + 4];
                fe_lrn_scale<8>(p, ss, sc);
                if (active && ph < p.Hy && pw < p.Wy) {
                    uint4 u;
                    u.x = pack_bf16(v[2] * sc[0], v[3] * sc[1]); u.y = pack_bf16(v[4] * sc[2], v[5] * sc[3]);
                    u.z = pack_bf16(v[6] * sc[4], v[7] * sc[5]); u.w = pack_bf16(v[8] * sc[6], v[9] * sc[7]);
                    const long long q = ((long long)n * p.Hy + ph) * p.Wy + pw;
                    *reinterpret_cast<uint4*>(y + q * p.ldc + p.coff + (c8 << 3)) = u;
                }
                pq += dpp8; c8 += dc8;
                if (c8 >= C8) { c8 -= C8; ++pq; }
            }
        }
    }
    fe_bar(bar_id);                                       // the stage may be overwritten by the next tile
}

// fe_lrn_chunk for threads with few registers (bfloat16 output only): the bound that selects the series is the sum of
// all 36 squares (every window sum is at most that), so no window sum has to be kept; sums and scales are consumed
// eight channels at a time.
__device__ __forceinline__ void fe_lrn_chunk_lean(const ConvParams& p, const float* cur, const float* nxt, float& pm2, float& pm1, uint8_t* dst,
                                                  bool valid) {
    float total = fmaf(pm2, pm2, pm1 * pm1);
#pragma unroll
    for (int j = 0; j < 32; ++j) total = fmaf(cur[j], cur[j], total);
    total = fmaf(nxt[0], nxt[0], fmaf(nxt[1], nxt[1], total));
    const int mode = __all_sync(0xffffffffu, total < p.lrn_ss_max2) ? 0 : (__all_sync(0xffffffffu, total < p.lrn_ss_max) ? 1 : 2);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        float x[12];                               // channels 8q-2 .. 8q+9 of the chunk
#pragma unroll
        for (int j = 0; j < 12; ++j) {
            const int c = 8 * q - 2 + j;
            x[j] = c == -2 ? pm2 : c == -1 ? pm1 : c < 32 ? cur[c < 0 ? 0 : (c > 31 ? 31 : c)] : nxt[c - 32 > 1 ? 1 : c - 32];
        }
        float sq[12], ss[8], sc[8];
#pragma unroll
        for (int j = 0; j < 12; ++j) sq[j] = x[j] * x[j];
        ss[0] = (sq[0] + sq[1]) + (sq[2] + sq[3]) + sq[4];
#pragma unroll
        for (int j = 1; j < 8; ++j) ss[j] = (ss[j - 1] - sq[j - 1]) + sq[j + 4];
        if (mode == 0) {
#pragma unroll
            for (int j = 0; j < 8; ++j) sc[j] = fmaf(ss[j], fmaf(ss[j], p.lrn_s2, p.lrn_s1), p.lrn_kpow);
        } else if (mode == 1) {
#pragma unroll
            for (int j = 0; j < 8; ++j) sc[j] = fmaf(ss[j], fmaf(ss[j], fmaf(ss[j], fmaf(ss[j], p.lrn_s4, p.lrn_s3), p.lrn_s2), p.lrn_s1), p.lrn_kpow);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) sc[j] = __powf(fmaf(p.lrn_alpha_n, ss[j], p.lrn_k), -p.lrn_beta);
        }
        uint4 v;
        if (valid) {
            v.x = pack_bf16(x[2] * sc[0], x[3] * sc[1]);
            v.y = pack_bf16(x[4] * sc[2], x[5] * sc[3]);
            v.z = pack_bf16(x[6] * sc[4], x[7] * sc[5]);
            v.w = pack_bf16(x[8] * sc[6], x[9] * sc[7]);
        } else {
            v.x = v.y = v.z = v.w = 0xFF80FF80u;     // -inf, -inf
        }
        *reinterpret_cast<uint4*>(dst + 16 * q) = v;
    }
    pm2 = cur[30];
    pm1 = cur[31];
}

// The LRN-first epilogue (ReLU -> LRN -> pool, no positions) run by TWO groups of four warps on one tile: part 0 takes
// channels [0, C/2), part 1 [C/2, C) of every row (C a multiple of 64), each with the two channels beyond its range
// that the window of five needs; both parts pool and store together (256 threads).  A tile's accumulator is then
// held half as long, which is what bounds a layer whose drain (the LRN arithmetic) takes longer than its MMAs.
// `row` = 0..127 within the part; the named barrier `bar_id` is shared by the 256 threads.
constexpr int FE_SPLIT_THREADS = 2 * FE_THREADS;
__device__ __forceinline__ void fe_bar_split(int id) { asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(FE_SPLIT_THREADS) : "memory"); }
inline bool fe_split_supports(const ConvParams& p) { return fe_supports(p) && fe_lrn_first(p) && !p.argmax && p.Cout % 64 == 0; }

template <class Release>
__device__ __forceinline__ void fused_epilogue_split(const ConvParams& p, int tile, uint32_t taddr, uint8_t* stage, int row, int part, int bar_id,
                                                     Release release) {
    const int C = p.Cout, H = C >> 1;
    const bool relu = p.flags & DR_RELU;
    const int pitch = fe_stage_pitch(p);
    const float* bias_s = reinterpret_cast<const float*>(stage + TILE_M * pitch);
    const int pwc = 2 * p.PW + 1, phc = 2 * p.PH + 1;
    const int per = p.tiles_h * p.tiles_w;
    const int n = tile / per, t = tile - n * per;
    const int th = t / p.tiles_w, tw = t - th * p.tiles_w;
    const int pi = row / pwc, pj = row - pi * pwc;
    const int ho = 2 * th * p.PH - 1 + pi, wo = 2 * tw * p.PW - 1 + pj;
    const bool valid = pi < phc && ho >= 0 && ho < p.Ho && wo >= 0 && wo < p.Wo;
    uint8_t* srow = stage + (size_t)row * pitch;
    const int c_lo = part * H, c_hi = c_lo + H;

    // ---- drain this part's channels: + bias, ReLU, LRN, stage as bf16.  One 32-channel chunk is live at a time; the
    // two channels after it come from a two-column load of their own (tensor-memory loads are cheap, registers are not).
    float pm2 = 0.f, pm1 = 0.f;
    if (part) {                                            // channels c_lo-2, c_lo-1: the last two of the 16 columns before c_lo
        uint32_t r[16];
        ptx::tmem_ld_x16(taddr + c_lo - 16, r);
        ptx::tmem_ld_wait();
        const float v2 = __uint_as_float(r[14]) + bias_s[c_lo - 2], v1 = __uint_as_float(r[15]) + bias_s[c_lo - 1];
        pm2 = relu ? fmaxf(v2, 0.f) : v2;
        pm1 = relu ? fmaxf(v1, 0.f) : v1;
    }
    for (int c0 = c_lo; c0 < c_hi; c0 += 32) {
        uint32_t r[32], r2[2] = {0u, 0u};
        const bool more = c0 + 32 < C;
        ptx::tmem_ld_x32(taddr + c0, r);
        if (more) ptx::tmem_ld_x2(taddr + c0 + 32, r2);
        ptx::tmem_ld_wait();
        fe_pin32(r);
        asm volatile("" : "+r"(r2[0]), "+r"(r2[1]));
        float x[32], nx[2];
        fe_convert_chunk(r, bias_s, c0, relu, x);
        if (more) {
            const float v0 = __uint_as_float(r2[0]) + bias_s[c0 + 32], v1 = __uint_as_float(r2[1]) + bias_s[c0 + 33];
            nx[0] = relu ? fmaxf(v0, 0.f) : v0;
            nx[1] = relu ? fmaxf(v1, 0.f) : v1;
        } else {
            nx[0] = 0.f; nx[1] = 0.f;
        }
        fe_lrn_chunk_lean(p, x, nx, pm2, pm1, srow + c0 * 2, valid);
    }
    ptx::tc_fence_before();
    release();                                            // this warp no longer needs the accumulator
    fe_bar_split(bar_id);

    // ---- 3x3 / 2 max over the staged patch, all 256 threads
    __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(p.y);
    const int npp = p.PH * p.PW;
    const int C8 = C >> 3;
    const int tix = part * FE_THREADS + row;
    const int dpp = FE_SPLIT_THREADS / C8, dc8 = FE_SPLIT_THREADS - dpp * C8;
    int pp = tix / C8, c8 = tix - pp * C8;
    while (pp < npp) {
        const int ppi = pp / p.PW, ppj = pp - ppi * p.PW;
        const int ph = th * p.PH + ppi, pw = tw * p.PW + ppj;
        if (ph < p.Hy && pw < p.Wy) {
            const uint8_t* base = stage + (size_t)((2 * ppi) * pwc + 2 * ppj) * pitch + c8 * 16;
            uint4 m = *reinterpret_cast<const uint4*>(base);
            __nv_bfloat162* mm = reinterpret_cast<__nv_bfloat162*>(&m);
#pragma unroll
            for (int d = 1; d < 9; ++d) {
                const uint4 u = *reinterpret_cast<const uint4*>(base + (size_t)((d / 3) * pwc + (d % 3)) * pitch);
                const __nv_bfloat162* uu = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
                for (int k = 0; k < 4; ++k) mm[k] = __hmax2(mm[k], uu[k]);
            }
            const long long q = ((long long)n * p.Hy + ph) * p.Wy + pw;
            *reinterpret_cast<uint4*>(y + q * p.ldc + p.coff + c8 * 8) = m;
        }
        pp += dpp; c8 += dc8;
        if (c8 >= C8) { c8 -= C8; ++pp; }
    }
    fe_bar_split(bar_id);                                 // the stage may be overwritten by the next tile
}

}  // namespace dr
