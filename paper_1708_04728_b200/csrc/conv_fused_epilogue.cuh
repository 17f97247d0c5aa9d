// Fused pooling / LRN epilogue of the patch-tiled convolution kernels (conv_patch.cu).
//
// A tile is a (2*PH+1) x (2*PW+1) patch of convolution outputs (GEMM row = i*(2*PW+1) + j) whose
// accumulators sit in tensor memory, one row per TMEM lane.  Four warps (thread = row) drain them:
//   LRN first (ReLU -> LRN -> pool):  the thread owns all channels of its pixel, so the LRN window is a
//       register sliding window over 32-column TMEM chunks; the result goes to shared memory as
//       bf16 (max-pooling commutes with the monotone bf16 rounding, so rounding before the max gives
//       the same stored value as rounding after it), then 3x3/2 max over rows.
//   pool first (ReLU -> pool [-> LRN]): ReLU'd float32 values are staged, the 3x3/2 max is taken in
//       float32, and LRN (if any) runs on the pooled float32 values before the single bf16 rounding.
// Rows of the patch that fall outside the convolution plane are staged as -inf, so the max needs no
// masks ("padding never wins"; every window holds at least one real pixel).
#pragma once
#include "conv_common.cuh"
#include "umma_ptx.cuh"

namespace dr {

constexpr int FE_THREADS = 128;          // epilogue threads (4 warps)

__device__ __forceinline__ void fe_bar(int id) { asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(FE_THREADS) : "memory"); }

// bytes of shared memory the epilogue needs for a layer
__host__ __device__ inline int fe_stage_pitch(const ConvParams& p) {
    const bool lrn_first = (p.flags & DR_LRN) && (p.flags & DR_LRN_BEFORE_POOL);
    const bool f32 = (p.flags & DR_LRN) && !lrn_first;          // pool first and LRN after: keep float32
    return f32 ? (p.Cout * 4 + 16) : (p.Cout * 2 + 16);          // +16 B: conflict-free 16-byte row-wise stores
}
__host__ __device__ inline int fe_smem_bytes(const ConvParams& p) {
    const bool lrn_first = (p.flags & DR_LRN) && (p.flags & DR_LRN_BEFORE_POOL);
    const bool f32 = (p.flags & DR_LRN) && !lrn_first;
    int b = TILE_M * fe_stage_pitch(p);
    if (f32) b += p.PH * p.PW * (p.Cout + 8) * 4;               // pooled float32 values, 4 floats of halo each side
    return (b + 1023) & ~1023;
}
inline bool fe_supports(const ConvParams& p) {
    if (!(p.flags & DR_POOL) || p.argmax) return false;          // argmax and LRN-only layers: gather kernel
    if (p.Cout % 32 || p.Cout > 256) return false;
    if ((p.flags & DR_LRN) && p.lrn_half != 2) return false;
    if (p.flags & (DR_RESIDUAL | DR_OUT_F32)) return false;
    if ((p.ldc & 7) || (p.coff & 7)) return false;
    return true;
}

__device__ __forceinline__ float fe_lrn5(float a, float b, float c, float d, float e, float alpha_n, float beta, float kappa) {
    return c * lrn_pow(kappa + alpha_n * (a * a + b * b + c * c + d * d + e * e), beta);
}

// taddr: TMEM address of this thread's lane, column 0 of the accumulator.  row = 0..127.
// Called by the 4 epilogue warps together; `release` is invoked by each warp once its TMEM reads are done.
template <class Release>
__device__ __forceinline__ void fused_epilogue(const ConvParams& p, int tile, uint32_t taddr, uint8_t* stage, int row, int bar_id,
                                               Release release) {
    const int C = p.Cout;
    const bool lrn = p.flags & DR_LRN;
    const bool lrn_first = lrn && (p.flags & DR_LRN_BEFORE_POOL);
    const bool f32 = lrn && !lrn_first;
    const int pitch = fe_stage_pitch(p);
    const int pwc = 2 * p.PW + 1, phc = 2 * p.PH + 1;
    const int per = p.tiles_h * p.tiles_w;
    const int n = tile / per, t = tile - n * per;
    const int th = t / p.tiles_w, tw = t - th * p.tiles_w;
    const int pi = row / pwc, pj = row - pi * pwc;
    const int ho = 2 * th * p.PH - 1 + pi, wo = 2 * tw * p.PW - 1 + pj;
    const bool valid = pi < phc && ho >= 0 && ho < p.Ho && wo >= 0 && wo < p.Wo;
    uint8_t* srow = stage + (size_t)row * pitch;

    // ---- drain TMEM, bias, ReLU, (LRN), stage
    if (lrn_first) {
        float cur[32], nxt[32];
        float pm2 = 0.f, pm1 = 0.f;                      // x[c-2], x[c-1] of the chunk before
        {
            uint32_t r[32];
            ptx::tmem_ld_x32(taddr, r);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                float v = __uint_as_float(r[j]) + ((p.flags & DR_BIAS) ? __ldg(p.bias + j) : 0.f);
                cur[j] = (p.flags & DR_RELU) ? fmaxf(v, 0.f) : v;
            }
        }
        for (int c0 = 0; c0 < C; c0 += 32) {
            if (c0 + 32 < C) {
                uint32_t r[32];
                ptx::tmem_ld_x32(taddr + c0 + 32, r);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float v = __uint_as_float(r[j]) + ((p.flags & DR_BIAS) ? __ldg(p.bias + c0 + 32 + j) : 0.f);
                    nxt[j] = (p.flags & DR_RELU) ? fmaxf(v, 0.f) : v;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) nxt[j] = 0.f;
            }
            float o[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float a = j >= 2 ? cur[j - 2] : (j == 0 ? pm2 : pm1);
                const float b = j >= 1 ? cur[j - 1] : pm1;
                const float d = j + 1 < 32 ? cur[j + 1] : nxt[0];
                const float e = j + 2 < 32 ? cur[j + 2] : nxt[j + 2 - 32];
                o[j] = fe_lrn5(a, b, cur[j], d, e, p.lrn_alpha_n, p.lrn_beta, p.lrn_k);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint4 v;
                if (valid) {
                    v.x = pack_bf16(o[8 * q + 0], o[8 * q + 1]); v.y = pack_bf16(o[8 * q + 2], o[8 * q + 3]);
                    v.z = pack_bf16(o[8 * q + 4], o[8 * q + 5]); v.w = pack_bf16(o[8 * q + 6], o[8 * q + 7]);
                } else {
                    v.x = v.y = v.z = v.w = 0xFF80FF80u;     // -inf, -inf
                }
                *reinterpret_cast<uint4*>(srow + (c0 + 8 * q) * 2) = v;
            }
            pm2 = cur[30];
            pm1 = cur[31];
#pragma unroll
            for (int j = 0; j < 32; ++j) cur[j] = nxt[j];
        }
    } else {
        for (int c0 = 0; c0 < C; c0 += 32) {
            uint32_t r[32];
            ptx::tmem_ld_x32(taddr + c0, r);
            ptx::tmem_ld_wait();
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                float x = __uint_as_float(r[j]) + ((p.flags & DR_BIAS) ? __ldg(p.bias + c0 + j) : 0.f);
                x = (p.flags & DR_RELU) ? fmaxf(x, 0.f) : x;
                v[j] = valid ? x : __int_as_float(0xff800000);
            }
            if (f32) {
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    *reinterpret_cast<float4*>(srow + (c0 + 4 * q) * 4) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            } else {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 u;
                    u.x = pack_bf16(v[8 * q + 0], v[8 * q + 1]); u.y = pack_bf16(v[8 * q + 2], v[8 * q + 3]);
                    u.z = pack_bf16(v[8 * q + 4], v[8 * q + 5]); u.w = pack_bf16(v[8 * q + 6], v[8 * q + 7]);
                    *reinterpret_cast<uint4*>(srow + (c0 + 8 * q) * 2) = u;
                }
            }
        }
    }
    ptx::tc_fence_before();
    release();                                            // this warp no longer needs the accumulator
    fe_bar(bar_id);

    // ---- 3x3 / 2 max over the staged patch
    __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(p.y);
    if (!f32) {
        const int C8 = C >> 3;
        for (int it = row; it < p.PH * p.PW * C8; it += FE_THREADS) {
            const int pp = it / C8, c = (it - pp * C8) << 3;
            const int ppi = pp / p.PW, ppj = pp - ppi * p.PW;
            const int ph = th * p.PH + ppi, pw = tw * p.PW + ppj;
            if (ph >= p.Hy || pw >= p.Wy) continue;
            const uint8_t* base = stage + (size_t)((2 * ppi) * pwc + 2 * ppj) * pitch + c * 2;
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
            *reinterpret_cast<uint4*>(y + q * p.ldc + p.coff + c) = m;
        }
    } else {
        float* pooled = reinterpret_cast<float*>(stage + (size_t)TILE_M * pitch);   // [pp][4 halo | C | 4 halo]
        const int ldp = C + 8;
        const int C4 = C >> 2;
        for (int it = row; it < p.PH * p.PW * C4; it += FE_THREADS) {
            const int pp = it / C4, c = (it - pp * C4) << 2;
            const int ppi = pp / p.PW, ppj = pp - ppi * p.PW;
            const uint8_t* base = stage + (size_t)((2 * ppi) * pwc + 2 * ppj) * pitch + c * 4;
            float4 m = *reinterpret_cast<const float4*>(base);
#pragma unroll
            for (int d = 1; d < 9; ++d) {
                const float4 u = *reinterpret_cast<const float4*>(base + (size_t)((d / 3) * pwc + (d % 3)) * pitch);
                m.x = fmaxf(m.x, u.x); m.y = fmaxf(m.y, u.y); m.z = fmaxf(m.z, u.z); m.w = fmaxf(m.w, u.w);
            }
            *reinterpret_cast<float4*>(pooled + pp * ldp + 4 + c) = m;
            if (c == 0) { pooled[pp * ldp + 2] = 0.f; pooled[pp * ldp + 3] = 0.f; pooled[pp * ldp + C + 4] = 0.f; pooled[pp * ldp + C + 5] = 0.f; }
        }
        fe_bar(bar_id);
        // LRN on the pooled float32 values, 8 channels per thread
        const int C8 = C >> 3;
        for (int it = row; it < p.PH * p.PW * C8; it += FE_THREADS) {
            const int pp = it / C8, c = (it - pp * C8) << 3;
            const int ppi = pp / p.PW, ppj = pp - ppi * p.PW;
            const int ph = th * p.PH + ppi, pw = tw * p.PW + ppj;
            if (ph >= p.Hy || pw >= p.Wy) continue;
            const float* s = pooled + pp * ldp + 2 + c;       // s[0] = x[c-2]
            float v[12];
#pragma unroll
            for (int j = 0; j < 12; ++j) v[j] = s[j];
            float o[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) o[j] = fe_lrn5(v[j], v[j + 1], v[j + 2], v[j + 3], v[j + 4], p.lrn_alpha_n, p.lrn_beta, p.lrn_k);
            uint4 u;
            u.x = pack_bf16(o[0], o[1]); u.y = pack_bf16(o[2], o[3]); u.z = pack_bf16(o[4], o[5]); u.w = pack_bf16(o[6], o[7]);
            const long long q = ((long long)n * p.Hy + ph) * p.Wy + pw;
            *reinterpret_cast<uint4*>(y + q * p.ldc + p.coff + c) = u;
        }
    }
    fe_bar(bar_id);                                       // the stage may be overwritten by the next tile
}

}  // namespace dr
