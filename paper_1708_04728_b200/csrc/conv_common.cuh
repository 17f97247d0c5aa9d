// Pieces shared by the convolution kernels: the launch parameter block, the mapping from
// a GEMM row of an output tile to an output pixel, and the two epilogues.
//
// GEMM view of a convolution (Eq. (tY_j = tW), Section 3.1 of the paper): M = B*Ho*Wo output
// pixels, N = Cout, K = k*k*Cin with K ordered (r, s, c) like the filter layout [Cout][k][k][Cin].
//
// Tiles.  A tile is 128 GEMM rows.  In LINEAR mode the rows are 128 consecutive output pixels in
// (n, ho, wo) order.  In PATCH mode (layers whose epilogue max-pools 3x3 / 2, pad 1) the rows are a
// (2*PH+1) x (2*PW+1) patch of convolution outputs of one image, which is exactly what a
// PH x PW tile of pooled outputs needs; the patch's first row and column are a halo that the
// neighbouring tile also computes, so pooling needs no exchange between tiles.
//
// Epilogues.  DIRECT: a thread owns consecutive channels of one output pixel and applies
// bias, ReLU, residual add, ReLU and the bf16/f32 store straight from registers.  STAGED (pooling
// and/or LRN): the tile's ReLU'd float32 values are staged in shared memory as [row][C+1], then
// LRN (window along the row) and the 3x3 max (window across rows) read it from there.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace dr {

constexpr int TILE_M = 128;

struct ConvParams {
    const __nv_bfloat16* x;
    const __nv_bfloat16* w;
    const float* bias;
    const __nv_bfloat16* residual;
    void* y;
    int32_t* argmax;
    int* status;
    int B, H, W, Cin, Cout, k, stride, pad;
    int Ho, Wo;            // convolution output plane
    int Hy, Wy;            // stored plane (pooled when DR_POOL)
    int K;                 // k*k*Cin
    unsigned flags;
    int lrn_half;
    float lrn_alpha_n, lrn_beta, lrn_k;
    float lrn_inv_k, lrn_kpow;   // 1/k and k^(-beta)
    float lrn_c1, lrn_c2, lrn_c3, lrn_c4;   // binomial series of (1+u)^(-beta)
    // the same series in the window sum ss itself, k^(-beta) folded in: scale = s0 + ss (s1 + ss (s2 + ss (s3 + ss s4))),
    // valid while ss < lrn_ss_max (u = (alpha/n) ss / k below 1/32)
    float lrn_s1, lrn_s2, lrn_s3, lrn_s4, lrn_ss_max;
    float lrn_ss_max2;     // below this (u < 1/256) the series stops after the ss^2 term: the next one is under 4e-8 relative
    int ldc, coff;
    long long M;           // B*Ho*Wo
    int Nt;                // output channels per n-block (multiple of 16, <= 256)
    int n_blocks;
    int m_tiles;
    int patch;             // 0 linear, 1 patch
    int PH, PW;            // pooled tile extent in patch mode
    int tiles_h, tiles_w;  // pooled tiles per image
    int overlap_prev;      // TMA kernel: 1 = the layer does not read what the kernel before it in the stream writes; it is
                           // launched with programmatic serialization (its CTAs fill SMs that kernel has left) and waits
                           // for that kernel only before it exits, so that whatever follows sees both complete
    int pdl_wait;          // TMA kernel: 1 = launched with programmatic serialization behind the kernel whose output it reads: its
                           // CTAs may start (barriers, tensor memory, descriptors) while that kernel's last CTAs still run, and
                           // wait for its completion before the first load of activations
    int* sk_counters;      // split-K kernel only (nullptr: not available): DR_CONV_WS_COUNTER_BYTES of zeroed tile counters
    float* sk_scratch;     // and scratch for the partial tiles
    size_t sk_scratch_bytes;
};

struct RowPix {
    int n, ho, wo;
    bool valid;            // the row is a real output pixel of the convolution
};

__device__ __forceinline__ RowPix row_pixel(const ConvParams& p, int tile, int i) {
    RowPix r;
    if (!p.patch) {
        const long long m = (long long)tile * TILE_M + i;
        r.valid = m < p.M;
        const int hw = p.Ho * p.Wo;
        r.n = (int)(m / hw);
        const int rem = (int)(m - (long long)r.n * hw);
        r.ho = rem / p.Wo;
        r.wo = rem - r.ho * p.Wo;
    } else {
        const int per = p.tiles_h * p.tiles_w;
        r.n = tile / per;
        const int t = tile - r.n * per;
        const int th = t / p.tiles_w, tw = t - th * p.tiles_w;
        const int pwc = 2 * p.PW + 1;
        const int pi = i / pwc, pj = i - pi * pwc;
        r.ho = 2 * th * p.PH - 1 + pi;
        r.wo = 2 * tw * p.PW - 1 + pj;
        r.valid = (pi < 2 * p.PH + 1) && r.ho >= 0 && r.ho < p.Ho && r.wo >= 0 && r.wo < p.Wo;
    }
    return r;
}

// ---- DIRECT epilogue: N consecutive channels [c0, c0+N) of output pixel m (linear mode) -----
// v holds the raw accumulators.  N is 4, 8, 16 or 32; c0 is a multiple of N.
template <int N>
__device__ __forceinline__ void epilogue_direct(const ConvParams& p, long long m, int c0, float* v) {
    if (c0 >= p.Cout) return;
    const bool full = (c0 + N <= p.Cout);
    if (p.flags & DR_BIAS) {
#pragma unroll
        for (int j = 0; j < N; ++j) v[j] += (full || c0 + j < p.Cout) ? __ldg(p.bias + c0 + j) : 0.f;
    }
    if (p.flags & DR_RELU) {
#pragma unroll
        for (int j = 0; j < N; ++j) v[j] = fmaxf(v[j], 0.f);
    }
    if (p.flags & DR_RESIDUAL) {
        const __nv_bfloat16* r = p.residual + m * p.Cout + c0;
        if (full && (p.Cout & 7) == 0 && N >= 8) {
#pragma unroll
            for (int q = 0; q < N / 8; ++q) {
                const uint4 u4 = __ldg(reinterpret_cast<const uint4*>(r) + q);
                const uint32_t* u = reinterpret_cast<const uint32_t*>(&u4);
#pragma unroll
                for (int j = 0; j < 4; ++j) { v[8 * q + 2 * j] += bf16_lo(u[j]); v[8 * q + 2 * j + 1] += bf16_hi(u[j]); }
            }
        } else {
#pragma unroll
            for (int j = 0; j < N; ++j)
                if (c0 + j < p.Cout) v[j] += __bfloat162float(r[j]);
        }
        if (p.flags & DR_RELU_AFTER_RESIDUAL) {
#pragma unroll
            for (int j = 0; j < N; ++j) v[j] = fmaxf(v[j], 0.f);
        }
    }
    if (p.flags & DR_OUT_F32) {
        float* y = reinterpret_cast<float*>(p.y) + m * p.ldc + p.coff + c0;
        if (full && (p.ldc & 3) == 0 && (p.coff & 3) == 0) {
#pragma unroll
            for (int q = 0; q < N / 4; ++q)
                reinterpret_cast<float4*>(y)[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        } else {
#pragma unroll
            for (int j = 0; j < N; ++j)
                if (c0 + j < p.Cout) y[j] = v[j];
        }
        return;
    }
    __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(p.y) + m * p.ldc + p.coff + c0;
    if (full && (p.ldc & 7) == 0 && (p.coff & 7) == 0) {
        if constexpr (N >= 8) {
#pragma unroll
            for (int q = 0; q < N / 8; ++q) {
                uint4 o;
                o.x = pack_bf16(v[8 * q + 0], v[8 * q + 1]);
                o.y = pack_bf16(v[8 * q + 2], v[8 * q + 3]);
                o.z = pack_bf16(v[8 * q + 4], v[8 * q + 5]);
                o.w = pack_bf16(v[8 * q + 6], v[8 * q + 7]);
                reinterpret_cast<uint4*>(y)[q] = o;
            }
        } else {
            uint2 o;
            o.x = pack_bf16(v[0], v[1]);
            o.y = pack_bf16(v[2], v[3]);
            *reinterpret_cast<uint2*>(y) = o;
        }
    } else {
#pragma unroll
        for (int j = 0; j < N; ++j)
            if (c0 + j < p.Cout) y[j] = __float2bfloat16_rn(v[j]);
    }
}

// ---- STAGED epilogue -------------------------------------------------------------------
// stage: float [TILE_M][C+1] holding acc + bias, ReLU'd (the caller wrote it), C = Cout <= 256.
// stage2: float [PH*PW][C+1], used only for pool-then-LRN.  NT threads, named barrier BAR.
template <int NT, int BAR>
__device__ __forceinline__ void bar_sync() {
    asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(NT) : "memory");
}

__device__ __forceinline__ size_t staged_smem_floats(int C, int PH, int PW, bool pool_then_lrn) {
    return (size_t)TILE_M * (C + 1) + (pool_then_lrn ? (size_t)PH * PW * (C + 1) : 0);
}

// In-place LRN along each row of the stage: thread t owns row t and keeps the 2*HALF+1
// original values of the window in registers while it overwrites the centre.
template <int HALF>
__device__ __forceinline__ void lrn_rows_inplace(float* stage, int rows, int C, int ld, int tid, int nthreads,
                                                 int half, float alpha_n, float beta, float kappa) {
    for (int row = tid; row < rows; row += nthreads) {
        float* s = stage + (size_t)row * ld;
        float win[2 * HALF + 1];          // win[HALF + d] = x[c + d]
#pragma unroll
        for (int i = 0; i < 2 * HALF + 1; ++i) win[i] = 0.f;
#pragma unroll
        for (int d = 0; d < HALF; ++d) win[HALF + 1 + d] = (d < C) ? s[d] : 0.f;   // x[0..HALF-1] ahead of c = -1
        for (int c = 0; c < C; ++c) {
#pragma unroll
            for (int i = 0; i < 2 * HALF; ++i) win[i] = win[i + 1];
            win[2 * HALF] = (c + HALF < C) ? s[c + HALF] : 0.f;
            float ss = win[HALF] * win[HALF];
#pragma unroll
            for (int d = 1; d <= HALF; ++d)
                if (d <= half) ss += win[HALF - d] * win[HALF - d] + win[HALF + d] * win[HALF + d];
            s[c] = win[HALF] * lrn_pow(kappa + alpha_n * ss, beta);
        }
    }
}

template <int NT, int BAR>
__device__ void epilogue_staged(const ConvParams& p, int tile, float* stage, float* stage2, int tid) {
    const int C = p.Cout, ld = C + 1;
    const bool lrn = p.flags & DR_LRN, pool = p.flags & DR_POOL;
    const bool lrn_first = lrn && (!pool || (p.flags & DR_LRN_BEFORE_POOL));
    bar_sync<NT, BAR>();                                   // stage complete
    if (lrn_first) {
        if (p.lrn_half <= 2) lrn_rows_inplace<2>(stage, TILE_M, C, ld, tid, NT, p.lrn_half, p.lrn_alpha_n, p.lrn_beta, p.lrn_k);
        else lrn_rows_inplace<7>(stage, TILE_M, C, ld, tid, NT, p.lrn_half, p.lrn_alpha_n, p.lrn_beta, p.lrn_k);
        bar_sync<NT, BAR>();
    }
    __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(p.y);
    if (!pool) {
        // store pass, two channels per thread, consecutive threads on consecutive channels
        const int C2 = C >> 1;
        for (int it = tid; it < TILE_M * C2; it += NT) {
            const int row = it / C2, c = (it - row * C2) * 2;
            const RowPix r = row_pixel(p, tile, row);
            if (!r.valid) continue;
            const long long m = ((long long)r.n * p.Ho + r.ho) * p.Wo + r.wo;
            *reinterpret_cast<uint32_t*>(y + m * p.ldc + p.coff + c) = pack_bf16(stage[row * ld + c], stage[row * ld + c + 1]);
        }
        return;
    }
    // pooled tile origin
    const int per = p.tiles_h * p.tiles_w;
    const int n = tile / per, t = tile - n * per;
    const int th = t / p.tiles_w, tw = t - th * p.tiles_w;
    const int pwc = 2 * p.PW + 1;
    const bool lrn_after = lrn && !lrn_first;
    const int C2 = C >> 1;
    for (int it = tid; it < p.PH * p.PW * C2; it += NT) {
        const int pp = it / C2, c = (it - pp * C2) * 2;
        const int pi = pp / p.PW, pj = pp - pi * p.PW;
        const int ph = th * p.PH + pi, pw = tw * p.PW + pj;
        if (ph >= p.Hy || pw >= p.Wy) continue;
        float b0 = 0.f, b1 = 0.f;
        int w0 = -1, w1 = -1;
#pragma unroll
        for (int dr_ = 0; dr_ < 3; ++dr_) {
            const int ho = 2 * ph - 1 + dr_;
            if (ho < 0 || ho >= p.Ho) continue;
#pragma unroll
            for (int dc = 0; dc < 3; ++dc) {
                const int wo = 2 * pw - 1 + dc;
                if (wo < 0 || wo >= p.Wo) continue;
                const int row = (2 * pi + dr_) * pwc + 2 * pj + dc;
                const float v0 = stage[row * ld + c], v1 = stage[row * ld + c + 1];
                if (w0 < 0 || v0 > b0) { b0 = v0; w0 = ho * p.Wo + wo; }
                if (w1 < 0 || v1 > b1) { b1 = v1; w1 = ho * p.Wo + wo; }
            }
        }
        const long long q = ((long long)n * p.Hy + ph) * p.Wy + pw;
        if (p.argmax) { p.argmax[q * C + c] = w0; p.argmax[q * C + c + 1] = w1; }
        if (lrn_after) { stage2[pp * ld + c] = b0; stage2[pp * ld + c + 1] = b1; }
        else *reinterpret_cast<uint32_t*>(y + q * p.ldc + p.coff + c) = pack_bf16(b0, b1);
    }
    if (!lrn_after) return;
    bar_sync<NT, BAR>();
    for (int it = tid; it < p.PH * p.PW * C2; it += NT) {
        const int pp = it / C2, c = (it - pp * C2) * 2;
        const int pi = pp / p.PW, pj = pp - pi * p.PW;
        const int ph = th * p.PH + pi, pw = tw * p.PW + pj;
        if (ph >= p.Hy || pw >= p.Wy) continue;
        const float* s = stage2 + pp * ld;
        float ss0 = 0.f, ss1 = 0.f;
        for (int d = -p.lrn_half; d <= p.lrn_half; ++d) {
            const int c0 = c + d, c1 = c + 1 + d;
            if (c0 >= 0 && c0 < C) ss0 += s[c0] * s[c0];
            if (c1 >= 0 && c1 < C) ss1 += s[c1] * s[c1];
        }
        const float o0 = s[c] * lrn_pow(p.lrn_k + p.lrn_alpha_n * ss0, p.lrn_beta);
        const float o1 = s[c + 1] * lrn_pow(p.lrn_k + p.lrn_alpha_n * ss1, p.lrn_beta);
        const long long q = ((long long)n * p.Hy + ph) * p.Wy + pw;
        *reinterpret_cast<uint32_t*>(y + q * p.ldc + p.coff + c) = pack_bf16(o0, o1);
    }
}

// Host side: fill the tiling fields of ConvParams (defined in conv_api.cu).
int conv_simt_launch(const ConvParams& p, cudaStream_t stream);
int conv_umma_gather_launch(const ConvParams& p, cudaStream_t stream);
int conv_umma_tma_launch(const ConvParams& p, cudaStream_t stream);
bool conv_umma_tma_supports(const ConvParams& p);
int conv_patch_tma_launch(const ConvParams& p, cudaStream_t stream);
bool conv_patch_tma_supports(const ConvParams& p);
int conv_stem_launch(const ConvParams& p, cudaStream_t stream);
bool conv_stem_supports(const ConvParams& p);
int conv_stem_d_launch(const ConvParams& p, cudaStream_t stream);
bool conv_stem_d_supports(const ConvParams& p);
bool conv_umma_gather_supports(const ConvParams& p);
int conv_qlin_launch(const ConvParams& p, cudaStream_t stream);
bool conv_qlin_supports(const ConvParams& p);
double conv_qlin_fill(const ConvParams& p);               // share of a tile's GEMM rows that are stored outputs
int conv_qlin_nt(const ConvParams& p);                    // output channels per accumulator block on that kernel
void conv_umma_tma_shape(ConvParams* p, bool* use_pair, bool* wide);
int conv_splitk_launch(const ConvParams& p, cudaStream_t stream);
bool conv_splitk_supports(const ConvParams& p);
size_t conv_splitk_scratch_bytes(const ConvParams& p);   // partial-tile scratch the split-K kernel wants; 0: it would not take the layer
// layers of one inception module in one split-K launch: a (long K) and b (short, e.g. the 1x1 reducer) read the same
// input; c (optional) reads b's output.  Scratch and counters are taken from a.
int conv_splitk_group_launch(const ConvParams& a, const ConvParams& b, const ConvParams* c, cudaStream_t stream);
bool conv_splitk_group_supports(const ConvParams& a, const ConvParams& b, const ConvParams* c);
size_t conv_splitk_group_scratch_bytes(const ConvParams& a, const ConvParams& b, const ConvParams* c);
int encode_conv_maps(const ConvParams& p, int b_box_rows, CUtensorMap* map_a, CUtensorMap* map_b, int* a_mode);
int encode_input_map(const ConvParams& p, CUtensorMap* map_a, int* a_mode, int box_rows = TILE_M);
int encode_rows_map(const void* ptr, long long rows, int cols, int ld, CUtensorMap* map, int box_rows = TILE_M);
int tunable(const char* name, int dflt);
// tensor_map.cu: memoised tensor-map encoders (bf16, element strides 1, zero fill)
int tmap_tiled(CUtensorMap* map, int rank, const void* ptr, const cuuint64_t* dims, const cuuint64_t* strides, const cuuint32_t* box,
               CUtensorMapSwizzle swizzle, CUtensorMapL2promotion l2);
int tmap_im2col(CUtensorMap* map, const void* ptr, const cuuint64_t dims[4], const cuuint64_t strides[3], const int lower[2], const int upper[2],
                unsigned channels, unsigned pixels, unsigned stride, CUtensorMapL2promotion l2);
long long tmap_driver_encodes();

}  // namespace dr
