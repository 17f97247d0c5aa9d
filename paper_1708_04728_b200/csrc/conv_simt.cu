// CUDA-core implicit-GEMM convolution: runs any layer shape (any Cin, stride, pad, tail sizes).
// It is the path for shapes the tensor-core kernels do not take; it is slow and is never
// chosen for the layers that dominate the evaluated networks.
//
// One block computes one tile of 128 GEMM rows; it walks the tile's output channels 64 at a
// time.  Per 64-channel chunk: K is walked in blocks of 32 (flattened (r,s,c) index), the A
// (im2col) and B (filter) blocks are converted to float32 in shared memory, and each of the 256
// threads accumulates an 8-row x 4-channel register tile.
#include "conv_common.cuh"

namespace dr {

constexpr int SIMT_THREADS = 256;
constexpr int SIMT_BK = 32;
constexpr int SIMT_BN = 64;

__global__ void __launch_bounds__(SIMT_THREADS) conv_simt_kernel(const ConvParams p) {
    extern __shared__ __align__(16) float smem[];
    float* As = smem;                                   // [BK][128+4]
    float* Bs = As + SIMT_BK * (TILE_M + 4);            // [BK][64+4]
    float* stage = Bs + SIMT_BK * (SIMT_BN + 4);        // staged epilogue only
    const bool staged = p.flags & (DR_POOL | DR_LRN);
    const bool pool_then_lrn = (p.flags & DR_POOL) && (p.flags & DR_LRN) && !(p.flags & DR_LRN_BEFORE_POOL);
    float* stage2 = stage + (size_t)TILE_M * (p.Cout + 1);
    (void)pool_then_lrn;

    const int tid = threadIdx.x;
    const int tile = blockIdx.x;
    const int ty = tid >> 4, tx = tid & 15;             // 16 x 16 threads: rows 8*ty.., channels 4*tx..

    // A-load role: row a_row, 16 consecutive k of the block
    const int a_row = tid & 127, a_k0 = (tid >> 7) * 16;
    const RowPix a_pix = row_pixel(p, tile, a_row);
    const int a_h0 = a_pix.ho * p.stride - p.pad, a_w0 = a_pix.wo * p.stride - p.pad;
    // B-load role: channel b_col, 8 consecutive k
    const int b_col = tid & 63, b_k0 = (tid >> 6) * 8;

    const int n_first = staged ? 0 : blockIdx.y * p.Nt;
    const int n_last = staged ? p.Cout : min(p.Cout, n_first + p.Nt);

    for (int n0 = n_first; n0 < n_last; n0 += SIMT_BN) {
        float acc[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

        for (int k0 = 0; k0 < p.K; k0 += SIMT_BK) {
            {   // A block
                int kg = k0 + a_k0;
                int r = kg / (p.k * p.Cin);
                int rem = kg - r * p.k * p.Cin;
                int s = rem / p.Cin;
                int c = rem - s * p.Cin;
#pragma unroll 4
                for (int j = 0; j < 16; ++j) {
                    float v = 0.f;
                    const int hi = a_h0 + r, wi = a_w0 + s;
                    if (a_pix.valid && kg < p.K && hi >= 0 && hi < p.H && wi >= 0 && wi < p.W)
                        v = __bfloat162float(p.x[(((size_t)a_pix.n * p.H + hi) * p.W + wi) * p.Cin + c]);
                    As[(a_k0 + j) * (TILE_M + 4) + a_row] = v;
                    ++kg;
                    if (++c == p.Cin) { c = 0; if (++s == p.k) { s = 0; ++r; } }
                }
            }
            {   // B block
                const int col = n0 + b_col;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int kg = k0 + b_k0 + j;
                    float v = 0.f;
                    if (col < p.Cout && kg < p.K) v = __bfloat162float(p.w[(size_t)col * p.K + kg]);
                    Bs[(b_k0 + j) * (SIMT_BN + 4) + b_col] = v;
                }
            }
            __syncthreads();
#pragma unroll 8
            for (int kk = 0; kk < SIMT_BK; ++kk) {
                const float4 a0 = *reinterpret_cast<const float4*>(&As[kk * (TILE_M + 4) + ty * 8]);
                const float4 a1 = *reinterpret_cast<const float4*>(&As[kk * (TILE_M + 4) + ty * 8 + 4]);
                const float4 b = *reinterpret_cast<const float4*>(&Bs[kk * (SIMT_BN + 4) + tx * 4]);
                const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                const float bb[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
            }
            __syncthreads();
        }

        const int c0 = n0 + tx * 4;
        if (!staged) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const long long m = (long long)tile * TILE_M + ty * 8 + i;
                if (m < p.M) epilogue_direct<4>(p, m, c0, acc[i]);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int c = c0 + j;
                    if (c < p.Cout) {
                        float v = acc[i][j] + ((p.flags & DR_BIAS) ? __ldg(p.bias + c) : 0.f);
                        if (p.flags & DR_RELU) v = fmaxf(v, 0.f);
                        stage[(ty * 8 + i) * (p.Cout + 1) + c] = v;
                    }
                }
        }
    }
    if (staged) epilogue_staged<SIMT_THREADS, 1>(p, tile, stage, stage2, tid);
}

int conv_simt_launch(const ConvParams& p, cudaStream_t stream) {
    const bool staged = p.flags & (DR_POOL | DR_LRN);
    const bool pool_then_lrn = (p.flags & DR_POOL) && (p.flags & DR_LRN) && !(p.flags & DR_LRN_BEFORE_POOL);
    size_t smem = sizeof(float) * (SIMT_BK * (TILE_M + 4) + SIMT_BK * (SIMT_BN + 4));
    if (staged) smem += sizeof(float) * ((size_t)TILE_M * (p.Cout + 1) + (pool_then_lrn ? (size_t)p.PH * p.PW * (p.Cout + 1) : 0));
    if (smem > 227 * 1024) return DR_ERR_UNSUPPORTED;
    static PerDeviceFlag attr_set;
    if (!attr_set.get()) {
        if (cudaFuncSetAttribute(conv_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
            return DR_ERR_CUDA;
        attr_set.set();
    }
    if (p.m_tiles <= 0) return DR_OK;
    dim3 grid(p.m_tiles, staged ? 1 : p.n_blocks);
    conv_simt_kernel<<<grid, SIMT_THREADS, smem, stream>>>(p);
    count_launch();
    return launch_status();
}

}  // namespace dr
