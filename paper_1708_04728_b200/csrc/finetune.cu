// One SGD step of the layer-wise regression that re-learns a slim layer (Section 3.1, Eq. (w_b), Lemma 1):
//   f~(W, b; X) = ReLU(conv(X; W) + b) is fitted to the feature map Y_CNN of the layer group it replaces.
// The forward pass is the slim-layer convolution itself.  This file holds what the step adds:
//   regress_grad_kernel   dZ = (Y - Y_CNN) / B where Y > 0, as bf16; per-block partial sums of the loss and of dL/db
//   conv_wgrad_kernel     dL/dW[j, r, s, c] = sum over output pixels of dZ[m, j] * x[m @ tap (r, s), c] on the tensor
//                         cores: both operands are read with the pixel index as the contraction dimension
//   wgrad_reduce_kernel   sums the pixel-range partials in a fixed order
//   sgd_update_kernel     v <- momentum v + lr (g + decay w);  w <- w - v;  bf16 copy of w for the next forward pass
#include "conv_common.cuh"
#include "umma_ptx.cuh"

namespace dr {
using namespace ptx;

constexpr int WG_THREADS = 224;          // warp 0: TMA producer of x, warp 1: MMA issue, warps 2-5: drain, warp 6: TMA producer of dZ
constexpr int WG_MAX_STAGES = 8;
constexpr int WG_SMEM_MAX = 200 * 1024;
constexpr int RG_BLOCKS = 512;           // blocks (and partial rows) of regress_grad_kernel
constexpr int RG_THREADS = 256;

// The gradient as a matrix: rows = filter columns (tap, input channel) in units of one tap x 64 channels, columns =
// output channels.  A CTA owns a tile of two units (128 accumulator lanes) x cpt output channels (at most 256
// accumulator columns) and a range of pixel blocks.  In pair mode two CTAs of a cluster share a tile of four units x
// cpt channels: each loads its own two units of x and its half of the dZ columns, the even CTA issues MMAs of 256 rows
// that read both halves, and each drains its own 128 accumulator lanes: half the shared-memory fill per FLOP.
struct WgParams {
    int Cin, Cout, k, stride, pad, Ho, Wo;
    long long M;        // output pixels B*Ho*Wo: the contraction length
    int K;              // k*k*Cin
    int cpb;            // 64-channel blocks per tap
    int units;          // k*k*cpb
    int pair;           // 1: CTA pairs
    int n_rt;           // row tiles: ceil(units / 2), pairs: ceil(units / 4)
    int n_ct;           // column tiles
    int cpt;            // output channels per column tile (a multiple of 64, <= 256; pairs: 128 or 256)
    int splits;         // pixel ranges; each writes its own partial
    int pix;            // pixels (contraction rows) per pipeline stage: 64 or 128
    int pblocks;        // ceil(M / pix)
    int stages, stage_bytes;
    int a_mode;         // 0: x read as a [M][Cin] matrix (1x1 / stride 1 / pad 0), 1: im2col
    float* partial;     // [splits][Cout][K]
    int* status;
};

struct WgShared {
    uint64_t full[WG_MAX_STAGES], empty[WG_MAX_STAGES], accum;
    uint32_t tmem_base;
    int abort;
};

// Shared-memory operand descriptor for an operand whose contraction index is the row of a 128-byte-swizzled tile
// (rows of 64 non-contracted elements, 128 bytes): groups of 8 contraction rows are 1024 bytes apart (stride offset);
// the next 64 non-contracted elements are a whole box further (leading offset).  This is its low word (start
// address, leading offset); the high word (stride offset, version, swizzle) is that of the K-major form, SDESC_HI_SW128.
__device__ __forceinline__ uint32_t sdesc_mn_lo(uint32_t smem_addr, uint32_t chunk_bytes) {
    return ((smem_addr & 0x3FFFFu) >> 4) | (((chunk_bytes >> 4) & 0x3FFFu) << 16);
}

template <bool PAIR, int PIX>
__global__ void __launch_bounds__(WG_THREADS, 1)
conv_wgrad_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_dz, const WgParams p) {
    constexpr int BOX = PIX * 128;                               // one TMA box: PIX pixels x 64 channels of bf16
    extern __shared__ uint8_t wg_smem_raw[];
    __shared__ WgShared sh;
    const uint32_t smem_base = (smem_u32(wg_smem_raw) + 1023u) & ~1023u;
    uint8_t* const smem_al = wg_smem_raw + (smem_base - smem_u32(wg_smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;       // pairs: 0 issues the MMAs
    const int bid = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int rt = bid % p.n_rt;
    const int ct = (bid / p.n_rt) % p.n_ct;
    const int split = bid / (p.n_rt * p.n_ct);
    const int u0 = PAIR ? 4 * rt + 2 * (int)rank : 2 * rt;
    const int n_units = max(0, min(2, p.units - u0));           // units in this CTA's accumulator lanes (0: pairs only)
    const int tile_units = PAIR ? min(4, p.units - 4 * rt) : n_units;
    const int j0 = ct * p.cpt;                                  // first output channel of the tile
    // 64-channel boxes of dZ: all of the tile's, or in a pair this CTA's half of N = 128 or 256 columns
    const int N = PAIR ? (p.Cout - j0 > 128 ? 256 : 128) : ((min(p.cpt, p.Cout - j0) + 63) >> 6) * 64;
    const int nb = PAIR ? N >> 7 : N >> 6;
    const int jb = PAIR ? j0 + (int)rank * (N >> 1) : j0;       // first channel this CTA loads
    const int pb0 = (int)((long long)split * p.pblocks / p.splits);
    const int pb1 = (int)((long long)(split + 1) * p.pblocks / p.splits);
    const int stages = p.stages;
    volatile int* abort_flag = &sh.abort;

    if (threadIdx.x == 0) {
        for (int i = 0; i < WG_MAX_STAGES; ++i) { mbar_init(&sh.full[i], 1); mbar_init(&sh.empty[i], 1); }
        mbar_init(&sh.accum, 1);
        sh.abort = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_x);
        prefetch_tensormap(&map_dz);
    }
    if (warp == 1) {
        if (PAIR) { tmem_alloc_pair(&sh.tmem_base, 256); tmem_relinquish_pair(); }
        else { tmem_alloc(&sh.tmem_base, 256); tmem_relinquish(); }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();                               // both CTAs' barriers exist before any remote arrive
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            // bytes that land per stage: in a pair both CTAs' loads report to the even CTA's barrier
            const uint32_t tx = (uint32_t)(tile_units + (PAIR ? 2 : 1) * nb) * BOX;
            // the single issuing thread is on the critical path: everything that does not change per stage is computed
            // here, and the pixel coordinates advance with one division per stage
            const uint32_t hw = (uint32_t)(p.Ho * p.Wo), Wo = (uint32_t)p.Wo;
            int uc0[2], ur[2], ut[2];
            for (int u = 0; u < 2; ++u) {
                const int unit = min(u0 + u, p.units - 1);
                const int tap = unit / p.cpb;
                uc0[u] = (unit - tap * p.cpb) << 6;
                ur[u] = tap / p.k;
                ut[u] = tap - ur[u] * p.k;
            }
            long long m0 = (long long)pb0 * PIX;
            uint32_t img = (uint32_t)(m0 / hw);
            uint32_t rem = (uint32_t)(m0 - (long long)img * hw);
            int s = 0;
            uint32_t ph = 0;
            for (int pb = pb0; pb < pb1; ++pb, m0 += PIX, rem += PIX) {
                if (pb - pb0 >= stages && !mbar_wait(&sh.empty[s], ph ^ 1, abort_flag)) {
                    if (!*abort_flag) report_timeout(p.status, 61, bid);
                    *abort_flag = 1;
                    break;
                }
                uint8_t* dst = smem_al + (size_t)s * p.stage_bytes;
                if (rank == 0) mbar_arrive_expect_tx(&sh.full[s], tx);
                while (rem >= hw) { rem -= hw; ++img; }
                const uint32_t ho = rem / Wo, wo = rem - ho * Wo;
                const int hb = (int)ho * p.stride - p.pad, wb = (int)wo * p.stride - p.pad;
                for (int u = 0; u < n_units; ++u) {
                    const int c0 = uc0[u], r = ur[u], t = ut[u];
                    uint8_t* xd = dst + (size_t)u * BOX;
                    if (PAIR) {
                        if (p.a_mode == 0) tma_load_2d_pair(xd, &map_x, &sh.full[s], c0, (int)m0);
                        else tma_load_im2col_4d_pair(xd, &map_x, &sh.full[s], c0, wb, hb, (int)img, (uint16_t)t, (uint16_t)r);
                    } else {
                        if (p.a_mode == 0) tma_load_2d(xd, &map_x, &sh.full[s], c0, (int)m0);
                        else tma_load_im2col_4d(xd, &map_x, &sh.full[s], c0, wb, hb, (int)img, (uint16_t)t, (uint16_t)r);
                    }
                }
                if (++s == stages) { s = 0; ph ^= 1; }
            }
        }
        __syncwarp();
    } else if (warp == 6) {
        if (lane == 0) {
            // the dZ boxes of every stage, issued by a thread of their own so that the two operands' loads go out side by
            // side; the bytes are expected on the barrier by the x producer of the even CTA (they may land first)
            int s = 0;
            uint32_t ph = 0;
            int m0 = pb0 * PIX;
            for (int pb = pb0; pb < pb1; ++pb, m0 += PIX) {
                if (pb - pb0 >= stages && !mbar_wait(&sh.empty[s], ph ^ 1, abort_flag)) {
                    if (!*abort_flag) report_timeout(p.status, 64, bid);
                    *abort_flag = 1;
                    break;
                }
                uint8_t* dst = smem_al + (size_t)s * p.stage_bytes + 2 * BOX;
                for (int i = 0; i < nb; ++i) {
                    if (PAIR) tma_load_2d_pair(dst + (size_t)i * BOX, &map_dz, &sh.full[s], jb + 64 * i, m0);
                    else tma_load_2d(dst + (size_t)i * BOX, &map_dz, &sh.full[s], jb + 64 * i, m0);
                }
                if (++s == stages) { s = 0; ph ^= 1; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = make_idesc_bf16(PAIR ? 2 * TILE_M : TILE_M, N) | (1u << 15) | (1u << 16);   // both operands contraction-row ("MN-major")
            int s = 0;
            uint32_t ph = 0, accum = 0;
            for (int pb = pb0; pb < pb1; ++pb) {
                if (!mbar_wait(&sh.full[s], ph, abort_flag)) {
                    if (!*abort_flag) report_timeout(p.status, 62, bid);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t a = smem_base + (uint32_t)s * (uint32_t)p.stage_bytes;       // x: the accumulator's lanes
                const uint32_t b = a + 2 * BOX;                                          // dZ: its columns
#pragma unroll
                for (int ks = 0; ks < PIX / 16; ++ks) {       // 16 pixels per MMA: two 8-row groups
                    // descriptors as 32-bit low words (start address, leading offset); the high word is the constant
                    // of the 128-byte swizzle: one MMA costs the issuing thread a few instructions, not a few dozen
                    umma_bf16_lo<PAIR>(tmem, sdesc_mn_lo(a, BOX) + ks * 128, sdesc_mn_lo(b, BOX) + ks * 128, idesc, accum, 1u);
                    accum = 1;
                }
                if (PAIR) umma_commit_pair(&sh.empty[s], 3);
                else umma_commit(&sh.empty[s]);
                if (++s == stages) { s = 0; ph ^= 1; }
            }
            if (PAIR) umma_commit_pair(&sh.accum, 3);   // also after a timeout: fires once whatever was issued has finished
            else umma_commit(&sh.accum);
        }
        __syncwarp();
    } else {
        // drain: TMEM lane = (unit, input channel within the unit), column = output channel of the tile.  The 32
        // lanes of a warp are 32 consecutive input channels of one tap: each store instruction writes 128 contiguous bytes.
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const int unit = u0 + (row >> 6);
        const int tap = unit / p.cpb;
        const int ch = ((unit - tap * p.cpb) << 6) + (row & 63);
        const bool row_ok = (row >> 6) < n_units && ch < p.Cin;
        const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.accum, 0, abort_flag));
        if (!ok) {
            if (!*abort_flag) report_timeout(p.status, 63, bid);
            *abort_flag = 1;
        } else if (!*abort_flag && pb1 > pb0) {
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16);
            float* out = p.partial + ((size_t)split * p.Cout + j0) * p.K + (size_t)tap * p.Cin + ch;
            for (int c = 0; c < N; c += 32) {
                uint32_t v[32];
                tmem_ld_x32(taddr + c, v);
                tmem_ld_wait();
                if (row_ok) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (j0 + c + i < p.Cout) out[(size_t)(c + i) * p.K] = __uint_as_float(v[i]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();                               // neither CTA leaves while the other may still signal it
    if (warp == 1) {
        if (PAIR) tmem_dealloc_pair(tmem, 256);
        else tmem_dealloc(tmem, 256);
    }
}

// Layers the tensor-core kernel does not take (fewer than 64 input channels, channel counts that are not multiples of
// 8): one thread per filter element walks all output pixels in order.  For completeness, not speed.
__global__ void conv_wgrad_simt_kernel(int B, int H, int W, int Cin, int Cout, int k, int stride, int pad, int Ho, int Wo,
                                       const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ dz, float* __restrict__ dw) {
    const int jt = blockIdx.x;                      // (filter j, tap)
    const int j = jt / (k * k), tap = jt - j * (k * k);
    const int r = tap / k, t = tap - r * k;
    for (int c = threadIdx.x; c < Cin; c += blockDim.x) {
        float acc = 0.f;
        for (int n = 0; n < B; ++n)
            for (int ho = 0; ho < Ho; ++ho) {
                const int hi = ho * stride - pad + r;
                if (hi < 0 || hi >= H) continue;
                for (int wo = 0; wo < Wo; ++wo) {
                    const int wi = wo * stride - pad + t;
                    if (wi < 0 || wi >= W) continue;
                    acc = fmaf(__bfloat162float(dz[(((size_t)n * Ho + ho) * Wo + wo) * Cout + j]),
                               __bfloat162float(x[(((size_t)n * H + hi) * W + wi) * Cin + c]), acc);
                }
            }
        dw[(size_t)jt * Cin + c] = acc;
    }
}

// dw[i] = sum over the pixel-range partials, in range order (the same result on every run).
__global__ void wgrad_reduce_kernel(const float4* __restrict__ partial, int splits, size_t n4, float4* __restrict__ dw) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 a = partial[i];
        for (int s = 1; s < splits; ++s) {
            const float4 b = partial[(size_t)s * n4 + i];
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        }
        dw[i] = a;
    }
}

// dZ, loss and bias-gradient partials.  y, yt, dz: dense [M][C] bf16, C a multiple of 8, C / 8 <= RG_THREADS.
// Thread t works on the 8-channel vector t % (C/8) of rows t / (C/8), + rows_per_pass, ...: a thread stays on its
// channels, so its eight bias sums live in registers; the rows of a block are contiguous, so loads are coalesced.
// partials: [RG_BLOCKS][C + 1] floats, column C = the block's sum of (y - yt)^2.
__global__ void __launch_bounds__(RG_THREADS)
regress_grad_kernel(const uint4* __restrict__ y, const uint4* __restrict__ yt, long long M, int C, float scale, int relu,
                    uint4* __restrict__ dz, float* __restrict__ partials) {
    __shared__ float red[RG_THREADS * 9];
    const int nv = C >> 3;
    const int rows_per_pass = RG_THREADS / nv;
    const int t = threadIdx.x;
    const int vc = t % nv, ro = t / nv;
    const long long rows_per_block = (M + gridDim.x - 1) / gridDim.x;
    const long long r0 = (long long)blockIdx.x * rows_per_block;
    const long long r1 = r0 + rows_per_block < M ? r0 + rows_per_block : M;
    float sb[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    float sl = 0.f;
    if (ro < rows_per_pass) {
        for (long long r = r0 + ro; r < r1; r += rows_per_pass) {
            const size_t i = (size_t)r * nv + vc;
            const uint4 a = y[i], b = yt[i];
            const uint32_t au[4] = {a.x, a.y, a.z, a.w}, bu[4] = {b.x, b.y, b.z, b.w};
            uint32_t o[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float y0 = bf16_lo(au[k]), y1 = bf16_hi(au[k]);
                const float e0 = y0 - bf16_lo(bu[k]), e1 = y1 - bf16_hi(bu[k]);
                sl = fmaf(e0, e0, sl);
                sl = fmaf(e1, e1, sl);
                const float g0 = (relu && !(y0 > 0.f)) ? 0.f : e0 * scale;
                const float g1 = (relu && !(y1 > 0.f)) ? 0.f : e1 * scale;
                o[k] = pack_bf16(g0, g1);
                sb[2 * k] += bf16_lo(o[k]);          // the bias gradient sums what the filter gradient sees: the rounded dZ
                sb[2 * k + 1] += bf16_hi(o[k]);
            }
            dz[i] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) red[t * 9 + k] = sb[k];
    red[t * 9 + 8] = sl;
    __syncthreads();
    float* out = partials + (size_t)blockIdx.x * (C + 1);
    if (t < nv) {                                   // fixed order over the rows-in-flight of this block
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int rr = 0; rr < rows_per_pass; ++rr)
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] += red[(rr * nv + t) * 9 + k];
#pragma unroll
        for (int k = 0; k < 8; ++k) out[t * 8 + k] = acc[k];
    }
    if (t == RG_THREADS - 1) {
        float acc = 0.f;
        for (int i = 0; i < RG_THREADS; ++i) acc += red[i * 9 + 8];
        out[C] = acc;
    }
}

// Channel counts the vector kernel does not take (not a multiple of 8, or more than 2048): element-wise dZ, then one
// block per channel (and one for the loss) summing its column with a fixed-order tree.  For completeness, not speed.
__global__ void regress_grad_scalar_kernel(size_t n, float scale, int relu, const __nv_bfloat16* __restrict__ y,
                                           const __nv_bfloat16* __restrict__ yt, __nv_bfloat16* __restrict__ dz) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float a = __bfloat162float(y[i]);
        const float g = (relu && !(a > 0.f)) ? 0.f : (a - __bfloat162float(yt[i])) * scale;
        dz[i] = __float2bfloat16_rn(g);
    }
}
__global__ void __launch_bounds__(256)
regress_sums_scalar_kernel(long long M, int C, float loss_scale, const __nv_bfloat16* __restrict__ y, const __nv_bfloat16* __restrict__ yt,
                           const __nv_bfloat16* __restrict__ dz, float* __restrict__ db, float* __restrict__ loss) {
    __shared__ float red[256];
    const int c = blockIdx.x;                       // c == C: the loss
    float acc = 0.f;
    if (c < C) {
        for (long long m = threadIdx.x; m < M; m += 256) acc += __bfloat162float(dz[(size_t)m * C + c]);
    } else {
        const size_t n = (size_t)M * C;
        for (size_t i = threadIdx.x; i < n; i += 256) {
            const float e = __bfloat162float(y[i]) - __bfloat162float(yt[i]);
            acc = fmaf(e, e, acc);
        }
    }
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if ((int)threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        if (c < C) db[c] = red[0];
        else if (loss) *loss = red[0] * loss_scale;
    }
}

// db[c] = sum over blocks of the partials, loss = loss_scale * sum of the squared-error partials.  32 columns per
// block, 16 threads per column: each sums every 16th partial row in order, then the 16 sums are added in order.
__global__ void __launch_bounds__(512)
regress_finalize_kernel(const float* __restrict__ partials, int blocks, int C, float loss_scale, float* __restrict__ db,
                        float* __restrict__ loss) {
    __shared__ float red[16][33];
    const int cx = threadIdx.x & 31, part = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + cx;
    float acc = 0.f;
    if (c <= C)
        for (int b = part; b < blocks; b += 16) acc += partials[(size_t)b * (C + 1) + c];
    red[part][cx] = acc;
    __syncthreads();
    if (part == 0 && c <= C) {
        float t = 0.f;
#pragma unroll
        for (int k = 0; k < 16; ++k) t += red[k][cx];
        if (c < C) db[c] = t;
        else if (loss) *loss = t * loss_scale;
    }
}

__global__ void sgd_update_kernel(size_t n, float* __restrict__ w, float* __restrict__ v, const float* __restrict__ g, float lr, float momentum,
                                  float decay, __nv_bfloat16* __restrict__ w_bf16) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float wi = w[i];
        const float vi = momentum * v[i] + lr * (g[i] + decay * wi);
        const float wn = wi - vi;
        v[i] = vi;
        w[i] = wn;
        if (w_bf16) w_bf16[i] = __float2bfloat16_rn(wn);
    }
}

// ------------------------------------------------------------------------------------------------ host side
struct WgPlan { WgParams p; size_t partial_bytes; int ctas; bool simt; };

static int wgrad_plan(const dr_conv_desc* d, int B, int H, int W, WgPlan* out) {
    if (!d || d->k <= 0 || d->stride <= 0 || d->pad < 0 || d->Cin <= 0 || d->Cout <= 0 || B < 0 || H <= 0 || W <= 0) return DR_ERR_INVALID_ARG;
    if (H + 2 * d->pad < d->k || W + 2 * d->pad < d->k) return DR_ERR_INVALID_ARG;
    if (d->k > 255) return DR_ERR_UNSUPPORTED;
    WgParams& p = out->p;
    out->simt = (d->Cin & 7) || d->Cin < 64 || (d->Cout & 7);     // TMA wants rows of 128 bytes and 16-byte pitches
    p.Cin = d->Cin; p.Cout = d->Cout; p.k = d->k; p.stride = d->stride; p.pad = d->pad;
    p.Ho = (H + 2 * d->pad - d->k) / d->stride + 1;
    p.Wo = (W + 2 * d->pad - d->k) / d->stride + 1;
    p.M = (long long)B * p.Ho * p.Wo;
    if (p.M > 0x7fffffffLL - 128) return DR_ERR_UNSUPPORTED;
    p.K = d->k * d->k * d->Cin;
    p.cpb = (d->Cin + 63) / 64;
    p.units = d->k * d->k * p.cpb;
    p.n_rt = (p.units + 1) / 2;
    p.n_ct = (d->Cout + 255) / 256;
    p.cpt = ((d->Cout + p.n_ct - 1) / p.n_ct + 63) / 64 * 64;    // even column tiles: 288 filters run as 192 + 96, not 256 + 32
    p.n_ct = (d->Cout + p.cpt - 1) / p.cpt;
    // CTA pairs where their coarser tiles (4 units x 128 or 256 channels) waste little: share of the MMA work that is real
    {
        const int n_rt2 = (p.units + 3) / 4, n_ct2 = (d->Cout + 255) / 256;
        const int cols2 = (n_ct2 - 1) * 256 + (d->Cout - (n_ct2 - 1) * 256 > 128 ? 256 : 128);
        const double eff1 = (double)p.units / (2 * p.n_rt) * d->Cout / ((double)(p.n_ct - 1) * p.cpt + ((d->Cout - (p.n_ct - 1) * p.cpt + 63) / 64 * 64));
        const double eff2 = (double)p.units / (4 * n_rt2) * d->Cout / cols2;
        const int pref = tunable("DR_WGRAD_PAIR", -1);
        p.pair = pref >= 0 ? (pref != 0) : (eff2 >= 0.85 * eff1);
        if (p.pair) { p.n_rt = n_rt2; p.n_ct = n_ct2; p.cpt = 256; }
    }
    // Pipeline shape, measured at batch 256 on B200.  Pairs with 256 columns: stages of 128 pixels, three of them.  Pairs
    // with 128 columns: stages of 64 pixels, three of them, so that two CTAs share an SM (one drains or starts while
    // the other computes; each holds 256 of the 512 TMEM columns).  Single CTAs: stages of 64 pixels, as many as fit.
    const bool narrow_pair = p.pair && d->Cout <= 128;
    {
        const int px = tunable("DR_WGRAD_PIX", 0);
        p.pix = px == 64 || px == 128 ? px : ((p.pair && !narrow_pair) ? 128 : 64);
    }
    p.stage_bytes = (p.pair ? (narrow_pair ? 3 : 4) : 2 + p.cpt / 64) * p.pix * 128;
    p.stages = WG_SMEM_MAX / p.stage_bytes;
    if (p.stages > WG_MAX_STAGES) p.stages = WG_MAX_STAGES;
    if (narrow_pair && p.pix == 64 && p.stages > 4) p.stages = 4;   // 4 x 24 KB: two CTAs per SM
    {
        const int st = tunable("DR_WGRAD_STAGES", 0);
        if (st >= 1 && st < p.stages) p.stages = st;
    }
    p.pblocks = (int)((p.M + p.pix - 1) / p.pix);
    p.a_mode = (d->k == 1 && d->stride == 1 && d->pad == 0) ? 0 : 1;
    // Pixel ranges.  The launch runs in rounds of as many CTAs as the SMs hold: take the number of ranges with the least
    // rounds x (pixel blocks per range + what a range adds).  Fitted on the 4e merged 5x5 layer at batch 256
    // (3 .. 14 ranges: 472 .. 601 us): a CTA's start, drain and the trip of its partial tile through the reduction cost
    // as much as 14 blocks of 128 pixels.  At least four blocks of 128 pixels per range.
    const int tiles = p.n_rt * p.n_ct;
    int s = tunable("DR_WGRAD_SPLITS", 0);
    if (s <= 0) {
        // CTAs that run at a time: one per SM, two where the pipeline leaves room in shared memory
        const int slots = num_sms() * ((p.stages * p.stage_bytes + 1024) * 2 <= 226 * 1024 ? 2 : 1);
        long long best = -1;
        const int per128 = 128 / p.pix;                          // pixel blocks per 128 pixels
        const int smax = p.pblocks / (4 * per128) < 64 ? p.pblocks / (4 * per128) : 64;
        s = 1;
        for (int c = 1; c <= smax; ++c) {
            const long long rounds = ((long long)tiles * c * (p.pair ? 2 : 1) + slots - 1) / slots;
            const long long cost = rounds * ((p.pblocks + c - 1) / c + 14 * per128);
            if (best < 0 || cost < best) { best = cost; s = c; }
        }
    }
    if (s > p.pblocks) s = p.pblocks;
    if (s < 1) s = 1;
    p.splits = s;
    out->ctas = tiles * s * (p.pair ? 2 : 1);
    out->partial_bytes = (p.M && !out->simt) ? (size_t)s * d->Cout * p.K * sizeof(float) : 0;   // an empty batch needs no scratch
    return DR_OK;
}

}  // namespace dr

using namespace dr;

extern "C" int dr_conv_wgrad_workspace_bytes(const dr_conv_desc* desc, int B, int H, int W, size_t* bytes) {
    if (!bytes) return DR_ERR_INVALID_ARG;
    WgPlan pl;
    const int st = wgrad_plan(desc, B, H, W, &pl);
    if (st != DR_OK) return st;
    *bytes = (pl.partial_bytes + 255) / 256 * 256;
    return DR_OK;
}

extern "C" int dr_conv_wgrad(const dr_conv_desc* desc, int B, int H, int W, const void* x, const void* dz, float* dw, void* workspace,
                             size_t workspace_bytes, void* stream) {
    WgPlan pl;
    const int st = wgrad_plan(desc, B, H, W, &pl);
    if (st != DR_OK) return st;
    if (!x || !dz || !dw || (!workspace && pl.partial_bytes)) return DR_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(dz) || !aligned16(dw) || ((uintptr_t)workspace & 255)) return DR_ERR_ALIGNMENT;
    if (workspace_bytes < pl.partial_bytes) return DR_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    WgParams& p = pl.p;
    const size_t n = (size_t)p.Cout * p.K;
    if (p.M == 0) return cuda_status(cudaMemsetAsync(dw, 0, n * sizeof(float), s));
    if (pl.simt) {
        const int threads = p.Cin >= 128 ? 128 : (p.Cin >= 64 ? 64 : 32);
        conv_wgrad_simt_kernel<<<(unsigned)(p.Cout * p.k * p.k), threads, 0, s>>>(B, H, W, p.Cin, p.Cout, p.k, p.stride, p.pad, p.Ho, p.Wo,
                                                                                reinterpret_cast<const __nv_bfloat16*>(x),
                                                                                reinterpret_cast<const __nv_bfloat16*>(dz), dw);
        count_launch();
        return launch_status();
    }
    p.partial = reinterpret_cast<float*>(workspace);
    p.status = dev_status_ptr();
    ConvParams cp = {};
    cp.x = reinterpret_cast<const __nv_bfloat16*>(x);
    cp.B = B; cp.H = H; cp.W = W; cp.Cin = p.Cin; cp.Cout = p.Cout; cp.k = p.k; cp.stride = p.stride; cp.pad = p.pad;
    cp.Ho = p.Ho; cp.Wo = p.Wo; cp.M = p.M; cp.K = p.K;
    alignas(64) CUtensorMap map_x, map_dz;
    int a_mode = 0;
    int est = encode_input_map(cp, &map_x, &a_mode, p.pix);
    if (est == DR_OK) est = encode_rows_map(dz, p.M, p.Cout, p.Cout, &map_dz, p.pix);
    if (est != DR_OK) return est;
    static PerDeviceFlag attr_set;
    if (!attr_set.get()) {
        if (cudaFuncSetAttribute(conv_wgrad_kernel<false, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, WG_SMEM_MAX + 1024) != cudaSuccess ||
            cudaFuncSetAttribute(conv_wgrad_kernel<true, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, WG_SMEM_MAX + 1024) != cudaSuccess ||
            cudaFuncSetAttribute(conv_wgrad_kernel<false, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WG_SMEM_MAX + 1024) != cudaSuccess ||
            cudaFuncSetAttribute(conv_wgrad_kernel<true, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WG_SMEM_MAX + 1024) != cudaSuccess) {
            (void)cudaGetLastError();
            return DR_ERR_CUDA;
        }
        attr_set.set();
    }
    {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.gridDim = dim3((unsigned)pl.ctas); cfg.blockDim = dim3(WG_THREADS);
        cfg.dynamicSmemBytes = (size_t)p.stages * p.stage_bytes + 1024; cfg.stream = s;
        cfg.attrs = attr; cfg.numAttrs = p.pair ? 1 : 0;
        cudaError_t e;
        if (p.pix == 64) e = p.pair ? cudaLaunchKernelEx(&cfg, conv_wgrad_kernel<true, 64>, map_x, map_dz, p)
                                    : cudaLaunchKernelEx(&cfg, conv_wgrad_kernel<false, 64>, map_x, map_dz, p);
        else e = p.pair ? cudaLaunchKernelEx(&cfg, conv_wgrad_kernel<true, 128>, map_x, map_dz, p)
                        : cudaLaunchKernelEx(&cfg, conv_wgrad_kernel<false, 128>, map_x, map_dz, p);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return DR_ERR_CUDA; }
    }
    count_launch();
    int lst = launch_status();
    if (lst != DR_OK) return lst;
    const size_t n4 = n / 4;                       // K is a multiple of 8
    size_t blocks = (n4 + 255) / 256;
    if (blocks > (size_t)num_sms() * 8) blocks = (size_t)num_sms() * 8;
    wgrad_reduce_kernel<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const float4*>(p.partial), p.splits, n4, reinterpret_cast<float4*>(dw));
    count_launch();
    return launch_status();
}

extern "C" int dr_regress_workspace_bytes(int C, size_t* bytes) {
    if (!bytes || C <= 0) return DR_ERR_INVALID_ARG;
    *bytes = ((size_t)RG_BLOCKS * (C + 1) * sizeof(float) + 255) / 256 * 256;
    return DR_OK;
}

extern "C" int dr_regress_grad(int B, int H, int W, int C, const void* y, const void* yt, int relu, void* dz, float* db, float* loss,
                               void* workspace, size_t workspace_bytes, void* stream) {
    return dr_regress_grad_shard(B, B, H, W, C, y, yt, relu, dz, db, loss, workspace, workspace_bytes, stream);
}

extern "C" int dr_regress_grad_shard(int B, int batch, int H, int W, int C, const void* y, const void* yt, int relu, void* dz, float* db,
                                     float* loss, void* workspace, size_t workspace_bytes, void* stream) {
    if (B <= 0 || batch < B || H <= 0 || W <= 0 || C <= 0 || !y || !yt || !dz || !db || !workspace) return DR_ERR_INVALID_ARG;
    if (!aligned16(y) || !aligned16(yt) || !aligned16(dz) || ((uintptr_t)workspace & 255)) return DR_ERR_ALIGNMENT;
    size_t need = 0;
    dr_regress_workspace_bytes(C, &need);
    if (workspace_bytes < need) return DR_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    const long long M = (long long)B * H * W;
    if ((C & 7) || (C >> 3) > RG_THREADS) {
        const size_t n = (size_t)M * C;
        size_t blocks = (n + 255) / 256;
        if (blocks > (size_t)num_sms() * 8) blocks = (size_t)num_sms() * 8;
        regress_grad_scalar_kernel<<<(unsigned)blocks, 256, 0, s>>>(n, 1.f / (float)batch, relu ? 1 : 0, reinterpret_cast<const __nv_bfloat16*>(y),
                                                                   reinterpret_cast<const __nv_bfloat16*>(yt), reinterpret_cast<__nv_bfloat16*>(dz));
        count_launch();
        int st0 = launch_status();
        if (st0 != DR_OK) return st0;
        regress_sums_scalar_kernel<<<C + 1, 256, 0, s>>>(M, C, 0.5f / (float)batch, reinterpret_cast<const __nv_bfloat16*>(y),
                                                        reinterpret_cast<const __nv_bfloat16*>(yt), reinterpret_cast<const __nv_bfloat16*>(dz), db, loss);
        count_launch();
        return launch_status();
    }
    float* partials = reinterpret_cast<float*>(workspace);
    regress_grad_kernel<<<RG_BLOCKS, RG_THREADS, 0, s>>>(reinterpret_cast<const uint4*>(y), reinterpret_cast<const uint4*>(yt), M, C, 1.f / (float)batch,
                                                       relu ? 1 : 0, reinterpret_cast<uint4*>(dz), partials);
    count_launch();
    int st = launch_status();
    if (st != DR_OK) return st;
    regress_finalize_kernel<<<(C + 1 + 31) / 32, 512, 0, s>>>(partials, RG_BLOCKS, C, 0.5f / (float)batch, db, loss);
    count_launch();
    return launch_status();
}

extern "C" int dr_sgd_update(size_t n, float* w, float* v, const float* g, float lr, float momentum, float decay, void* w_bf16, void* stream) {
    if (!w || !v || !g) return DR_ERR_INVALID_ARG;
    if (n == 0) return DR_OK;
    size_t blocks = (n + 255) / 256;
    if (blocks > (size_t)num_sms() * 8) blocks = (size_t)num_sms() * 8;
    sgd_update_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(n, w, v, g, lr, momentum, decay, reinterpret_cast<__nv_bfloat16*>(w_bf16));
    count_launch();
    return launch_status();
}

static size_t round256(size_t b) { return (b + 255) / 256 * 256; }

extern "C" int dr_regress_step_workspace_bytes(const dr_conv_desc* desc, int B, int H, int W, size_t* bytes) {
    if (!bytes || !desc) return DR_ERR_INVALID_ARG;
    size_t a = 0, b = 0, c = 0;
    int st = dr_conv_wgrad_workspace_bytes(desc, B, H, W, &a);
    if (st == DR_OK) st = dr_regress_workspace_bytes(desc->Cout, &b);
    if (st == DR_OK) st = dr_conv_workspace_bytes(desc, B, H, W, &c);
    if (st != DR_OK) return st;
    *bytes = round256(a) + round256(b) + round256(c);
    return DR_OK;
}

extern "C" int dr_regress_shard_grads(const dr_conv_desc* desc, int B, int batch, int H, int W, const void* x, const void* yt, const void* w_bf16,
                                      const float* b, void* y, void* dz, float* dw, float* db, float* loss, void* workspace,
                                      size_t workspace_bytes, void* stream) {
    if (!desc || !x || !yt || !b || !w_bf16 || !y || !dz || !dw || !db || !workspace || batch < B) return DR_ERR_INVALID_ARG;
    if (!(desc->flags & DR_BIAS) || (desc->flags & ~(unsigned)(DR_BIAS | DR_RELU))) return DR_ERR_UNSUPPORTED;
    if ((desc->y_ldc && desc->y_ldc != desc->Cout) || desc->y_coff) return DR_ERR_UNSUPPORTED;
    if ((uintptr_t)workspace & 255) return DR_ERR_ALIGNMENT;
    size_t wa = 0, wb = 0, wc = 0, need = 0;
    int st = dr_regress_step_workspace_bytes(desc, B, H, W, &need);
    if (st != DR_OK) return st;
    if (workspace_bytes < need) return DR_ERR_WORKSPACE;
    dr_conv_wgrad_workspace_bytes(desc, B, H, W, &wa);
    dr_regress_workspace_bytes(desc->Cout, &wb);
    dr_conv_workspace_bytes(desc, B, H, W, &wc);
    char* ws = reinterpret_cast<char*>(workspace);
    const int Ho = (H + 2 * desc->pad - desc->k) / desc->stride + 1, Wo = (W + 2 * desc->pad - desc->k) / desc->stride + 1;
    st = dr_conv_slim_ws(desc, B, H, W, x, w_bf16, b, nullptr, y, nullptr, wc ? ws + round256(wa) + round256(wb) : nullptr, wc, stream);
    if (st != DR_OK) return st;
    st = dr_regress_grad_shard(B, batch, Ho, Wo, desc->Cout, y, yt, (desc->flags & DR_RELU) ? 1 : 0, dz, db, loss, ws + round256(wa), wb, stream);
    if (st != DR_OK) return st;
    return dr_conv_wgrad(desc, B, H, W, x, dz, dw, ws, wa, stream);
}

extern "C" int dr_regress_step(const dr_conv_desc* desc, int B, int H, int W, const void* x, const void* yt, float* w, float* b, float* vw,
                               float* vb, void* w_bf16, float lr, float momentum, float decay, void* y, void* dz, float* dw, float* db,
                               float* loss, void* workspace, size_t workspace_bytes, void* stream) {
    if (!desc || !x || !yt || !w || !b || !vw || !vb || !w_bf16 || !y || !dz || !dw || !db || !workspace) return DR_ERR_INVALID_ARG;
    if (!(desc->flags & DR_BIAS) || (desc->flags & ~(unsigned)(DR_BIAS | DR_RELU))) return DR_ERR_UNSUPPORTED;
    if ((desc->y_ldc && desc->y_ldc != desc->Cout) || desc->y_coff) return DR_ERR_UNSUPPORTED;
    if ((uintptr_t)workspace & 255) return DR_ERR_ALIGNMENT;
    size_t wa = 0, wb = 0, wc = 0, need = 0;
    int st = dr_regress_step_workspace_bytes(desc, B, H, W, &need);
    if (st != DR_OK) return st;
    if (workspace_bytes < need) return DR_ERR_WORKSPACE;
    dr_conv_wgrad_workspace_bytes(desc, B, H, W, &wa);
    dr_regress_workspace_bytes(desc->Cout, &wb);
    dr_conv_workspace_bytes(desc, B, H, W, &wc);
    char* ws = reinterpret_cast<char*>(workspace);
    const int Ho = (H + 2 * desc->pad - desc->k) / desc->stride + 1, Wo = (W + 2 * desc->pad - desc->k) / desc->stride + 1;
    st = dr_conv_slim_ws(desc, B, H, W, x, w_bf16, b, nullptr, y, nullptr, wc ? ws + round256(wa) + round256(wb) : nullptr, wc, stream);
    if (st != DR_OK) return st;
    st = dr_regress_grad(B, Ho, Wo, desc->Cout, y, yt, (desc->flags & DR_RELU) ? 1 : 0, dz, db, loss, ws + round256(wa), wb, stream);
    if (st != DR_OK) return st;
    st = dr_conv_wgrad(desc, B, H, W, x, dz, dw, ws, wa, stream);
    if (st != DR_OK) return st;
    const size_t n = (size_t)desc->Cout * desc->k * desc->k * desc->Cin;
    st = dr_sgd_update(n, w, vw, dw, lr, momentum, decay, w_bf16, stream);
    if (st != DR_OK) return st;
    return dr_sgd_update((size_t)desc->Cout, b, vb, db, lr, momentum, 0.f, nullptr, stream);
}
