// Implicit-GEMM convolution on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// tensor memory), NHWC bf16 in, float32 accumulate.  Two kernels share the MMA issue loop, the
// shared-memory operand layout and the epilogues of conv_common.cuh:
//
//   conv_umma_tma_kernel     the hot path.  Persistent, one CTA per SM.  Warp 0 streams operand
//       tiles with TMA: the activation tile in im2col mode (128 consecutive output pixels x 64
//       channels of one filter tap; the hardware walks rows/images and zero-fills the padding),
//       the filter tile in tiled mode.  Warp 1 issues the MMAs.  Warps 2-5 drain the finished
//       accumulator (bias, ReLU, residual, bf16 store) while the next tile is already being
//       multiplied into the second TMEM buffer.
//   conv_umma_gather_kernel  same MMA pipeline, but four producer warps build the operand tiles
//       in shared memory with ordinary loads.  Takes what TMA cannot describe (3-channel stem)
//       and the layers whose epilogue pools: there a tile is a 2-D patch of outputs.
//
// Operand tiles in shared memory: [rows][64 bf16] = 128-byte rows, 128-byte swizzle (16-byte chunk
// index XOR row%8), 8-row groups 1024 bytes apart — the K-major layout both TMA and the MMA
// descriptor understand.  One k-block = one filter tap x 64 input channels (zero-filled past Cin);
// only ceil(valid/16) MMAs of K=16 are issued for a partial block.
//
// Every wait on an mbarrier is bounded (see ptx::mbar_wait); on a timeout the CTA records
// DR_ERR_DEVICE_TIMEOUT, all roles leave their loops, and TMEM is released before exit.
#include "conv_common.cuh"
#include "umma_ptx.cuh"
#include "conv_drain.cuh"

namespace dr {
using namespace ptx;

constexpr int A_TILE_BYTES = TILE_M * 128;   // 128 rows x 64 bf16
constexpr int B_TILE_BYTES = 256 * 128;      // up to 256 filters x 64 bf16
constexpr int STAGE_BYTES = A_TILE_BYTES + B_TILE_BYTES;

__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// Issue the MMAs of one k-block: A tile at a_smem, B tile at b_smem, nk16 steps of K=16.
__device__ __forceinline__ void issue_kblock(uint32_t tmem_d, uint32_t a_smem, uint32_t b_smem, uint32_t idesc, int nk16, bool first) {
    const uint64_t ad = make_sdesc_sw128(a_smem), bd = make_sdesc_sw128(b_smem);
#pragma unroll
    for (int k = 0; k < 4; ++k)
        if (k < nk16) umma_bf16(tmem_d, ad + 2 * k, bd + 2 * k, idesc, (first && k == 0) ? 0u : 1u);
}

// Barrier of one epilogue group (128 threads): ids 1 and 2 as immediates, so that the kernel is seen to use three named
// barriers and not all sixteen (an SM has sixteen for all of its resident CTAs).
__device__ __forceinline__ void group_bar_sync(int bar) {
    if (bar == 1) asm volatile("bar.sync 1, 128;" ::: "memory");
    else asm volatile("bar.sync 2, 128;" ::: "memory");
}

// Lean epilogue with TMA stores (bias and/or ReLU, bf16 out): row-per-thread 16-byte global stores cost 32 memory
// wavefronts per warp instruction (32 rows, 32 different lines), which bounds the layers whose output is large
// against their K (1x1 convolutions at 56x56: 4.2 us per 128 x 256 tile).  Here the four warps of an epilogue group
// write 64-column chunks of their rows into a shared-memory buffer in the 128-byte-swizzled layout (16-byte
// shared-memory stores: 4 wavefronts per instruction) and one thread hands the 128 x 64 box to the TMA unit, which
// writes full lines; two buffers per group, so the store of chunk c overlaps the drain of chunk c+1.  Rows past M
// are clipped by the tensor map.  Columns beyond the last full 64 go out through drain_fast.
template <bool RELU>
__device__ __forceinline__ void drain_tma_store(const ConvParams& p, const CUtensorMap* map_y, uint32_t taddr, int ncols, long long m, bool row_ok,
                                                bool tile_ok, long long m0, int n0, const float* bias_s, uint8_t* stage, int row, bool elected, int bar,
                                                int& it) {
    const uint32_t stage_u32 = smem_u32(stage);
    const int sw = row & 7;
    int c = 0;
    // `it` counts this group's chunks across tiles: buffer it & 1 was last read by store it - 2, whose reading the elected
    // thread waited for before the barrier of chunk it - 1
    for (; c + 64 <= ncols; c += 64, ++it) {
        uint8_t* srow = stage + (it & 1) * 16384 + row * 128;
#pragma unroll
        for (int h = 0; h < 64; h += 32) {
            uint32_t r[32];
            tmem_ld_x32(taddr + c + h, r);
            tmem_ld_wait();
            const float4* b4 = reinterpret_cast<const float4*>(bias_s + n0 + c + h);
#pragma unroll
            for (int q = 0; q < 4; ++q) {                            // 8 columns = one 16-byte chunk of bfloat16
                const float4 ba = b4[2 * q], bb = b4[2 * q + 1];
                float v[8] = {__uint_as_float(r[8 * q]) + ba.x,     __uint_as_float(r[8 * q + 1]) + ba.y, __uint_as_float(r[8 * q + 2]) + ba.z,
                              __uint_as_float(r[8 * q + 3]) + ba.w, __uint_as_float(r[8 * q + 4]) + bb.x, __uint_as_float(r[8 * q + 5]) + bb.y,
                              __uint_as_float(r[8 * q + 6]) + bb.z, __uint_as_float(r[8 * q + 7]) + bb.w};
                if (RELU) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[e] = fmaxf(v[e], 0.f);
                }
                *reinterpret_cast<uint4*>(srow + ((((h >> 3) + q) ^ sw) << 4)) =
                    make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
            }
        }
        fence_proxy_async_smem();                                     // these writes are read by the TMA unit
        if (elected) tma_store_wait_read();                           // the store before this one has let go of the other buffer
        group_bar_sync(bar);
        if (elected && tile_ok) {
            tma_store_2d(map_y, stage_u32 + (uint32_t)(it & 1) * 16384u, p.coff + n0 + c, (int)m0);
            tma_store_commit();
        }
    }
    if (c < ncols) {
        if (RELU) drain_fast<1>(p, taddr + c, ncols - c, m, row_ok, n0 + c, bias_s);
        else drain_fast<0>(p, taddr + c, ncols - c, m, row_ok, n0 + c, bias_s);
    }
}

// The same with a residual (bias, + residual, optional ReLU): the residual's 128 x 64 box is brought into the buffer
// by a TMA load (ring of three buffers per group: the box of chunk j+2 is requested when chunk j has been stored; the
// first two of a tile before the group waits for the tile's MMAs), each thread adds its accumulator row to its row
// of the buffer in place, and the box goes back out by a TMA store.  ncols is a multiple of 64 (host side).
__device__ __forceinline__ void residual_box_load(const CUtensorMap* map_r, uint8_t* stage, uint64_t* rfull, int it, int col, int m0) {
    const int b = it % 3;
    mbar_arrive_expect_tx(&rfull[b], 16384u);
    tma_load_2d(stage + b * 16384, map_r, &rfull[b], col, m0);
}

template <bool RELU>
__device__ __forceinline__ bool drain_tma_residual(const ConvParams& p, const CUtensorMap* map_y, const CUtensorMap* map_r, uint32_t taddr, int ncols,
                                                   long long m0, int n0, const float* bias_s, uint8_t* stage, uint64_t* rfull, int row, bool elected,
                                                   int bar, int& it, volatile int* abort_flag) {
    const uint32_t stage_u32 = smem_u32(stage);
    const int sw = row & 7;
    const int nch = ncols >> 6;
    for (int j = 0; j < nch; ++j, ++it) {
        const int b = it % 3, c = j << 6;
        if (!__all_sync(0xffffffffu, mbar_wait(&rfull[b], (uint32_t)(it / 3) & 1u, abort_flag))) return false;
        uint8_t* srow = stage + b * 16384 + row * 128;
#pragma unroll
        for (int h = 0; h < 64; h += 32) {
            uint32_t r[32];
            tmem_ld_x32(taddr + c + h, r);
            tmem_ld_wait();
            const float4* b4 = reinterpret_cast<const float4*>(bias_s + n0 + c + h);
#pragma unroll
            for (int q = 0; q < 4; ++q) {                            // 8 columns = one 16-byte chunk of bfloat16
                uint4* cell = reinterpret_cast<uint4*>(srow + ((((h >> 3) + q) ^ sw) << 4));
                const uint4 u = *cell;
                const float4 ba = b4[2 * q], bb = b4[2 * q + 1];
                float v[8] = {__uint_as_float(r[8 * q]) + ba.x + bf16_lo(u.x),     __uint_as_float(r[8 * q + 1]) + ba.y + bf16_hi(u.x),
                              __uint_as_float(r[8 * q + 2]) + ba.z + bf16_lo(u.y), __uint_as_float(r[8 * q + 3]) + ba.w + bf16_hi(u.y),
                              __uint_as_float(r[8 * q + 4]) + bb.x + bf16_lo(u.z), __uint_as_float(r[8 * q + 5]) + bb.y + bf16_hi(u.z),
                              __uint_as_float(r[8 * q + 6]) + bb.z + bf16_lo(u.w), __uint_as_float(r[8 * q + 7]) + bb.w + bf16_hi(u.w)};
                if (RELU) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[e] = fmaxf(v[e], 0.f);
                }
                *cell = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
            }
        }
        fence_proxy_async_smem();
        group_bar_sync(bar);
        if (elected) {
            tma_store_2d(map_y, stage_u32 + (uint32_t)b * 16384u, p.coff + n0 + c, (int)m0);
            tma_store_commit();
            if (j + 2 < nch) {
                asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the store of chunk it-1 has let go of buffer (it+2) % 3
                residual_box_load(map_r, stage, rfull, it + 2, n0 + c + 128, (int)m0);
            }
        }
    }
    return true;
}

// Epilogue of a layer that ends in LRN across channels without pooling (bias, ReLU, LRN, bf16 store): the thread owns
// every channel of its output pixel (one tile spans all of Cout <= 256), so the LRN window is a sliding sum over the
// accumulator row, read from TMEM in chunks of W columns with two columns of look-back (kept in registers) and two
// of look-ahead (a two-column TMEM load).  Windows of 1, 3 or 5 channels (half <= 2); beyond the row: zeros.
template <int W>
__device__ __forceinline__ void lrn_chunk(const ConvParams& p, uint32_t taddr, int c, int ncols, bool row_ok, const float* bias_s,
                                          float& pm2, float& pm1, __nv_bfloat16* yrow) {
    uint32_t r[W], nx[2] = {0u, 0u};
    if (W == 32) tmem_ld_x32(taddr + c, r); else tmem_ld_x16(taddr + c, r);
    const bool more = c + W < ncols;
    if (more) tmem_ld_x2(taddr + c + W, nx);
    tmem_ld_wait();
    const bool relu = p.flags & DR_RELU;
    float x[W + 4];
    x[0] = pm2; x[1] = pm1;
#pragma unroll
    for (int j = 0; j < W; ++j) {
        float v = __uint_as_float(r[j]) + bias_s[c + j];
        x[2 + j] = relu ? fmaxf(v, 0.f) : v;
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        float v = more ? __uint_as_float(nx[j]) + bias_s[c + W + j] : 0.f;
        x[2 + W + j] = (relu && more) ? fmaxf(v, 0.f) : v;
    }
    pm2 = x[W]; pm1 = x[W + 1];
    const bool h1 = p.lrn_half >= 1, h2 = p.lrn_half >= 2;
    // scale^(-beta), scale = k (1 + u), u = (alpha/n) ss / k.  While u < 1/32 for the whole chunk of the warp (always so
    // for the usual alpha = 1e-4) the binomial series of (1 + u)^(-beta) to u^4 is exact to float32 resolution and
    // needs no special-function unit (evaluated in ss itself, k^(-beta) folded into its coefficients); otherwise exp2/log2.
    float sq[W + 4], ss[W];
#pragma unroll
    for (int j = 0; j < W + 4; ++j) sq[j] = x[j] * x[j];
    float total = 0.f;                                        // sum of all squares: an upper bound of every window sum
#pragma unroll
    for (int j = 0; j < W; ++j) {
        float v = sq[2 + j];
        if (h1) v += sq[1 + j] + sq[3 + j];
        if (h2) v += sq[j] + sq[4 + j];
        ss[j] = v;
    }
#pragma unroll
    for (int j = 0; j < W + 4; j += 4) total += (sq[j] + sq[j + 1]) + (sq[j + 2] + sq[j + 3]);
    const bool series = !__any_sync(0xffffffffu, !(total < p.lrn_ss_max));
    const bool series2 = !__any_sync(0xffffffffu, !(total < p.lrn_ss_max2));   // two terms are exact to float32 resolution
    uint32_t o[W / 2];
#pragma unroll
    for (int j = 0; j < W; j += 2) {
        float y2[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const float s1 = ss[j + e];
            float f;
            if (series2) f = fmaf(s1, fmaf(s1, p.lrn_s2, p.lrn_s1), p.lrn_kpow);
            else if (series) f = fmaf(s1, fmaf(s1, fmaf(s1, fmaf(s1, p.lrn_s4, p.lrn_s3), p.lrn_s2), p.lrn_s1), p.lrn_kpow);
            else f = exp2f(-p.lrn_beta * log2f(fmaf(p.lrn_alpha_n, s1, p.lrn_k)));
            y2[e] = x[2 + j + e] * f;
        }
        o[j >> 1] = pack_bf16(y2[0], y2[1]);
    }
    if (row_ok) {
        uint4* y = reinterpret_cast<uint4*>(yrow + c);
#pragma unroll
        for (int q = 0; q < W / 8; ++q) y[q] = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
    }
}

__device__ __forceinline__ void drain_lrn(const ConvParams& p, uint32_t taddr, int ncols, long long m, bool row_ok, const float* bias_s) {
    __nv_bfloat16* yrow = reinterpret_cast<__nv_bfloat16*>(p.y) + m * p.ldc + p.coff;
    float pm2 = 0.f, pm1 = 0.f;
    int c = 0;
    for (; c + 32 <= ncols; c += 32) lrn_chunk<32>(p, taddr, c, ncols, row_ok, bias_s, pm2, pm1, yrow);
    if (c < ncols) lrn_chunk<16>(p, taddr, c, ncols, row_ok, bias_s, pm2, pm1, yrow);
}

// =====================================================================================
//                                   gather kernel
// =====================================================================================
constexpr int G_STAGES = 3;
constexpr int G_THREADS = 160;   // warps 0-3: producers, then epilogue; warp 4: MMA issue + TMEM owner
constexpr int G_PIPE_BYTES = G_STAGES * STAGE_BYTES;
constexpr int G_SMEM = G_PIPE_BYTES + 1024;

struct GatherShared {
    uint64_t full[G_STAGES], empty[G_STAGES], accum, drain;
    uint32_t tmem_base;
    int abort;
};

__global__ void __launch_bounds__(G_THREADS, 1) conv_umma_gather_kernel(const ConvParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ GatherShared sh;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile = blockIdx.x, n0 = blockIdx.y * p.Nt;
    const int cout16 = (p.Cout + 15) & ~15;
    const int Nj = min(p.Nt, cout16 - n0);
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < Nj) tmem_cols <<= 1;

    if (tid == 0) {
        for (int s = 0; s < G_STAGES; ++s) { mbar_init(&sh.full[s], 128); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        mbar_init(&sh.drain, 1);
        sh.abort = 0;
        fence_barrier_init();
    }
    if (warp == 4) { tmem_alloc(&sh.tmem_base, tmem_cols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort;

    const bool scalar_k = (p.Cin & 7) != 0;          // K walked as one flat index (3-channel stem)
    const int cpb = (p.Cin + 63) >> 6;               // 64-channel blocks per tap
    const int nkb = scalar_k ? (p.K + 63) >> 6 : p.k * p.k * cpb;
    const bool staged = p.flags & (DR_POOL | DR_LRN);

    if (warp < 4) {
        // ------------------------------------------------ producers: thread = tile row
        const RowPix px = row_pixel(p, tile, tid);
        const int h0 = px.ho * p.stride - p.pad, w0 = px.wo * p.stride - p.pad;
        const __nv_bfloat16* ximg = p.x + (size_t)px.n * p.H * p.W * p.Cin;
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % G_STAGES, u = kb / G_STAGES;
            if (!mbar_wait(&sh.empty[s], (u & 1) ^ 1, abort_flag)) {
                if (!*abort_flag) report_timeout(p.status, 1, tile);
                *abort_flag = 1;
                break;
            }
            uint8_t* As = smem + s * STAGE_BYTES;
            uint8_t* Bs = As + A_TILE_BYTES;
            if (!scalar_k) {
                const int tap = kb / cpb, c0 = (kb - tap * cpb) << 6;
                const int r = tap / p.k, t = tap - r * p.k;
                const int hi = h0 + r, wi = w0 + t;
                const bool ok = px.valid && hi >= 0 && hi < p.H && wi >= 0 && wi < p.W;
                const uint4* src = reinterpret_cast<const uint4*>(ximg + ((size_t)hi * p.W + wi) * p.Cin + c0);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (ok && c0 + 8 * j < p.Cin) v = __ldg(src + j);
                    *reinterpret_cast<uint4*>(As + swz(tid, j)) = v;
                }
                for (int row = tid; row < Nj; row += 128) {
                    const int jn = n0 + row;
                    const uint4* wsrc = reinterpret_cast<const uint4*>(p.w + (size_t)jn * p.K + (size_t)tap * p.Cin + c0);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (jn < p.Cout && c0 + 8 * j < p.Cin) v = __ldg(wsrc + j);
                        *reinterpret_cast<uint4*>(Bs + swz(row, j)) = v;
                    }
                }
            } else {
                const int k0 = kb << 6;
                int r = k0 / (p.k * p.Cin);
                int rem = k0 - r * p.k * p.Cin;
                int t = rem / p.Cin;
                int c = rem - t * p.Cin;
                const unsigned short* xs = reinterpret_cast<const unsigned short*>(ximg);
                for (int j = 0; j < 8; ++j) {
                    unsigned short e[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const int kg = k0 + 8 * j + q;
                        const int hi = h0 + r, wi = w0 + t;
                        unsigned short v = 0;
                        if (px.valid && kg < p.K && hi >= 0 && hi < p.H && wi >= 0 && wi < p.W)
                            v = __ldg(xs + ((size_t)hi * p.W + wi) * p.Cin + c);
                        e[q] = v;
                        if (++c == p.Cin) { c = 0; if (++t == p.k) { t = 0; ++r; } }
                    }
                    uint4 v;
                    v.x = e[0] | ((uint32_t)e[1] << 16); v.y = e[2] | ((uint32_t)e[3] << 16);
                    v.z = e[4] | ((uint32_t)e[5] << 16); v.w = e[6] | ((uint32_t)e[7] << 16);
                    *reinterpret_cast<uint4*>(As + swz(tid, j)) = v;
                }
                const unsigned short* wsh = reinterpret_cast<const unsigned short*>(p.w);
                for (int row = tid; row < Nj; row += 128) {
                    const int jn = n0 + row;
                    for (int j = 0; j < 8; ++j) {
                        unsigned short e[8];
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const int kg = k0 + 8 * j + q;
                            e[q] = (jn < p.Cout && kg < p.K) ? __ldg(wsh + (size_t)jn * p.K + kg) : (unsigned short)0;
                        }
                        uint4 v;
                        v.x = e[0] | ((uint32_t)e[1] << 16); v.y = e[2] | ((uint32_t)e[3] << 16);
                        v.z = e[4] | ((uint32_t)e[5] << 16); v.w = e[6] | ((uint32_t)e[7] << 16);
                        *reinterpret_cast<uint4*>(Bs + swz(row, j)) = v;
                    }
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(&sh.full[s]);
        }
    } else {
        // ------------------------------------------------ MMA issue: one thread
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(TILE_M, Nj);
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const int s = kb % G_STAGES, u = kb / G_STAGES;
                if (!mbar_wait(&sh.full[s], u & 1, abort_flag)) {
                    if (!*abort_flag) report_timeout(p.status, 2, tile);
                    *abort_flag = 1;
                    ok = false;
                    break;
                }
                tc_fence_after();
                int valid;
                if (scalar_k) valid = min(64, p.K - (kb << 6));
                else valid = min(64, p.Cin - ((kb % cpb) << 6));
                const uint32_t a = smem_u32(smem + s * STAGE_BYTES);
                issue_kblock(tmem, a, a + A_TILE_BYTES, idesc, (valid + 15) >> 4, kb == 0);
                umma_commit(&sh.empty[s]);
            }
            if (ok) umma_commit(&sh.accum);
            else {   // let whatever was issued finish before TMEM is released
                umma_commit(&sh.drain);
                mbar_wait(&sh.drain, 0, nullptr);
            }
        }
        __syncwarp();
    }

    // ---------------------------------------------------- epilogue: warps 0-3, thread = TMEM lane
    if (warp < 4) {
        bool ok = !*abort_flag && mbar_wait(&sh.accum, 0, abort_flag);
        ok = __all_sync(0xffffffffu, ok);            // warp-uniform: tcgen05.ld needs the whole warp
        if (!ok) {
            if (!*abort_flag) report_timeout(p.status, 3, tile);
            *abort_flag = 1;
        } else {
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16);
            if (!staged) {
                const long long m = (long long)tile * TILE_M + tid;
                drain_direct(p, taddr, Nj, m, m < p.M, n0);
            } else {
                float* stage = reinterpret_cast<float*>(smem);            // the pipeline buffers are free now
                float* stage2 = stage + (size_t)TILE_M * (p.Cout + 1);
                const int ld = p.Cout + 1;
                for (int c = 0; c < Nj; c += 16) {
                    uint32_t r[16];
                    tmem_ld_x16(taddr + c, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int ch = c + j;
                        if (ch < p.Cout) {
                            float v = __uint_as_float(r[j]) + ((p.flags & DR_BIAS) ? __ldg(p.bias + ch) : 0.f);
                            if (p.flags & DR_RELU) v = fmaxf(v, 0.f);
                            stage[tid * ld + ch] = v;
                        }
                    }
                }
                epilogue_staged<128, 1>(p, tile, stage, stage2, tid);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, tmem_cols);
}

bool conv_umma_gather_supports(const ConvParams& p) {
    if (p.Cout < 1 || p.Nt > 256) return false;
    const bool staged = p.flags & (DR_POOL | DR_LRN);
    if (staged) {
        const bool ptl = (p.flags & DR_POOL) && (p.flags & DR_LRN) && !(p.flags & DR_LRN_BEFORE_POOL);
        const size_t bytes = sizeof(float) * ((size_t)TILE_M * (p.Cout + 1) + (ptl ? (size_t)p.PH * p.PW * (p.Cout + 1) : 0));
        if (bytes > (size_t)G_PIPE_BYTES) return false;
    }
    return true;
}

int conv_umma_gather_launch(const ConvParams& p, cudaStream_t stream) {
    if (!conv_umma_gather_supports(p)) return DR_ERR_UNSUPPORTED;
    static PerDeviceFlag attr_set;
    if (!attr_set.get()) {
        if (cudaFuncSetAttribute(conv_umma_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, G_SMEM) != cudaSuccess) return DR_ERR_CUDA;
        attr_set.set();
    }
    if (p.m_tiles <= 0) return DR_OK;
    dim3 grid(p.m_tiles, p.n_blocks);
    conv_umma_gather_kernel<<<grid, G_THREADS, G_SMEM, stream>>>(p);
    count_launch();
    return launch_status();
}

// =====================================================================================
//                                     TMA kernel
// =====================================================================================
// One template, two launch shapes:
//   PAIR = false  one CTA per tile of 128 pixels x Nt channels.
//   PAIR = true   clusters of two CTAs act as one MMA unit (tcgen05 cta_group::2): a pair tile is
//       256 pixels x Nt channels; each CTA loads its own 128 activation rows and HALF of the filter
//       tile, the even CTA issues M=256 MMAs that read both shared memories, and each CTA keeps and
//       drains its own 128 accumulator rows.  Per SM and k-block this moves 16 KB + Nt*64 B through
//       shared memory instead of 16 KB + Nt*128 B.  TMA loads of both CTAs report to the even CTA's
//       `full` barrier; the even CTA's commits arrive on `empty` / `tfull` of both CTAs; epilogue
//       warps of both CTAs arrive on the even CTA's `tempty`.  No multicast loads.
// The producer and the MMA issuer are single threads whose loop bodies sit on the critical path
// (a lone thread issues dependent instructions several cycles apart), so both loops are kept to a
// few dozen instructions: nested tap / channel-block loops instead of divisions, barrier and
// stage addresses advanced incrementally, descriptors assembled from 32-bit halves.
constexpr int T_MAX_STAGES = 12;  // stage = A tile (16 KB) + B tile; as many as fit (DUAL: two rings of half as many)
constexpr int T_THREADS = 384;    // warp 0: TMA producer, warp 1: MMA issue + TMEM owner, warps 2-5 / 6-9: two epilogue groups,
                                  // warp 10: second MMA issuer, warp 11: second producer (DUAL)
constexpr int T_MMA2_WARP = 10;
constexpr int T_PROD2_WARP = 11;
constexpr int T_BIAS_MAX = 2048;  // channels of the shared-memory bias copy (lean epilogue)
constexpr int T_SMEM_MAX = 227 * 1024 - 9216;   // dynamic part; the static part holds barriers and the bias copy
constexpr int T_ACC_COLS = 256;   // columns per accumulator buffer; two buffers = all 512 TMEM columns

struct TmaShared {
    uint64_t full[T_MAX_STAGES], empty[T_MAX_STAGES], tfull[4], tempty[4];
    uint64_t rfull[2][3];      // residual boxes of the TMA epilogue: per epilogue group, ring of three
    uint32_t tmem_base;
    int abort;
};

// a_mode 0: activations as a plain [M][Cin] matrix (1x1, stride 1, pad 0): 2-D tiled load.
// a_mode 1: im2col load.
// WIDE: a tile carries TWO n-blocks of Nt columns (accumulators at TMEM columns 0 and 256): the activation tile
// is loaded once and multiplied against both filter sub-tiles, which halves the activation traffic of layers
// with more than 256 output channels.  All 512 TMEM columns then belong to one tile: the MMAs of the next tile
// start when both epilogue groups (group g drains sub-block g) have emptied it.
// DUAL: the CTA runs TWO tile pipelines side by side, each with its own producer warp, MMA-issuing warp, epilogue group,
// ring of stages (half of the shared memory) and accumulators (half of TMEM: two of up to 128 columns, or one of up to
// 256).  One thread hands the tensor core an MMA about every 64 clocks at best and pays the stage hand-over (barrier
// probe, fence, commit) on top, which MMAs of fewer than 256 columns do not cover: with two issuers working on different
// tiles the tensor core stays fed, and one pipeline's epilogue runs under the other's MMAs.  (Two CTAs per SM would do the
// same, but a kernel that uses tcgen05 is given an SM to itself.)
template <bool PAIR, int KPB, bool WIDE, bool DUAL>
__global__ void __launch_bounds__(T_THREADS, 1)
conv_umma_tma_kernel(const ConvParams p, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_r, const int a_mode, const int stages,
                     const int sub_bytes, const int ep_stage_off) {
    constexpr int kpb = KPB;
    constexpr int NTHREADS = T_THREADS;
    constexpr int BIAS_MAX = T_BIAS_MAX;
    constexpr uint32_t TMEM_COLS = 2 * T_ACC_COLS;
    // accumulator buffers of a tile pipeline and their width in TMEM columns (WIDE: the two sub-blocks of one tile instead)
    const int nacc = DUAL ? (p.Nt <= 128 ? 2 : 1) : 2;
    const uint32_t acc_cols = DUAL ? (uint32_t)(T_ACC_COLS / nacc) : (uint32_t)T_ACC_COLS;
    // a pipeline stage holds `kpb` k-blocks (sub-stages of sub_bytes = A tile + B tile): one barrier
    // round trip then covers kpb * 4 MMAs, which keeps the issuing thread ahead of the tensor pipe
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ TmaShared sh;
    __shared__ __align__(16) float bias_s[BIAS_MAX];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int stage_bytes = kpb * sub_bytes;
    // lean epilogue: bias, ReLU, residual (+ReLU); bf16 out, every 16-column chunk inside Cout, aligned slice.
    // (ReLU before a residual add is the one order it does not take.)
    const bool lean = !(p.flags & DR_OUT_F32) && !((p.flags & DR_RESIDUAL) && (p.flags & DR_RELU)) && (p.Cout & 15) == 0 &&
                      p.Cout <= BIAS_MAX && (p.ldc & 7) == 0 && (p.coff & 7) == 0;
    const bool lrn_ep = (p.flags & DR_LRN) != 0;                // host side guarantees: no pooling, one n-block, lean preconditions
    const int lean_mode = (p.flags & DR_RESIDUAL) ? ((p.flags & DR_RELU_AFTER_RESIDUAL) ? 3 : 2) : ((p.flags & DR_RELU) ? 1 : 0);
    if (lean)
        for (int i = tid; i < p.Cout; i += NTHREADS) bias_s[i] = (p.flags & DR_BIAS) ? p.bias[i] : 0.f;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;        // 0 issues the MMAs
    const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int nunits = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

    if (tid == 0) {
        for (int s = 0; s < (DUAL ? 2 * stages : stages); ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], WIDE ? 2 : 1); }   // WIDE: both issuers commit
        for (int a = 0; a < 4; ++a) { mbar_init(&sh.tfull[a], WIDE ? 2 : 1); mbar_init(&sh.tempty[a], (PAIR ? 8 : 4) * (WIDE ? 2 : 1)); }
        for (int a = 0; a < 6; ++a) mbar_init(&sh.rfull[a / 3][a % 3], 1);
        sh.abort = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
    }
    if (warp == 1) {
        if (PAIR) { tmem_alloc_pair(&sh.tmem_base, TMEM_COLS); tmem_relinquish_pair(); }
        else { tmem_alloc(&sh.tmem_base, TMEM_COLS); tmem_relinquish(); }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();                               // both CTAs' barriers exist before any remote arrive
    tc_fence_after();
    grid_launch_dependents();                                   // a kernel launched behind this one with programmatic serialization may be scheduled
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort;

    const int cpb = (p.Cin + 63) >> 6;
    const int nkb = p.k * p.k * cpb;
    const int m_units = PAIR ? (p.m_tiles + 1) >> 1 : p.m_tiles;
    const int total = m_units * p.n_blocks;
    const int cout16 = (p.Cout + 15) & ~15;
    const int hw = p.Ho * p.Wo;
    const int tile_n = WIDE ? 2 * p.Nt : p.Nt;                 // output channels per tile
    const uint32_t b_sub_bytes = WIDE ? (uint32_t)(sub_bytes - A_TILE_BYTES) >> 1 : 0u;   // one filter sub-tile
    const uint32_t smem_base = smem_u32(smem);

    if (warp == 0 || warp == T_PROD2_WARP) {
        if (lane == 0 && (warp == 0 || DUAL)) {
            // -------------------------------------------- TMA producer (DUAL: of pipeline g, ring g)
            const int g = warp == 0 ? 0 : 1;
            const uint32_t full0 = smem_u32(&sh.full[g * stages]), empty0 = smem_u32(&sh.empty[g * stages]);
            const uint32_t ring_base = smem_base + (uint32_t)(g * stages) * (uint32_t)stage_bytes;
            if (p.pdl_wait) grid_dependency_wait();            // the kernel before this one has written the activations
            const uint32_t cta_tx = A_TILE_BYTES + (uint32_t)(PAIR ? p.Nt >> 1 : p.Nt) * 128 * (WIDE ? 2 : 1);
            const uint32_t full_mask = PAIR ? PEER_BIT_MASK : 0xFFFFFFFFu;   // pair: bytes are reported to the even CTA
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            uint32_t ready = mbar_test_u32(empty0, 1);
            for (int t = DUAL ? unit + g * nunits : unit; t < total && ok; t += DUAL ? 2 * nunits : nunits) {
                const int nb = t / m_units, mu = t - nb * m_units;
                const int n0 = nb * tile_n;
                int mt = PAIR ? 2 * mu + (int)rank : mu;
                if (mt >= p.m_tiles) mt = p.m_tiles - 1;   // odd tile count: the peer recomputes the last tile, stores nothing
                const long long m0 = (long long)mt * TILE_M;
                const int img = (int)(m0 / hw);
                const int rem = (int)(m0 - (long long)img * hw);
                const int ho = rem / p.Wo, wo = rem - ho * p.Wo;
                const int hb = ho * p.stride - p.pad, wb = wo * p.stride - p.pad;
                const int brow = PAIR ? n0 + (int)rank * (min(p.Nt, cout16 - n0) >> 1) : n0;
                // second sub-block (WIDE); may be narrower than the first, or empty (its rows are then past the tensor: zero fill)
                const int brow1 = PAIR ? n0 + p.Nt + (int)rank * (max(0, min(p.Nt, cout16 - n0 - p.Nt)) >> 1) : n0 + p.Nt;
                int r = 0, tt = 0, tap = 0, c0 = 0;
                for (int remaining = nkb; remaining > 0;) {
                    const int nk = remaining < kpb ? remaining : kpb;
                    if (!ready && !mbar_wait_slow_u32(empty0 + 8 * s, ph ^ 1, abort_flag)) {
                        if (!*abort_flag) report_timeout(p.status, 11, t);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    int s2 = s + 1;
                    uint32_t ph2 = ph;
                    if (s2 == stages) { s2 = 0; ph2 ^= 1; }
                    ready = mbar_test_u32(empty0 + 8 * s2, ph2 ^ 1);      // probe the next slot while this one is filled
                    uint32_t a_dst = ring_base + (uint32_t)s * (uint32_t)stage_bytes;
                    const uint32_t fb = (full0 + 8 * s) & full_mask;
                    if (!PAIR) mbar_expect_tx_u32(fb, (uint32_t)nk * cta_tx);
                    else if (rank == 0) mbar_expect_tx_u32(fb, 2u * (uint32_t)nk * cta_tx);
#pragma unroll
                    for (int j = 0; j < KPB; ++j, a_dst += (uint32_t)sub_bytes) {
                        const uint32_t en = j < nk ? 1u : 0u;
                        if (a_mode == 0) tma_load_2d_u32<PAIR>(a_dst, &map_a, fb, c0, (int)m0, en);
                        else tma_load_im2col_4d_u32<PAIR>(a_dst, &map_a, fb, c0, wb, hb, img, (uint16_t)tt, (uint16_t)r, en);
                        tma_load_3d_u32<PAIR>(a_dst + A_TILE_BYTES, &map_b, fb, c0, tap, brow, en);
                        if (WIDE) tma_load_3d_u32<PAIR>(a_dst + A_TILE_BYTES + b_sub_bytes, &map_b, fb, c0, tap, brow1, en);
                        c0 += 64;
                        const bool wrap_c = c0 >= p.Cin;
                        c0 = wrap_c ? 0 : c0;
                        tap += wrap_c ? 1 : 0;
                        tt += wrap_c ? 1 : 0;
                        const bool wrap_t = tt == p.k;
                        tt = wrap_t ? 0 : tt;
                        r += wrap_t ? 1 : 0;
                    }
                    remaining -= nk;
                    s = s2;
                    ph = ph2;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == T_MMA2_WARP) {
        if (rank == 0 && (warp == 1 || WIDE || DUAL)) {
            // -------------------------------------------- MMA issue.  The whole warp walks the loop (so that the
            // addresses and descriptors are warp-uniform values); lane 0 alone issues the MMAs and commits.
            // One thread hands the tensor core an MMA about every 64 clocks at best and pays the stage hand-over (barrier
            // probe, fence, commit) on top, which MMAs of fewer than 256 columns do not cover.  The two sub-blocks of a wide
            // tile have accumulators of their own, so each gets an issuing warp: both wait for the same stage, each
            // multiplies the shared activation tile by its filter sub-tile, and a stage is free when both have committed.
            const int sub = (WIDE && warp != 1) ? 1 : 0;          // WIDE: the sub-block this warp issues
            const int g = (DUAL && warp != 1) ? 1 : 0;            // DUAL: the pipeline this warp issues
            const uint32_t full0 = smem_u32(&sh.full[g * stages]), empty0 = smem_u32(&sh.empty[g * stages]);
            const uint32_t ring_base = smem_base + (uint32_t)(g * stages) * (uint32_t)stage_bytes;
            const uint32_t el = lane == 0 ? 1u : 0u;
            const uint32_t tfull0 = smem_u32(&sh.tfull[0]), tempty0 = smem_u32(&sh.tempty[0]);
            const int last_nk16 = ((p.Cin - ((cpb - 1) << 6)) + 15) >> 4;
            int s = 0, it = 0;
            uint32_t ph = 0;
            bool ok = true;
            bool ready = __all_sync(0xffffffffu, mbar_test_u32(full0, 0) != 0);
            for (int t = DUAL ? unit + g * nunits : unit; t < total && ok; t += DUAL ? 2 * nunits : nunits, ++it) {
                const int nb = t / m_units;
                const int Nj = min(p.Nt, cout16 - nb * tile_n - (WIDE ? sub * p.Nt : 0));   // this issuer's (sub-)block; <= 0: none
                const uint32_t idesc = make_idesc_bf16(PAIR ? 2 * TILE_M : TILE_M, Nj > 0 ? Nj : 16);
                const uint32_t elj = Nj > 0 ? el : 0u;
                // accumulator buffer of this tile: its hand-over barriers, their parity, its TMEM column
                const int bsel = WIDE ? 0 : (nacc == 2 ? (it & 1) : 0), au = WIDE ? it : (nacc == 2 ? (it >> 1) : it);
                const int acc = 2 * g + bsel;
                if (!__all_sync(0xffffffffu, mbar_wait_u32(tempty0 + 8 * acc, (au & 1) ^ 1, abort_flag))) {
                    if (el && !*abort_flag) report_timeout(p.status, 12, t);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d = tmem + (WIDE ? (uint32_t)sub * (uint32_t)T_ACC_COLS : (uint32_t)(g * T_ACC_COLS) + (uint32_t)bsel * acc_cols);
                const uint32_t b_off = (uint32_t)A_TILE_BYTES + (WIDE ? (uint32_t)sub * b_sub_bytes : 0u);
                uint32_t accum = 0;
                int cc = 0;
                for (int remaining = nkb; remaining > 0;) {
                    const int nk = remaining < kpb ? remaining : kpb;
                    if (!ready && !__all_sync(0xffffffffu, mbar_wait_slow_u32(full0 + 8 * s, ph, abort_flag))) {
                        if (el && !*abort_flag) report_timeout(p.status, 13, t);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    int s2 = s + 1;
                    uint32_t ph2 = ph;
                    if (s2 == stages) { s2 = 0; ph2 ^= 1; }
                    ready = __all_sync(0xffffffffu, mbar_test_u32(full0 + 8 * s2, ph2) != 0);   // probe the next slot while this one is issued
                    tc_fence_after();
                    uint32_t a = ring_base + (uint32_t)s * (uint32_t)stage_bytes;
#pragma unroll
                    for (int j = 0; j < KPB; ++j, a += (uint32_t)sub_bytes) {
                        const uint32_t alo = sdesc_lo(a), blo = sdesc_lo(a + b_off);
                        const int nk16 = j < nk ? ((cc == cpb - 1) ? last_nk16 : 4) : 0;    // 0: nothing in this sub-stage
                        cc = (cc + 1 == cpb) ? 0 : cc + 1;
                        umma_bf16_lo<PAIR>(d, alo, blo, idesc, accum, (nk16 > 0) & elj);
                        accum = 1;
                        umma_bf16_lo<PAIR>(d, alo + 2, blo + 2, idesc, 1u, (nk16 > 1) & elj);
                        umma_bf16_lo<PAIR>(d, alo + 4, blo + 4, idesc, 1u, (nk16 > 2) & elj);
                        umma_bf16_lo<PAIR>(d, alo + 6, blo + 6, idesc, 1u, (nk16 > 3) & elj);
                    }
                    if (el) umma_commit_u32<PAIR>(empty0 + 8 * s);
                    remaining -= nk;
                    s = s2;
                    ph = ph2;
                }
                if (ok && el) umma_commit_u32<PAIR>(tfull0 + 8 * acc);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue: two groups of four warps; group g drains
        // accumulator buffer g, i.e. every other tile of this CTA.  TMEM lane quarter = warp % 4.
        const int g = (warp - 2) >> 2;
        const int q = warp & 3;
        const int row = q * 32 + lane;
        if (p.pdl_wait && (p.flags & DR_RESIDUAL)) grid_dependency_wait();   // the residual may be that kernel's output too
        int ep_it = 0;                                           // chunks this group has handed to the TMA unit so far
        // tiles of this group: WIDE every tile (sub-block g); else every other tile of the CTA (DUAL: those are pipeline g's)
        for (int t = WIDE ? unit : unit + g * nunits, au = 0; t < total; t += WIDE ? nunits : 2 * nunits, ++au) {
            // accumulator buffer of this tile, the parity of its hand-over barriers, its TMEM column
            const int bsel = (DUAL && nacc == 2) ? (au & 1) : 0;
            const int ab = WIDE ? 0 : (DUAL ? 2 * g + bsel : g);
            const uint32_t par = (DUAL && nacc == 2) ? (uint32_t)(au >> 1) & 1u : (uint32_t)au & 1u;
            const int nb = t / m_units, mu = t - nb * m_units;
            const int n0 = WIDE ? nb * tile_n + g * p.Nt : nb * p.Nt;      // WIDE: group g drains sub-block g of every tile
            const int Nj = min(p.Nt, cout16 - n0);                         // WIDE: may be <= 0 (no second sub-block)
            const int mt = PAIR ? 2 * mu + (int)rank : mu;
            const bool res_tma = lean && ep_stage_off > 0 && lean_mode >= 2 && mt < p.m_tiles;
            if (res_tma && ((warp - 2) & 3) == 0 && lane == 0) {
                // this tile's first two residual boxes, requested before the wait for its MMAs
                uint8_t* st = smem + ep_stage_off + g * 49152;
                residual_box_load(&map_r, st, sh.rfull[g], ep_it, n0, (int)((long long)mt * TILE_M));
                if (Nj > 64) residual_box_load(&map_r, st, sh.rfull[g], ep_it + 1, n0 + 64, (int)((long long)mt * TILE_M));
            }
            const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.tfull[ab], par, abort_flag));
            if (!ok) {
                if (!*abort_flag) report_timeout(p.status, 14, t);
                *abort_flag = 1;
                break;
            }
            tc_fence_after();
            const long long m = (long long)mt * TILE_M + row;
            const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g * T_ACC_COLS) + (uint32_t)bsel * acc_cols;
            const bool row_ok = mt < p.m_tiles && m < p.M;
            if (WIDE && Nj <= 0) {
                // nothing to drain
            } else if (lrn_ep) {
                drain_lrn(p, taddr, Nj, m, row_ok, bias_s);
            } else if (lean && ep_stage_off > 0 && lean_mode >= 2) {
                if (res_tma) {
                    uint8_t* st = smem + ep_stage_off + g * 49152;
                    const bool elected = ((warp - 2) & 3) == 0 && lane == 0;
                    const long long m0 = (long long)mt * TILE_M;
                    const bool done = lean_mode == 3
                        ? drain_tma_residual<true>(p, &map_y, &map_r, taddr, Nj, m0, n0, bias_s, st, sh.rfull[g], row, elected, 1 + g, ep_it, abort_flag)
                        : drain_tma_residual<false>(p, &map_y, &map_r, taddr, Nj, m0, n0, bias_s, st, sh.rfull[g], row, elected, 1 + g, ep_it, abort_flag);
                    if (!done) {
                        if (!*abort_flag) report_timeout(p.status, 15, t);
                        *abort_flag = 1;
                        break;
                    }
                }
            } else if (lean && ep_stage_off > 0 && lean_mode < 2) {
                uint8_t* st = smem + ep_stage_off + g * 32768;
                const bool elected = ((warp - 2) & 3) == 0 && lane == 0;
                const long long m0 = (long long)mt * TILE_M;
                if (lean_mode == 1) drain_tma_store<true>(p, &map_y, taddr, Nj, m, row_ok, mt < p.m_tiles, m0, n0, bias_s, st, row, elected, 1 + g, ep_it);
                else drain_tma_store<false>(p, &map_y, taddr, Nj, m, row_ok, mt < p.m_tiles, m0, n0, bias_s, st, row, elected, 1 + g, ep_it);
            } else if (lean) {
                if (lean_mode == 1) drain_fast<1>(p, taddr, Nj, m, row_ok, n0, bias_s);
                else if (lean_mode == 3) drain_fast<3>(p, taddr, Nj, m, row_ok, n0, bias_s);
                else if (lean_mode == 0) drain_fast<0>(p, taddr, Nj, m, row_ok, n0, bias_s);
                else drain_fast<2>(p, taddr, Nj, m, row_ok, n0, bias_s);
            } else {
                drain_direct(p, taddr, Nj, m, row_ok, n0);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (PAIR) mbar_arrive_leader(&sh.tempty[ab]);
                else mbar_arrive(&sh.tempty[ab]);
            }
        }
    }
    if (ep_stage_off > 0 && warp >= 2 && ((warp - 2) & 3) == 0 && lane == 0) tma_store_wait_all();   // TMA stores of this thread have landed
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {   // give copies and MMAs still in flight time to land before shared memory and TMEM go away
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) {}
        __syncthreads();
    }
    if (PAIR) cluster_sync_all();                               // neither CTA leaves while the other may still signal it
    if (p.overlap_prev) grid_dependency_wait();                 // launched ahead of the previous kernel's end: do not finish before it has
    if (warp == 1) {
        if (PAIR) tmem_dealloc_pair(tmem, TMEM_COLS);
        else tmem_dealloc(tmem, TMEM_COLS);
    }
}

// ---- host: tensor maps ------------------------------------------------------------------
// Tensor maps of one convolution for the TMA kernels.  A: the activations, as a plain [M][Cin] matrix for
// 1x1 / stride 1 / pad 0 layers (*a_mode = 0, 2-D tiled boxes of 128 rows x 64 channels) and in im2col mode
// otherwise (*a_mode = 1: 128 output pixels x 64 channels of one filter tap per load).  B: the filters as
// (Cin, taps, Cout) with boxes of 64 channels x 1 tap x b_box_rows filters.
int encode_conv_maps(const ConvParams& p, int b_box_rows, CUtensorMap* map_a, CUtensorMap* map_b, int* a_mode) {
    const int st = encode_input_map(p, map_a, a_mode);
    if (st != DR_OK) return st;
    const cuuint64_t dims[3] = {(cuuint64_t)p.Cin, (cuuint64_t)(p.k * p.k), (cuuint64_t)p.Cout};
    const cuuint64_t strides[2] = {(cuuint64_t)p.Cin * 2, (cuuint64_t)p.K * 2};
    const cuuint32_t box[3] = {64, 1, (cuuint32_t)b_box_rows};
    return tmap_tiled(map_b, 3, p.w, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

// A [rows][cols] bf16 matrix with row pitch ld (elements) in boxes of box_rows rows x 64 columns, 128-byte swizzle.
int encode_rows_map(const void* ptr, long long rows, int cols, int ld, CUtensorMap* map, int box_rows) {
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    return tmap_tiled(map, 2, ptr, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

// The input-side map alone (see encode_conv_maps).
int encode_input_map(const ConvParams& p, CUtensorMap* map_a, int* a_mode, int box_rows) {
    *a_mode = (p.k == 1 && p.stride == 1 && p.pad == 0) ? 0 : 1;
    if (*a_mode == 0) {
        const cuuint64_t dims[2] = {(cuuint64_t)p.Cin, (cuuint64_t)p.M};
        const cuuint64_t strides[1] = {(cuuint64_t)p.Cin * 2};
        const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
        return tmap_tiled(map_a, 2, p.x, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
    }
    const cuuint64_t dims[4] = {(cuuint64_t)p.Cin, (cuuint64_t)p.W, (cuuint64_t)p.H, (cuuint64_t)p.B};
    const cuuint64_t strides[3] = {(cuuint64_t)p.Cin * 2, (cuuint64_t)p.W * p.Cin * 2, (cuuint64_t)p.H * p.W * p.Cin * 2};
    // bounding box of the positions the filter's first tap visits: [-pad, extent + pad - k]
    const int lower[2] = {-p.pad, -p.pad};
    const int upper[2] = {p.pad - (p.k - 1), p.pad - (p.k - 1)};
    return tmap_im2col(map_a, p.x, dims, strides, lower, upper, 64, (unsigned)box_rows, (unsigned)p.stride, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

bool conv_umma_tma_supports(const ConvParams& p) {
    if (p.flags & DR_POOL) return false;              // pooling epilogues live in the patch / stem / gather kernels
    if (p.flags & DR_LRN) {
        // LRN without pooling: the in-register sliding window of drain_lrn, one tile across all output channels
        if (p.flags & (DR_RESIDUAL | DR_OUT_F32)) return false;
        if (p.n_blocks != 1 || (p.Cout & 15) || p.Cout > 256 || p.lrn_half > 2 || !(p.lrn_k > 0.f) || p.lrn_alpha_n < 0.f || (p.ldc & 7) || (p.coff & 7) || p.argmax) return false;
    }
    if (p.patch) return false;
    if ((p.Cin & 7) || p.Cin < 64) return false;      // TMA strides are 16-byte multiples; 128-byte rows
    if (p.Nt > 256) return false;
    if (p.k > 255 || p.M <= 0) return false;
    if (p.M > 0x7fffffffLL) return false;
    return true;
}

// Pipeline shape: k-blocks per stage (kpb) and number of stages within `budget` bytes.  Measured on B200: tiles of at
// least 208 columns run best with one k-block per barrier round trip, narrower ones with two (their MMAs are short, so
// the round trip has to cover more of them); never more than the layer has.
static void pick_pipeline(int budget, int sub_bytes, int nkb, int nt, int* kpb, int* stages) {
    int k = tunable("DR_TMA_KPB", 0);
    if (k <= 0) k = nt >= 208 ? 1 : 2;
    if (k >= 4) k = 4; else if (k == 3) k = 2;          // instantiated: 1, 2, 4
    while (k > 1 && (k > nkb || budget / (k * sub_bytes) < 3)) k >>= 1;
    int st = budget / (k * sub_bytes);
    if (st > T_MAX_STAGES) st = T_MAX_STAGES;
    const int forced = tunable("DR_TMA_STAGES", 0);
    if (forced >= 2 && forced < st) st = forced;
    *kpb = k;
    *stages = st;
}

// The TMA epilogue pays where the output is large against K (few k-blocks per tile: the pipeline then needs little
// shared memory, and the row-per-thread stores would bound the layer): bias / ReLU and residual epilogues of layers
// with at most 4 k-blocks (residual: n-blocks that are multiples of 64 columns).  Returns the shared memory it needs
// (0: not used).  map_y: y as a [M][coff + Cout] matrix with row pitch ldc; map_r: the residual as [M][Cout]; boxes of
// 128 rows x 64 columns, 128-byte swizzle.
static int tma_epilogue_bytes(const ConvParams& p, bool pair_or_wide, CUtensorMap* map_y, CUtensorMap* map_r) {
    const int ep_pref = tunable("DR_TMA_STORE_EP", 1);          // 0: never, 1: where it pays, 2: wherever the shape allows
    if (ep_pref == 0 || pair_or_wide) return 0;
    if (ep_pref == 1 && p.m_tiles < num_sms()) return 0;        // less than one tile per SM: latency matters, not store bandwidth
    if (p.flags & (DR_OUT_F32 | DR_LRN)) return 0;
    if ((p.flags & DR_RESIDUAL) && (p.flags & DR_RELU)) return 0;
    if ((p.Cout & 15) || p.Cout > T_BIAS_MAX || (p.ldc & 7) || (p.coff & 7) || p.Nt < 64) return 0;
    const int nkb = p.k * p.k * ((p.Cin + 63) / 64);
    const bool res = (p.flags & DR_RESIDUAL) != 0;
    // measured (ResNet-50 at batch 128, GoogLeNet at 256): a gain up to 4 k-blocks with a residual or with at least 256
    // output channels, up to 2 k-blocks otherwise; beyond that the lost pipeline stages cost more than the stores
    if (res ? ((p.Nt & 63) || (p.Cout & 63)) : false) return 0;
    if (ep_pref == 1 && (res ? nkb > 4 : (nkb > 4 || (nkb > 2 && p.Cout < 256)))) return 0;
    const cuuint32_t box[2] = {64, TILE_M};
    {
        const cuuint64_t dims[2] = {(cuuint64_t)(p.coff + p.Cout), (cuuint64_t)p.M};
        const cuuint64_t strides[1] = {(cuuint64_t)p.ldc * 2};
        if (tmap_tiled(map_y, 2, p.y, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE) != DR_OK) return 0;
    }
    if (res) {
        const cuuint64_t dims[2] = {(cuuint64_t)p.Cout, (cuuint64_t)p.M};
        const cuuint64_t strides[1] = {(cuuint64_t)p.Cout * 2};
        if (tmap_tiled(map_r, 2, p.residual, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B) != DR_OK) return 0;
    }
    return res ? 2 * 3 * 16384 : 2 * 2 * 16384;                  // per epilogue group: three / two 16 KB buffers
}

// Tile shape of a layer on the TMA kernel: CTA pairs or single CTAs, and whether a tile carries two n-blocks that
// share the activation tile (then p->Nt / p->n_blocks are replaced by the wide tiling).
void conv_umma_tma_shape(ConvParams* pp, bool* use_pair_out, bool* wide_out) {
    ConvParams& p = *pp;
    // CTA pairs pay off where the MMAs dominate: long K, or a spatial filter with K >= 512 (measured: +12 % on the
    // 3x3 layers, -20 % on the 1x1 reducers)
    const int pair_pref = tunable("DR_TMA_PAIR", -1);
    const bool use_pair = pair_pref >= 0 ? pair_pref != 0 : ((p.K >= 1024 || (p.k > 1 && p.K >= 512)) && p.m_tiles >= 2);
    // More than 256 output channels and a long K: wide tiles (two n-blocks per tile sharing the activation tile) of
    // near-equal sub-blocks, e.g. 288 -> one tile of 144 + 144, unless the coarser tiles cost more in rounds of the
    // persistent grid than the shared activation tile saves (measured: 5 to 9 % on the merged 5x5 layers of stage 4;
    // short-K layers lose more to the epilogue, which wide tiles do not overlap with the next tile's MMAs; 3x3 layers of
    // 27 k-blocks still gain: 4d / 4e 3x3 at batch 256, 67.6 -> 57.4 and 68.0 -> 61.4 us).
    const int cout16_ = (p.Cout + 15) / 16 * 16;
    const int wide_pref = tunable("DR_TMA_WIDE", -1);
    bool wide = false;
    int nt_w = 0, n_wide = 0;
    if (cout16_ > 32) {
        n_wide = (cout16_ + 511) / 512;
        nt_w = ((cout16_ + 2 * n_wide - 1) / (2 * n_wide) + 15) / 16 * 16;
        const long long capacity = use_pair ? num_sms() / 2 : num_sms();
        const long long m_units = use_pair ? (p.m_tiles + 1) / 2 : p.m_tiles;
        const long long cost_n = (m_units * p.n_blocks + capacity - 1) / capacity * p.Nt;
        const long long cost_w = (m_units * n_wide + capacity - 1) / capacity * 2 * nt_w;
        const int nkb_ = p.k * p.k * ((p.Cin + 63) / 64);
        wide = wide_pref >= 0 ? wide_pref != 0 : (cout16_ > 256 && (nkb_ >= 48 || (p.k > 1 && nkb_ >= 24)) && cost_w * 95 <= cost_n * 100);
        if (p.flags & DR_LRN) wide = false;                      // the LRN window runs along one accumulator row
    }
    if (wide) {
        p.Nt = nt_w;
        p.n_blocks = n_wide;
    }
    *use_pair_out = use_pair;
    *wide_out = wide;
}

namespace {
struct TmaLaunch {
    const ConvParams* p;
    const CUtensorMap *map_a, *map_b, *map_y, *map_r;
    int a_mode, stages, sub_bytes, ep_off, smem_bytes, units;
    cudaStream_t stream;
};

// One instantiation: sets its attributes once per device, asks how many clusters fit, launches.
template <bool PAIR, int KPB, bool WIDE, bool DUAL>
int launch_variant(const TmaLaunch& L) {
    static bool ready[64] = {false};
    static int capacity[64] = {0};                               // resident CTAs (single) / clusters (pairs)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DR_ERR_CUDA;
    auto kern = conv_umma_tma_kernel<PAIR, KPB, WIDE, DUAL>;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (PAIR) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = 2; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.blockDim = dim3(T_THREADS); cfg.stream = L.stream; cfg.attrs = attr;
    if (!ready[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, T_SMEM_MAX) != cudaSuccess) return DR_ERR_CUDA;
        if (PAIR) {
            cfg.gridDim = dim3(2 * num_sms());
            cfg.dynamicSmemBytes = (size_t)T_SMEM_MAX;
            cfg.numAttrs = na;
            if (cudaOccupancyMaxActiveClusters(&capacity[dev], kern, &cfg) != cudaSuccess || capacity[dev] < 1) return DR_ERR_CUDA;
        } else {
            capacity[dev] = num_sms();
        }
        ready[dev] = true;
    }
    const int n = L.units < capacity[dev] ? L.units : capacity[dev];
    cfg.gridDim = dim3((unsigned)(PAIR ? 2 * n : n));
    cfg.dynamicSmemBytes = (size_t)L.smem_bytes;
    if (L.p->overlap_prev || L.p->pdl_wait) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.numAttrs = na;
    if (cudaLaunchKernelEx(&cfg, kern, *L.p, *L.map_a, *L.map_b, *L.map_y, *L.map_r, L.a_mode, L.stages, L.sub_bytes, L.ep_off) != cudaSuccess) {
        (void)cudaGetLastError();
        return DR_ERR_CUDA;
    }
    count_launch();
    return launch_status();
}

template <bool PAIR, bool DUAL>
int launch_kpb(const TmaLaunch& L, int kpb) {
    if (kpb == 4) return launch_variant<PAIR, 4, false, DUAL>(L);
    if (kpb == 2) return launch_variant<PAIR, 2, false, DUAL>(L);
    return launch_variant<PAIR, 1, false, DUAL>(L);
}
}  // namespace

// Whether the layer runs as two tile pipelines per CTA (DUAL), and its pipeline shape then: tiles without the TMA-store
// epilogue, without LRN and without a second sub-block, enough of them that CTAs have more than one, and room for at
// least three stages in each of the two rings.
static bool pick_dual(const ConvParams& p, bool use_pair, bool wide, int ep_bytes, int sub_bytes, int nkb, int total, int* kpb, int* stages) {
    const int pref = tunable("DR_TMA_DUAL", -1);
    if (pref == 0 || wide || ep_bytes || (p.flags & DR_LRN)) return false;
    const int capacity = use_pair ? num_sms() / 2 : num_sms();
    if (pref < 0 && total <= capacity) return false;
    // Measured at batch 256 (GoogLeNet): a gain where one issuer cannot keep up with its MMAs and the reduction is long
    // enough to matter, i.e. tiles of at most 224 columns over at least 48 k-blocks (3a / 5a / 5b merged 5x5: 250 -> 216,
    // 211 -> 174, 231 -> 204 us) and tiles of at most 128 columns (two accumulators per pipeline); a loss on tiles of
    // 240 and 256 columns, which one issuer keeps busy (4c / 4d merged 5x5: 224 -> 254, 219 -> 246 us), and on short
    // reductions with wide tiles, where each ring's three stages cover less of the load latency (3b 3x3: 92 -> 113 us), and
    // on 1x1 layers (4a reducer: 22.5 -> 24.6 us).
    // Spatial filters over 64-channel tiles (ResNet-50 stage 2, 3x3 with 64 output channels, 9 k-blocks): 78 -> 62 us.
    if (pref < 0 && !((p.Nt <= 224 && nkb >= 48) || (p.Nt <= 128 && nkb >= 16) || (p.Nt <= 128 && p.k > 1 && nkb >= 8))) return false;
    int k = tunable("DR_TMA_KPB", 0);
    if (k <= 0) k = 1;
    if (k >= 4) k = 4; else if (k == 3) k = 2;
    const int budget = (T_SMEM_MAX - 1024) / 2;
    while (k > 1 && (k > nkb || budget / (k * sub_bytes) < 3)) k >>= 1;
    int st = budget / (k * sub_bytes);
    if (st > T_MAX_STAGES / 2) st = T_MAX_STAGES / 2;
    if (st < 3) return false;
    *kpb = k;
    *stages = st;
    return true;
}

int conv_umma_tma_launch(const ConvParams& p_in, cudaStream_t stream) {
    if (!conv_umma_tma_supports(p_in)) return DR_ERR_UNSUPPORTED;
    ConvParams p = p_in;
    bool use_pair = false, wide = false;
    conv_umma_tma_shape(&p, &use_pair, &wide);
    alignas(64) CUtensorMap map_a, map_b;
    int a_mode = 0;
    const int est = encode_conv_maps(p, use_pair ? p.Nt / 2 : p.Nt, &map_a, &map_b, &a_mode);   // a pair's CTAs load half of B each
    if (est != DR_OK) return est;
    const int m_units = use_pair ? (p.m_tiles + 1) / 2 : p.m_tiles;
    const int total = m_units * p.n_blocks;
    if (total <= 0) return DR_OK;
    const int nkb = p.k * p.k * ((p.Cin + 63) / 64);
    // one k-block of a stage: the activation tile and this CTA's filter tile (half of it in a pair; two sub-tiles if wide)
    const int b_rows = use_pair ? p.Nt / 2 : p.Nt;
    const int sub_bytes = A_TILE_BYTES + (wide ? 2 : 1) * ((b_rows * 128 + 1023) & ~1023);
    alignas(64) CUtensorMap map_y = map_a, map_r = map_a;        // placeholders when the TMA epilogue is off
    int ep_bytes = tma_epilogue_bytes(p, use_pair || wide, &map_y, &map_r);
    int kpb, stages;
    pick_pipeline(T_SMEM_MAX - 1024 - ep_bytes, sub_bytes, nkb, wide ? 256 : p.Nt, &kpb, &stages);
    if (ep_bytes && stages < 2) {                                // not enough room left for the operand pipeline: do without
        ep_bytes = 0;
        pick_pipeline(T_SMEM_MAX - 1024, sub_bytes, nkb, wide ? 256 : p.Nt, &kpb, &stages);
    }
    const bool dual = pick_dual(p, use_pair, wide, ep_bytes, sub_bytes, nkb, total, &kpb, &stages);
    TmaLaunch L;
    L.p = &p; L.map_a = &map_a; L.map_b = &map_b; L.map_y = &map_y; L.map_r = &map_r;
    L.a_mode = a_mode; L.stages = stages; L.sub_bytes = sub_bytes; L.stream = stream; L.units = total;
    L.ep_off = ep_bytes ? stages * kpb * sub_bytes : 0;
    L.smem_bytes = (dual ? 2 : 1) * stages * kpb * sub_bytes + ep_bytes + 1024;
    // a CTA owns all of TMEM: it takes more than half of an SM's shared memory, so that no second one joins it
    if (L.smem_bytes < 120 * 1024) L.smem_bytes = 120 * 1024;
    if (wide) return use_pair ? launch_variant<true, 1, true, false>(L) : launch_variant<false, 1, true, false>(L);
    if (dual) return use_pair ? launch_kpb<true, true>(L, kpb) : launch_kpb<false, true>(L, kpb);
    return use_pair ? launch_kpb<true, false>(L, kpb) : launch_kpb<false, false>(L, kpb);
}


// ---- self-test of the bounded wait -------------------------------------------------------
// One CTA waits on an mbarrier that nothing ever arrives on, with a short cycle limit, and takes the
// same way out as the convolution kernels: record DR_ERR_DEVICE_TIMEOUT and return.
__global__ void wait_timeout_selftest_kernel(int* status, long long limit_cycles) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_barrier_init();
        const long long t0 = clock64();
        bool done = false;
        while (!done && clock64() - t0 < limit_cycles) done = mbar_try_wait(&bar, 0);
        if (!done) report_timeout(status, 99, -1);
    }
}

}  // namespace dr

extern "C" int dr_selftest_wait_timeout(long long limit_cycles, void* stream) {
    if (limit_cycles <= 0 || limit_cycles > 2000000000ll) return DR_ERR_INVALID_ARG;
    int* status = dr::dev_status_ptr();
    if (!status) return DR_ERR_CUDA;
    dr::wait_timeout_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(status, limit_cycles);
    dr::count_launch();
    return dr::launch_status();
}
