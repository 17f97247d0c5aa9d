// Stride-1 k x k convolution (k = 3, 5, pad k/2) with the input patch of a tile brought into shared memory ONCE per
// 64-channel block and every filter tap read out of it by the MMA's operand descriptor (Eq. (tY_j = tW), Section 3.1;
// the merged 5x5 branch of Section 3.2 is the layer this is for).
//
// The im2col kernel (conv_umma.cu) loads one 128-pixel x 64-channel box per tap: 25 boxes that hold the same pixels,
// shifted.  For tiles with few output channels that fill (16 KB per 4 MMAs) is what shared memory and the L2 path
// cannot deliver.  Here the tile's pixels are indexed in a PADDED linear space: a row of the padded plane is the W
// image pixels followed by `pad` zeros that serve as the right border of this row and the left border of the next,
// so with P = W + pad the output position q = i * P + j and the tap (r, s) of it is the input position
// q + r * P + s of the patch whose origin is (row i0 - pad, column -pad).  A tile is R = floor(128 / P) whole image rows,
// i.e. GEMM rows m = 0 .. 127 <-> q = m (rows with m mod P >= W or m / P >= R compute values nobody stores).  The patch is
// one tiled TMA box (64 channels x P columns x rows, zero-filled outside the image), laid out pixel after pixel in
// 128-byte rows with the 128-byte swizzle; the A operand of tap (r, s) is the SAME buffer with the descriptor's
// start address advanced by (r * P + s) * 128 bytes: the swizzle is a function of the shared-memory address, so a
// start inside an 8-row group reads the right chunks.  Only the filter tiles stream per tap.
//
// CTA pairs (cta_group::2, M = 256: each CTA its own tile and patch, half of every filter tile), accumulators in
// TMEM, double-buffered across tiles (or, WIDE: two n sub-blocks of one tile at TMEM columns 0 and 256 sharing the patch),
// roles as in conv_umma_tma_kernel: warp 0 producer, warp 1 MMA issue (WIDE: a second issuing warp for the second
// sub-block), warps 2-5 / 6-9 two epilogue groups.  A stage of the filter ring holds the tiles of several consecutive taps (a whole
// filter row where three such stages fit), so one barrier hand-over covers that many times four MMAs.
// Every wait is bounded; on a timeout the CTA records DR_ERR_DEVICE_TIMEOUT, all roles leave, TMEM is released.
#include "conv_common.cuh"
#include "umma_ptx.cuh"
#include "conv_drain.cuh"

namespace dr {
using namespace ptx;

constexpr int Q_THREADS = 352;      // warp 0 producer, warp 1 MMA issue, warps 2-5 / 6-9 epilogue groups, warp 10 second MMA issuer (WIDE)
constexpr int Q_MMA2_WARP = 10;
constexpr int Q_MAX_STAGES = 12;
constexpr int Q_BIAS_MAX = 512;
constexpr int Q_SMEM_MAX = 227 * 1024 - 4096;   // dynamic part; the static part holds barriers and the bias copy

struct QlinShared {
    uint64_t bfull[Q_MAX_STAGES], bempty[Q_MAX_STAGES], afull[2], aempty[2], tfull[2], tempty[2];
    uint32_t tmem_base;
    int abort;
};

struct QlinPlan {
    int P, R, tiles_per_img, rows_a;   // padded row pitch, image rows per tile, tiles per image, rows of the patch box
    int a_bytes, a_tx;                 // patch buffer (1024-byte multiple) and the bytes one patch load delivers
    int b_sub_bytes;                   // one CTA's half of one filter sub-tile (1024-byte multiple)
    int stages, wide, m_tiles;
    int tps;                           // filter taps per stage of the filter ring: one barrier hand-over covers 4 * tps MMAs
    int m2;                            // 1: two tiles per CTA share the filter ring (conv_qlin2_kernel)
};

template <bool WIDE>
__global__ void __launch_bounds__(Q_THREADS, 1)
conv_qlin_kernel(const ConvParams p, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const QlinPlan pl) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ QlinShared sh;
    __shared__ __align__(16) float bias_s[Q_BIAS_MAX];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool lean = !(p.flags & DR_OUT_F32) && !((p.flags & DR_RESIDUAL) && (p.flags & DR_RELU)) && (p.Cout & 15) == 0 &&
                      p.Cout <= Q_BIAS_MAX && (p.ldc & 7) == 0 && (p.coff & 7) == 0;
    const int lean_mode = (p.flags & DR_RESIDUAL) ? ((p.flags & DR_RELU_AFTER_RESIDUAL) ? 3 : 2) : ((p.flags & DR_RELU) ? 1 : 0);
    if (lean)
        for (int i = tid; i < p.Cout; i += Q_THREADS) bias_s[i] = (p.flags & DR_BIAS) ? p.bias[i] : 0.f;
    const uint32_t rank = cluster_ctarank();                    // 0 issues the MMAs
    const int unit = (int)(blockIdx.x >> 1), nunits = (int)(gridDim.x >> 1);
    const int stages = pl.stages;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&sh.bfull[s], 1); mbar_init(&sh.bempty[s], WIDE ? 2 : 1); }   // WIDE: both issuers commit
        for (int a = 0; a < 2; ++a) {
            mbar_init(&sh.afull[a], 1); mbar_init(&sh.aempty[a], WIDE ? 2 : 1);
            mbar_init(&sh.tfull[a], WIDE ? 2 : 1); mbar_init(&sh.tempty[a], 8 * (WIDE ? 2 : 1));
        }
        sh.abort = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
    }
    if (warp == 1) { tmem_alloc_pair(&sh.tmem_base, 512); tmem_relinquish_pair(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                         // both CTAs' barriers exist before any remote arrive
    tc_fence_after();
    grid_launch_dependents();
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort;

    const int cpb = (p.Cin + 63) >> 6;
    const int taps = p.k * p.k;
    const int total = (pl.m_tiles + 1) >> 1;                    // pair tiles
    const int cout16 = (p.Cout + 15) & ~15;
    const int Nj = min(p.Nt, cout16);                           // first sub-block
    const int Nj1 = WIDE ? cout16 - p.Nt : 0;                   // second sub-block (WIDE)
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t b_base = smem_base + 2u * (uint32_t)pl.a_bytes;
    const uint32_t b_tap_bytes = (uint32_t)pl.b_sub_bytes * (WIDE ? 2u : 1u);   // one tap's filter tile(s)
    const uint32_t b_stage_bytes = b_tap_bytes * (uint32_t)pl.tps;                // a stage: the tiles of `tps` consecutive taps
    const uint32_t bfull0 = smem_u32(&sh.bfull[0]), bempty0 = smem_u32(&sh.bempty[0]);
    const uint32_t afull0 = smem_u32(&sh.afull[0]), aempty0 = smem_u32(&sh.aempty[0]);

    if (warp == 0) {
        if (lane == 0) {
            // -------------------------------------------- TMA producer: per channel block one patch, then one stage per
            // filter row: the filter tiles of its k taps
            const uint32_t b_tx = (uint32_t)(p.Nt >> 1) * 128u * (WIDE ? 2u : 1u);   // per tap; boxes always deliver their full size
            int s = 0, ia = 0;
            uint32_t ph = 0;
            bool ok = true;
            uint32_t ready = mbar_test_u32(bempty0, 1);
            for (int t = unit; t < total && ok; t += nunits) {
                int mt = 2 * t + (int)rank;
                if (mt >= pl.m_tiles) mt = pl.m_tiles - 1;     // odd tile count: the peer recomputes the last tile, stores nothing
                const int img = mt / pl.tiles_per_img;
                const int i0 = (mt - img * pl.tiles_per_img) * pl.R;
                const int brow = (int)rank * (Nj >> 1), brow1 = p.Nt + (int)rank * (Nj1 >> 1);
                for (int cb = 0; cb < cpb && ok; ++cb, ++ia) {
                    const int ab = ia & 1;
                    if (!mbar_wait_u32(aempty0 + 8 * ab, ((uint32_t)(ia >> 1) & 1u) ^ 1u, abort_flag)) {
                        if (!*abort_flag) report_timeout(p.status, 71, t);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    const uint32_t fa = (afull0 + 8 * ab) & PEER_BIT_MASK;
                    if (rank == 0) mbar_expect_tx_u32(fa, 2u * (uint32_t)pl.a_tx);
                    tma_load_4d_u32<true>(smem_base + (uint32_t)ab * (uint32_t)pl.a_bytes, &map_a, fa, cb << 6, -p.pad, i0 - p.pad, img, 1u);
                    for (int tap = 0; tap < taps;) {
                        const int nt = min(pl.tps, taps - tap);
                        if (!ready && !mbar_wait_slow_u32(bempty0 + 8 * s, ph ^ 1, abort_flag)) {
                            if (!*abort_flag) report_timeout(p.status, 72, t);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        int s2 = s + 1;
                        uint32_t ph2 = ph;
                        if (s2 == stages) { s2 = 0; ph2 ^= 1; }
                        ready = mbar_test_u32(bempty0 + 8 * s2, ph2 ^ 1);      // probe the next slot while this one is filled
                        const uint32_t fb = (bfull0 + 8 * s) & PEER_BIT_MASK;
                        uint32_t dst = b_base + (uint32_t)s * b_stage_bytes;
                        if (rank == 0) mbar_expect_tx_u32(fb, 2u * b_tx * (uint32_t)nt);
                        for (int j = 0; j < nt; ++j, ++tap, dst += b_tap_bytes) {
                            tma_load_3d_u32<true>(dst, &map_b, fb, cb << 6, tap, brow, 1u);
                            if (WIDE) tma_load_3d_u32<true>(dst + (uint32_t)pl.b_sub_bytes, &map_b, fb, cb << 6, tap, brow1, 1u);
                        }
                        s = s2;
                        ph = ph2;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == Q_MMA2_WARP) {
        if (rank == 0 && (warp == 1 || WIDE)) {
            // -------------------------------------------- MMA issue: the whole warp walks the loop, lane 0 issues.  WIDE: warp 1
            // issues the first sub-block's MMAs, the second issuing warp the other's (accumulators of their own); a stage or a
            // patch buffer is free when both have committed.
            const int sub = warp == 1 ? 0 : 1;
            const int Ns = sub ? Nj1 : Nj;
            const uint32_t el = (lane == 0 && Ns > 0) ? 1u : 0u;
            const uint32_t elc = lane == 0 ? 1u : 0u;
            const uint32_t tfull0 = smem_u32(&sh.tfull[0]), tempty0 = smem_u32(&sh.tempty[0]);
            const int last_nk16 = ((p.Cin - ((cpb - 1) << 6)) + 15) >> 4;
            const uint32_t idesc = make_idesc_bf16(2 * TILE_M, Ns > 0 ? Ns : 16);
            const uint32_t row_step = (uint32_t)pl.P * 8u;      // one patch row in descriptor units of 16 bytes
            const uint32_t b_off = (uint32_t)sub * (uint32_t)pl.b_sub_bytes;
            int s = 0, it = 0, ia = 0;
            uint32_t ph = 0;
            bool ok = true;
            bool ready = __all_sync(0xffffffffu, mbar_test_u32(bfull0, 0) != 0);
            for (int t = unit; t < total && ok; t += nunits, ++it) {
                const int acc = WIDE ? 0 : (it & 1), au = WIDE ? it : (it >> 1);
                if (!__all_sync(0xffffffffu, mbar_wait_u32(tempty0 + 8 * acc, (au & 1) ^ 1, abort_flag))) {
                    if (elc && !*abort_flag) report_timeout(p.status, 73, t);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d = tmem + (uint32_t)((WIDE ? sub : acc) * 256);
                uint32_t accum = 0;
                for (int cb = 0; cb < cpb && ok; ++cb, ++ia) {
                    const int ab = ia & 1;
                    if (!__all_sync(0xffffffffu, mbar_wait_u32(afull0 + 8 * ab, (uint32_t)(ia >> 1) & 1u, abort_flag))) {
                        if (elc && !*abort_flag) report_timeout(p.status, 74, t);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    const int nk16 = (cb == cpb - 1) ? last_nk16 : 4;
                    uint32_t a_row = sdesc_lo(smem_base + (uint32_t)ab * (uint32_t)pl.a_bytes);
                    uint32_t alo = a_row;
                    int sx = 0;
                    for (int tap = 0; tap < taps;) {
                        const int nt = min(pl.tps, taps - tap);
                        if (!ready && !__all_sync(0xffffffffu, mbar_wait_slow_u32(bfull0 + 8 * s, ph, abort_flag))) {
                            if (elc && !*abort_flag) report_timeout(p.status, 75, t);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        int s2 = s + 1;
                        uint32_t ph2 = ph;
                        if (s2 == stages) { s2 = 0; ph2 ^= 1; }
                        ready = __all_sync(0xffffffffu, mbar_test_u32(bfull0 + 8 * s2, ph2) != 0);   // probe the next slot while this one is issued
                        tc_fence_after();
                        uint32_t blo = sdesc_lo(b_base + (uint32_t)s * b_stage_bytes + b_off);
                        for (int j = 0; j < nt; ++j, ++tap, blo += b_tap_bytes >> 4) {
                            umma_bf16_lo<true>(d, alo, blo, idesc, accum, (nk16 > 0) & el);
                            accum = 1;
                            umma_bf16_lo<true>(d, alo + 2, blo + 2, idesc, 1u, (nk16 > 1) & el);
                            umma_bf16_lo<true>(d, alo + 4, blo + 4, idesc, 1u, (nk16 > 2) & el);
                            umma_bf16_lo<true>(d, alo + 6, blo + 6, idesc, 1u, (nk16 > 3) & el);
                            // next tap: one pixel on, or the start of the next filter row
                            alo += 8u;
                            if (++sx == p.k) { sx = 0; a_row += row_step; alo = a_row; }
                        }
                        if (elc) umma_commit_u32<true>(bempty0 + 8 * s);
                        s = s2;
                        ph = ph2;
                    }
                    if (ok && elc) umma_commit_u32<true>(aempty0 + 8 * ab);   // the patch buffer may be refilled once these MMAs are done
                }
                if (ok && elc) umma_commit_u32<true>(tfull0 + 8 * acc);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue: two groups of four warps; group g drains accumulator
        // buffer g (every other tile), or, WIDE, sub-block g of every tile.  TMEM lane quarter = warp % 4.
        const int g = (warp - 2) >> 2;
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const int il = row / pl.P, j = row - il * pl.P;          // position of this GEMM row in the tile's padded rows
        for (int t = WIDE ? unit : unit + g * nunits, au = 0; t < total; t += WIDE ? nunits : 2 * nunits, ++au) {
            const int mt = 2 * t + (int)rank;
            const int n0 = WIDE ? g * p.Nt : 0;
            const int ncols = WIDE ? (g ? Nj1 : Nj) : Nj;
            const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.tfull[WIDE ? 0 : g], au & 1, abort_flag));
            if (!ok) {
                if (!*abort_flag) report_timeout(p.status, 76, t);
                *abort_flag = 1;
                break;
            }
            tc_fence_after();
            const int img = mt / pl.tiles_per_img;
            const int i = (mt - img * pl.tiles_per_img) * pl.R + il;
            const bool row_ok = mt < pl.m_tiles && il < pl.R && j < p.W && i < p.H;
            const long long m = ((long long)img * p.H + i) * p.W + j;
            const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g * 256);
            if (ncols <= 0) {
                // nothing to drain
            } else if (lean) {
                if (lean_mode == 1) drain_fast<1>(p, taddr, ncols, m, row_ok, n0, bias_s);
                else if (lean_mode == 3) drain_fast<3>(p, taddr, ncols, m, row_ok, n0, bias_s);
                else if (lean_mode == 0) drain_fast<0>(p, taddr, ncols, m, row_ok, n0, bias_s);
                else drain_fast<2>(p, taddr, ncols, m, row_ok, n0, bias_s);
            } else {
                drain_direct(p, taddr, ncols, m, row_ok, n0);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_leader(&sh.tempty[WIDE ? 0 : g]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {   // give copies and MMAs still in flight time to land before shared memory and TMEM go away
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) {}
        __syncthreads();
    }
    cluster_sync_all();                                         // neither CTA leaves while the other may still signal it
    if (p.overlap_prev) grid_dependency_wait();
    if (warp == 1) tmem_dealloc_pair(tmem, 512);
}

// =====================================================================================
// Two tiles per CTA that share the filter ring (layers with at most 256 output channels)
// =====================================================================================
// One thread cannot hand the tensor core MMAs of fewer than 256 columns as fast as it executes them once the stage
// hand-over (barrier probe, fence, commit) is paid, and the filter tiles are the only stream left here.  So a CTA takes
// TWO row tiles at a time (a CTA pair: four): each has its own patch buffers, accumulators, MMA-issuing warp (warp 1 and
// warp 10) and epilogue group, and both multiply against the SAME stage of the filter ring, which is released when both
// issuers have committed.  One issuer's hand-over runs under the other's MMAs, the filter traffic per output halves, and a
// tile's epilogue runs under the other tile's MMAs.  Accumulators: tile s at TMEM column 256 s, two buffers of up to 128
// columns (double-buffered across units) or one of up to 256.
struct Qlin2Shared {
    uint64_t bfull[Q_MAX_STAGES], bempty[Q_MAX_STAGES], afull[4], aempty[4], tfull[4], tempty[4];   // [tile s][buffer]
    uint32_t tmem_base;
    int abort;
};

__global__ void __launch_bounds__(Q_THREADS, 1)
conv_qlin2_kernel(const ConvParams p, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const QlinPlan pl) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ Qlin2Shared sh;
    __shared__ __align__(16) float bias_s[Q_BIAS_MAX];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool lean = !(p.flags & DR_OUT_F32) && !((p.flags & DR_RESIDUAL) && (p.flags & DR_RELU)) && (p.Cout & 15) == 0 &&
                      p.Cout <= Q_BIAS_MAX && (p.ldc & 7) == 0 && (p.coff & 7) == 0;
    const int lean_mode = (p.flags & DR_RESIDUAL) ? ((p.flags & DR_RELU_AFTER_RESIDUAL) ? 3 : 2) : ((p.flags & DR_RELU) ? 1 : 0);
    if (lean)
        for (int i = tid; i < p.Cout; i += Q_THREADS) bias_s[i] = (p.flags & DR_BIAS) ? p.bias[i] : 0.f;
    const uint32_t rank = cluster_ctarank();                    // 0 issues the MMAs
    const int unit = (int)(blockIdx.x >> 1), nunits = (int)(gridDim.x >> 1);
    const int stages = pl.stages;
    const int nacc = p.Nt <= 128 ? 2 : 1;
    const uint32_t acc_cols = nacc == 2 ? 128u : 256u;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&sh.bfull[s], 1); mbar_init(&sh.bempty[s], 2); }   // both issuers commit
        for (int a = 0; a < 4; ++a) {
            mbar_init(&sh.afull[a], 1); mbar_init(&sh.aempty[a], 1);
            mbar_init(&sh.tfull[a], 1); mbar_init(&sh.tempty[a], 8);
        }
        sh.abort = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
    }
    if (warp == 1) { tmem_alloc_pair(&sh.tmem_base, 512); tmem_relinquish_pair(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                         // both CTAs' barriers exist before any remote arrive
    tc_fence_after();
    grid_launch_dependents();
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort;

    const int cpb = (p.Cin + 63) >> 6;
    const int taps = p.k * p.k;
    const int total = (pl.m_tiles + 3) >> 2;                    // units of four tiles: tile = 4 u + 2 s + rank
    const int cout16 = (p.Cout + 15) & ~15;
    const int Nj = min(p.Nt, cout16);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t b_base = smem_base + 4u * (uint32_t)pl.a_bytes;
    const uint32_t b_tap_bytes = (uint32_t)pl.b_sub_bytes;
    const uint32_t b_stage_bytes = b_tap_bytes * (uint32_t)pl.tps;
    const uint32_t bfull0 = smem_u32(&sh.bfull[0]), bempty0 = smem_u32(&sh.bempty[0]);
    const uint32_t afull0 = smem_u32(&sh.afull[0]), aempty0 = smem_u32(&sh.aempty[0]);

    if (warp == 0) {
        if (lane == 0) {
            // -------------------------------------------- TMA producer: per channel block the two tiles' patches, then the
            // filter stages both tiles multiply against
            const uint32_t b_tx = (uint32_t)(p.Nt >> 1) * 128u;
            int s = 0, ia = 0;
            uint32_t ph = 0;
            bool ok = true;
            if (p.pdl_wait) grid_dependency_wait();
            uint32_t ready = mbar_test_u32(bempty0, 1);
            for (int t = unit; t < total && ok; t += nunits) {
                const int brow = (int)rank * (Nj >> 1);
                for (int cb = 0; cb < cpb && ok; ++cb, ++ia) {
                    const int ab = ia & 1;
                    for (int ts = 0; ts < 2 && ok; ++ts) {
                        int mt = 4 * t + 2 * ts + (int)rank;
                        if (mt >= pl.m_tiles) mt = pl.m_tiles - 1;     // past the end: the last tile again, nothing stored
                        const int img = mt / pl.tiles_per_img;
                        const int i0 = (mt - img * pl.tiles_per_img) * pl.R;
                        const int bi = 2 * ts + ab;
                        if (!mbar_wait_u32(aempty0 + 8 * bi, ((uint32_t)(ia >> 1) & 1u) ^ 1u, abort_flag)) {
                            if (!*abort_flag) report_timeout(p.status, 81, t);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        const uint32_t fa = (afull0 + 8 * bi) & PEER_BIT_MASK;
                        if (rank == 0) mbar_expect_tx_u32(fa, 2u * (uint32_t)pl.a_tx);
                        tma_load_4d_u32<true>(smem_base + (uint32_t)bi * (uint32_t)pl.a_bytes, &map_a, fa, cb << 6, -p.pad, i0 - p.pad, img, 1u);
                    }
                    for (int tap = 0; tap < taps && ok;) {
                        const int nt = min(pl.tps, taps - tap);
                        if (!ready && !mbar_wait_slow_u32(bempty0 + 8 * s, ph ^ 1, abort_flag)) {
                            if (!*abort_flag) report_timeout(p.status, 82, t);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        int s2 = s + 1;
                        uint32_t ph2 = ph;
                        if (s2 == stages) { s2 = 0; ph2 ^= 1; }
                        ready = mbar_test_u32(bempty0 + 8 * s2, ph2 ^ 1);
                        const uint32_t fb = (bfull0 + 8 * s) & PEER_BIT_MASK;
                        uint32_t dst = b_base + (uint32_t)s * b_stage_bytes;
                        if (rank == 0) mbar_expect_tx_u32(fb, 2u * b_tx * (uint32_t)nt);
                        for (int j = 0; j < nt; ++j, ++tap, dst += b_tap_bytes) tma_load_3d_u32<true>(dst, &map_b, fb, cb << 6, tap, brow, 1u);
                        s = s2;
                        ph = ph2;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == Q_MMA2_WARP) {
        if (rank == 0) {
            // -------------------------------------------- MMA issue for tile ts of every unit: the whole warp walks the loop,
            // lane 0 issues
            const int ts = warp == 1 ? 0 : 1;
            const uint32_t el = lane == 0 ? 1u : 0u;
            const uint32_t tfull0 = smem_u32(&sh.tfull[0]), tempty0 = smem_u32(&sh.tempty[0]);
            const int last_nk16 = ((p.Cin - ((cpb - 1) << 6)) + 15) >> 4;
            const uint32_t idesc = make_idesc_bf16(2 * TILE_M, Nj);
            const uint32_t row_step = (uint32_t)pl.P * 8u;
            int s = 0, it = 0, ia = 0;
            uint32_t ph = 0;
            bool ok = true;
            bool ready = __all_sync(0xffffffffu, mbar_test_u32(bfull0, 0) != 0);
            for (int t = unit; t < total && ok; t += nunits, ++it) {
                const int bsel = nacc == 2 ? (it & 1) : 0, au = nacc == 2 ? (it >> 1) : it;
                const int ti = 2 * ts + bsel;
                if (!__all_sync(0xffffffffu, mbar_wait_u32(tempty0 + 8 * ti, (au & 1) ^ 1, abort_flag))) {
                    if (el && !*abort_flag) report_timeout(p.status, 83, t);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d = tmem + (uint32_t)(ts * 256) + (uint32_t)bsel * acc_cols;
                uint32_t accum = 0;
                for (int cb = 0; cb < cpb && ok; ++cb, ++ia) {
                    const int bi = 2 * ts + (ia & 1);
                    if (!__all_sync(0xffffffffu, mbar_wait_u32(afull0 + 8 * bi, (uint32_t)(ia >> 1) & 1u, abort_flag))) {
                        if (el && !*abort_flag) report_timeout(p.status, 84, t);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    const int nk16 = (cb == cpb - 1) ? last_nk16 : 4;
                    uint32_t a_row = sdesc_lo(smem_base + (uint32_t)bi * (uint32_t)pl.a_bytes);
                    uint32_t alo = a_row;
                    int sx = 0;
                    for (int tap = 0; tap < taps;) {
                        const int nt = min(pl.tps, taps - tap);
                        if (!ready && !__all_sync(0xffffffffu, mbar_wait_slow_u32(bfull0 + 8 * s, ph, abort_flag))) {
                            if (el && !*abort_flag) report_timeout(p.status, 85, t);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        int s2 = s + 1;
                        uint32_t ph2 = ph;
                        if (s2 == stages) { s2 = 0; ph2 ^= 1; }
                        ready = __all_sync(0xffffffffu, mbar_test_u32(bfull0 + 8 * s2, ph2) != 0);
                        tc_fence_after();
                        uint32_t blo = sdesc_lo(b_base + (uint32_t)s * b_stage_bytes);
                        for (int j = 0; j < nt; ++j, ++tap, blo += b_tap_bytes >> 4) {
                            umma_bf16_lo<true>(d, alo, blo, idesc, accum, (nk16 > 0) & el);
                            accum = 1;
                            umma_bf16_lo<true>(d, alo + 2, blo + 2, idesc, 1u, (nk16 > 1) & el);
                            umma_bf16_lo<true>(d, alo + 4, blo + 4, idesc, 1u, (nk16 > 2) & el);
                            umma_bf16_lo<true>(d, alo + 6, blo + 6, idesc, 1u, (nk16 > 3) & el);
                            alo += 8u;
                            if (++sx == p.k) { sx = 0; a_row += row_step; alo = a_row; }
                        }
                        if (el) umma_commit_u32<true>(bempty0 + 8 * s);
                        s = s2;
                        ph = ph2;
                    }
                    if (ok && el) umma_commit_u32<true>(aempty0 + 8 * bi);
                }
                if (ok && el) umma_commit_u32<true>(tfull0 + 8 * ti);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue: group g drains tile g of every unit
        const int g = (warp - 2) >> 2;
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const int il = row / pl.P, j = row - il * pl.P;
        if (p.pdl_wait && (p.flags & DR_RESIDUAL)) grid_dependency_wait();
        for (int t = unit, it = 0; t < total; t += nunits, ++it) {
            const int bsel = nacc == 2 ? (it & 1) : 0;
            const uint32_t par = (uint32_t)(nacc == 2 ? (it >> 1) : it) & 1u;
            const int ti = 2 * g + bsel;
            const int mt = 4 * t + 2 * g + (int)rank;
            const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.tfull[ti], par, abort_flag));
            if (!ok) {
                if (!*abort_flag) report_timeout(p.status, 86, t);
                *abort_flag = 1;
                break;
            }
            tc_fence_after();
            const int img = mt / pl.tiles_per_img;
            const int i = (mt - img * pl.tiles_per_img) * pl.R + il;
            const bool row_ok = mt < pl.m_tiles && il < pl.R && j < p.W && i < p.H;
            const long long m = ((long long)img * p.H + i) * p.W + j;
            const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g * 256) + (uint32_t)bsel * acc_cols;
            if (lean) {
                if (lean_mode == 1) drain_fast<1>(p, taddr, Nj, m, row_ok, 0, bias_s);
                else if (lean_mode == 3) drain_fast<3>(p, taddr, Nj, m, row_ok, 0, bias_s);
                else if (lean_mode == 0) drain_fast<0>(p, taddr, Nj, m, row_ok, 0, bias_s);
                else drain_fast<2>(p, taddr, Nj, m, row_ok, 0, bias_s);
            } else {
                drain_direct(p, taddr, Nj, m, row_ok, 0);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_leader(&sh.tempty[ti]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) {}
        __syncthreads();
    }
    cluster_sync_all();
    if (p.overlap_prev) grid_dependency_wait();
    if (warp == 1) tmem_dealloc_pair(tmem, 512);
}

// ---- host ---------------------------------------------------------------------------------
static bool qlin_plan(const ConvParams& p, QlinPlan* out) {
    if (p.flags & (DR_POOL | DR_LRN)) return false;
    if (p.patch || p.argmax) return false;
    if (p.stride != 1 || p.k < 3 || !(p.k & 1) || p.k > 7 || p.pad != p.k / 2) return false;
    if ((p.Cin & 7) || p.Cin < 64) return false;
    if (p.Ho != p.H || p.Wo != p.W) return false;
    const int cout16 = (p.Cout + 15) & ~15;
    if (cout16 < 32 || cout16 > 512) return false;
    QlinPlan pl{};
    pl.P = p.W + p.pad;
    if (pl.P > TILE_M) return false;
    pl.R = TILE_M / pl.P;
    pl.tiles_per_img = (p.H + pl.R - 1) / pl.R;
    const long long mt = (long long)p.B * pl.tiles_per_img;
    if (mt < 2 || mt > 0x3fffffffLL) return false;
    pl.m_tiles = (int)mt;
    const int last = (TILE_M - 1) + (p.k - 1) * pl.P + (p.k - 1);   // last patch position any GEMM row reads
    pl.rows_a = last / pl.P + 1;
    if (pl.rows_a > 256 || pl.P > 256) return false;
    pl.a_tx = pl.rows_a * pl.P * 128;
    pl.a_bytes = (pl.a_tx + 1023) & ~1023;
    pl.wide = cout16 > 256;
    int nt = cout16;
    if (pl.wide) nt = ((cout16 / 2 + 15) / 16) * 16;               // near-equal sub-blocks, the first the larger
    if (pl.wide && cout16 - nt < 32) return false;                 // MMAs of 256 rows take N >= 32
    pl.b_sub_bytes = (((nt >> 1) * 128) + 1023) & ~1023;
    // two tiles per CTA (four patch buffers) where the layer has at most 256 output channels, enough tiles, and three
    // stages of the filter ring still fit
    pl.m2 = (!pl.wide && mt >= 8 && tunable("DR_QLIN_M2", 1) != 0 && (Q_SMEM_MAX - 1024 - 4 * pl.a_bytes) / pl.b_sub_bytes >= 3) ? 1 : 0;
    const int budget = Q_SMEM_MAX - 1024 - (pl.m2 ? 4 : 2) * pl.a_bytes;
    const int tap_bytes = pl.b_sub_bytes * (pl.wide ? 2 : 1);
    if (budget / tap_bytes < 3) return false;
    pl.tps = p.k;                                                  // a whole filter row per stage if three such stages fit
    while (pl.tps > 1 && budget / (tap_bytes * pl.tps) < 3) --pl.tps;
    const int st = budget / (tap_bytes * pl.tps);
    pl.stages = st > Q_MAX_STAGES ? Q_MAX_STAGES : st;
    *out = pl;
    return true;
}

int conv_qlin_nt(const ConvParams& p) {
    const int cout16 = (p.Cout + 15) & ~15;
    return cout16 > 256 ? ((cout16 / 2 + 15) / 16) * 16 : cout16;
}

bool conv_qlin_supports(const ConvParams& p) {
    QlinPlan pl;
    return qlin_plan(p, &pl);
}

// Share of a tile's 128 GEMM rows that are stored outputs: what the padded linear indexing costs in MMA work.
double conv_qlin_fill(const ConvParams& p) {
    QlinPlan pl;
    if (!qlin_plan(p, &pl)) return 0.0;
    return (double)p.H * p.W / ((double)pl.tiles_per_img * TILE_M);
}

int conv_qlin_launch(const ConvParams& p_in, cudaStream_t stream) {
    QlinPlan pl;
    if (!qlin_plan(p_in, &pl)) return DR_ERR_UNSUPPORTED;
    ConvParams p = p_in;
    p.Nt = conv_qlin_nt(p);
    p.n_blocks = 1;
    static PerDeviceFlag attr_set;
    static int max_clusters_dev[64] = {};
        int& max_clusters = max_clusters_dev[PerDeviceFlag::dev()];
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(Q_THREADS); cfg.stream = stream; cfg.attrs = attr; cfg.numAttrs = 1;
    if (!attr_set.get()) {
        if (cudaFuncSetAttribute(conv_qlin_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Q_SMEM_MAX) != cudaSuccess ||
            cudaFuncSetAttribute(conv_qlin2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Q_SMEM_MAX) != cudaSuccess ||
            cudaFuncSetAttribute(conv_qlin_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Q_SMEM_MAX) != cudaSuccess)
            return DR_ERR_CUDA;
        cfg.gridDim = dim3(2 * num_sms());
        cfg.dynamicSmemBytes = (size_t)Q_SMEM_MAX;
        if (cudaOccupancyMaxActiveClusters(&max_clusters, conv_qlin_kernel<false>, &cfg) != cudaSuccess || max_clusters < 1) return DR_ERR_CUDA;
        attr_set.set();
    }
    alignas(64) CUtensorMap map_a, map_b;
    {
        const cuuint64_t dims[4] = {(cuuint64_t)p.Cin, (cuuint64_t)p.W, (cuuint64_t)p.H, (cuuint64_t)p.B};
        const cuuint64_t strides[3] = {(cuuint64_t)p.Cin * 2, (cuuint64_t)p.W * p.Cin * 2, (cuuint64_t)p.H * p.W * p.Cin * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)pl.P, (cuuint32_t)pl.rows_a, 1};
        if (tmap_tiled(&map_a, 4, p.x, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B) != DR_OK) return DR_ERR_CUDA;
    }
    {
        // filters as (Cin, taps, Cout); a box is one CTA's half of a sub-block.  WIDE sub-blocks may differ in width: the
        // box has the rows of the larger half, the rows past the smaller one belong to the next filters or lie past the
        // tensor (zero fill) and are never multiplied (the MMA's N stops before them)
        const cuuint64_t dims[3] = {(cuuint64_t)p.Cin, (cuuint64_t)(p.k * p.k), (cuuint64_t)p.Cout};
        const cuuint64_t strides[2] = {(cuuint64_t)p.Cin * 2, (cuuint64_t)p.K * 2};
        const cuuint32_t box[3] = {64, 1, (cuuint32_t)(p.Nt >> 1)};
        if (tmap_tiled(&map_b, 3, p.w, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B) != DR_OK) return DR_ERR_CUDA;
    }
    const int units = pl.m2 ? (pl.m_tiles + 3) / 4 : (pl.m_tiles + 1) / 2;
    const int pairs = units < max_clusters ? units : max_clusters;
    int smem_bytes = (pl.m2 ? 4 : 2) * pl.a_bytes + pl.stages * pl.b_sub_bytes * (pl.wide ? 2 : 1) * pl.tps + 1024;
    if (smem_bytes < 120 * 1024) smem_bytes = 120 * 1024;       // one CTA per SM: each owns all of TMEM
    cfg.gridDim = dim3(2 * pairs);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.numAttrs = p.overlap_prev ? 2 : 1;
    cudaError_t e;
    cfg.numAttrs = (p.overlap_prev || p.pdl_wait) ? 2 : 1;
    if (pl.m2) e = cudaLaunchKernelEx(&cfg, conv_qlin2_kernel, p, map_a, map_b, pl);
    else if (pl.wide) e = cudaLaunchKernelEx(&cfg, conv_qlin_kernel<true>, p, map_a, map_b, pl);
    else e = cudaLaunchKernelEx(&cfg, conv_qlin_kernel<false>, p, map_a, map_b, pl);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return DR_ERR_CUDA; }
    count_launch();
    return launch_status();
}

}  // namespace dr
