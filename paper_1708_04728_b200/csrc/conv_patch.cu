// Patch-tiled convolution kernels for the slim layers whose epilogue max-pools (and optionally
// LRN-normalises): a tile is the (2*PH+1) x (2*PW+1) patch of convolution outputs that PH x PW pooled
// outputs need (the first row / column is a halo the neighbouring tile recomputes), so the pooled
// tensor is the only thing written to HBM.  Both kernels are persistent (one CTA per SM), use
// tcgen05 MMAs with two TMEM accumulator buffers, and share conv_fused_epilogue.cuh.
//
//   conv_patch_tma_kernel   stride-1 layers with Cin a multiple of 8 (GoogLeNet conv2/3x3): the
//       activation patch of one filter tap is ONE tiled 4-D TMA box (64 channels x patch width x patch
//       height), zero-filled outside the image; filters stream through TMA as in the main kernel.
//   conv_stem_kernel        the 7x7 / stride-2 / 3-channel stem (GoogLeNet and ResNet conv1).  TMA
//       cannot address 6-byte pixels, so four producer warps bring the input patch into shared memory
//       with 4-byte cp.async (next tile's patch in flight while this one is used) and build the im2col
//       tile from there.  K is laid out as 7 tap-rows x 24 slots (21 = 7 taps x 3 channels used, 3 slots
//       and the tail up to 192 carry zero weights), which makes every tap-row a 48-byte run that starts
//       4-byte aligned in the patch and 16-byte aligned in the operand tile.  The 64 x 192 filter tile is
//       built once per CTA and stays resident.
#include <cstdlib>

#include "conv_common.cuh"
#include "conv_fused_epilogue.cuh"
#include "umma_ptx.cuh"

namespace dr {
using namespace ptx;

constexpr int P_A_BYTES = TILE_M * 128;
constexpr int P_THREADS = 320;          // warp 0 TMA, warp 1 MMA, warps 2-5 and 6-9: two epilogue groups (alternate tiles)
constexpr int P_MAX_STAGES = 6;
constexpr int P_SMEM_MAX = 227 * 1024 - 256;

__device__ __forceinline__ uint32_t swz128(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

struct PatchShared {
    uint64_t full[P_MAX_STAGES], empty[P_MAX_STAGES], tfull[2], tempty[2];
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ void tma_load_4d_tile(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
                 "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}

__global__ void __launch_bounds__(P_THREADS, 1)
conv_patch_tma_kernel(const ConvParams p, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const int stages,
                      const int stage_bytes, const int groups) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ PatchShared sh;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* fe_stage = smem + stages * stage_bytes;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&sh.tfull[a], 1); mbar_init(&sh.tempty[a], 4); }
        sh.abort = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
    }
    if (warp == 1) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
    const int fe_bytes = fe_smem_bytes(p);
    fe_init(p, fe_stage, tid, P_THREADS);
    if (groups > 1) fe_init(p, fe_stage + fe_bytes, tid, P_THREADS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort;

    const int cpb = (p.Cin + 63) >> 6;
    const int total = p.m_tiles;
    const int per = p.tiles_h * p.tiles_w;
    const int pwc = 2 * p.PW + 1, phc = 2 * p.PH + 1;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0 = smem_u32(&sh.full[0]), empty0 = smem_u32(&sh.empty[0]);

    if (warp == 0) {
        if (lane == 0) {
            const uint32_t tx = (uint32_t)(pwc * phc) * 128u + (uint32_t)p.Nt * 128u;
            const int nkb = p.k * p.k * cpb;
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            uint32_t ready = mbar_test_u32(empty0, 1);
            for (int t = blockIdx.x; t < total && ok; t += gridDim.x) {
                const int n = t / per, tt_ = t - n * per;
                const int th = tt_ / p.tiles_w, tw = tt_ - th * p.tiles_w;
                const int h0 = 2 * th * p.PH - 1 - p.pad, w0 = 2 * tw * p.PW - 1 - p.pad;   // stride 1
                int r = 0, q = 0, tap = 0, c0 = 0;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ready && !mbar_wait_slow_u32(empty0 + 8 * s, ph ^ 1, abort_flag)) {
                        if (!*abort_flag) report_timeout(p.status, 31, t);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    int s2 = s + 1;
                    uint32_t ph2 = ph;
                    if (s2 == stages) { s2 = 0; ph2 ^= 1; }
                    ready = mbar_test_u32(empty0 + 8 * s2, ph2 ^ 1);
                    const uint32_t a_dst = smem_base + (uint32_t)s * (uint32_t)stage_bytes;
                    const uint32_t fb = full0 + 8 * s;
                    mbar_expect_tx_u32(fb, tx);
                    tma_load_4d_tile(a_dst, &map_a, fb, c0, w0 + q, h0 + r, n);
                    tma_load_3d_u32<false>(a_dst + P_A_BYTES, &map_b, fb, c0, tap, 0, 1u);
                    c0 += 64;
                    const bool wrap_c = c0 >= p.Cin;
                    c0 = wrap_c ? 0 : c0;
                    tap += wrap_c ? 1 : 0;
                    q += wrap_c ? 1 : 0;
                    const bool wrap_q = q == p.k;
                    q = wrap_q ? 0 : q;
                    r += wrap_q ? 1 : 0;
                    s = s2;
                    ph = ph2;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t tfull0 = smem_u32(&sh.tfull[0]), tempty0 = smem_u32(&sh.tempty[0]);
            const int nkb = p.k * p.k * cpb;
            const int last_nk16 = ((p.Cin - ((cpb - 1) << 6)) + 15) >> 4;
            const uint32_t idesc = make_idesc_bf16(TILE_M, p.Nt);
            int s = 0, it = 0;
            uint32_t ph = 0;
            bool ok = true;
            uint32_t ready = mbar_test_u32(full0, 0);
            for (int t = blockIdx.x; t < total && ok; t += gridDim.x, ++it) {
                const int acc = it & 1, au = it >> 1;
                if (!mbar_wait_u32(tempty0 + 8 * acc, (au & 1) ^ 1, abort_flag)) {
                    if (!*abort_flag) report_timeout(p.status, 32, t);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d = tmem + (uint32_t)(acc * 256);
                uint32_t accum = 0;
                int cc = 0;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ready && !mbar_wait_slow_u32(full0 + 8 * s, ph, abort_flag)) {
                        if (!*abort_flag) report_timeout(p.status, 33, t);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    int s2 = s + 1;
                    uint32_t ph2 = ph;
                    if (s2 == stages) { s2 = 0; ph2 ^= 1; }
                    ready = mbar_test_u32(full0 + 8 * s2, ph2);
                    tc_fence_after();
                    const uint32_t a = smem_base + (uint32_t)s * (uint32_t)stage_bytes;
                    const uint32_t alo = sdesc_lo(a), blo = sdesc_lo(a + P_A_BYTES);
                    const int nk16 = (cc == cpb - 1) ? last_nk16 : 4;
                    cc = (cc + 1 == cpb) ? 0 : cc + 1;
                    umma_bf16_lo<false>(d, alo, blo, idesc, accum, 1u);
                    accum = 1;
                    umma_bf16_lo<false>(d, alo + 2, blo + 2, idesc, 1u, nk16 > 1);
                    umma_bf16_lo<false>(d, alo + 4, blo + 4, idesc, 1u, nk16 > 2);
                    umma_bf16_lo<false>(d, alo + 6, blo + 6, idesc, 1u, nk16 > 3);
                    umma_commit_u32<false>(empty0 + 8 * s);
                    s = s2;
                    ph = ph2;
                }
                if (ok) umma_commit_u32<false>(tfull0 + 8 * acc);
            }
        }
        __syncwarp();
    } else {
        // epilogue groups of four warps: with two groups, group g takes the tiles whose accumulator buffer is g;
        // with one group (more shared memory left for pipeline stages) it takes every tile
        const int g = (warp - 2) >> 2;
        const int q = warp & 3;
        const int row = q * 32 + lane;
        if (g < groups) {
            for (int it = g;; it += groups) {
                const int t = blockIdx.x + it * gridDim.x;
                if (t >= total) break;
                const int acc = it & 1, au = it >> 1;
                const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.tfull[acc], au & 1, abort_flag));
                if (!ok) {
                    if (!*abort_flag) report_timeout(p.status, 34, t);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                uint64_t* te = &sh.tempty[acc];
                fused_epilogue<false>(p, t, tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * 256), fe_stage + g * fe_bytes, row, 1 + 2 * g, [&]() {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(te);
                });
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) {}
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// =====================================================================================
//                         patch kernel on CTA pairs, filters resident
// =====================================================================================
// conv_patch_tma_kernel streams the filter tile of every tap again for every patch: 24 KB of filters next to
// 15 KB of activations per k-block (GoogLeNet conv2: 1.9 GB of filter loads against 1.2 GB of activation loads
// per batch of 256).  Here two CTAs
// of a cluster form one MMA unit (tcgen05 cta_group::2, M = 256 = one patch per CTA); each keeps HALF of the
// filter bank in shared memory for the whole kernel (`resident`), or streams only its half (`!resident`), and the
// even CTA issues MMAs that read both shared memories.  Barrier protocol as in conv_umma_tma_kernel<PAIR>:
// loads of both CTAs report to the even CTA's barriers, its commits arrive in both CTAs, epilogue warps of both
// CTAs arrive on the even CTA's `tempty`.  No multicast loads.
struct PatchPairShared {
    uint64_t full[P_MAX_STAGES], empty[P_MAX_STAGES], tfull[2], tempty[2], wfull;
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ void tma_load_4d_tile_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(
                     dst),
                 "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}

// Warps in groups of four (the unit in which registers are re-assigned): warps 0-3 = producer, MMA issuer and two idle
// warps, which give registers up; warps 4-7 and 8-11 = the two epilogue groups, which take them (the fused LRN epilogue
// keeps two 32-channel chunks, their squares, window sums and scales, and a TMEM load in flight, in registers).
//
// SPLIT (LRN before the pool, channel count a multiple of 64): each of the two tile groups is eight warps, four per half
// of the channels (fused_epilogue_split).  The accumulator of a tile is occupied while its MMAs run and while it is
// drained, and with two accumulators a tile cannot take less than half of that sum; the drain of an LRN-first layer
// (the LRN arithmetic of 192 channels per row) is longer than the MMAs, and two warps per row halve it.  640 threads:
// 128 * 32 + 512 * 112 registers = 640 * 96.
constexpr int PP_THREADS = 384, PP_THREADS_SPLIT = 640;
constexpr int PP_REGS_AUX = 40, PP_REGS_EPI = 232;      // 128 * 40 + 256 * 232 = 384 * 168, the registers of the launch
constexpr int PP_REGS_AUX_SPLIT = 32, PP_REGS_EPI_SPLIT = 112;   // 128 * 32 + 512 * 112 = 640 * 96
template <bool SPLIT>
__global__ void __launch_bounds__(SPLIT ? PP_THREADS_SPLIT : PP_THREADS, 1)
conv_patch_pair_kernel(const ConvParams p, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const int stages,
                       const int stage_bytes, const int groups, const int resident, const int bsub_bytes) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ PatchPairShared sh;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cpb = (p.Cin + 63) >> 6;
    const int nkb = p.k * p.k * cpb;
    uint8_t* b_res = smem + stages * stage_bytes;                            // resident half filter bank: nkb sub-tiles
    uint8_t* fe_stage = b_res + (resident ? nkb * bsub_bytes : 0);
    const uint32_t rank = cluster_ctarank();                                 // 0 issues the MMAs
    const int unit = (int)(blockIdx.x >> 1), nunits = (int)(gridDim.x >> 1);

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&sh.tfull[a], 1); mbar_init(&sh.tempty[a], SPLIT ? 16 : 8); }   // the epilogue warps of both CTAs
        mbar_init(&sh.wfull, 1);
        sh.abort = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
    }
    if (warp == 1) { tmem_alloc_pair(&sh.tmem_base, 512); tmem_relinquish_pair(); }
    const int fe_bytes = fe_smem_bytes(p);
    fe_init(p, fe_stage, tid, (int)blockDim.x);
    if (groups > 1) fe_init(p, fe_stage + fe_bytes, tid, (int)blockDim.x);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                                      // both CTAs' barriers exist before any remote arrive
    tc_fence_after();
    grid_launch_dependents();                                                // a split-K layer behind this one may start its prologue
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort;

    const int total = p.m_tiles;
    const int units = (total + 1) >> 1;                                      // pair tiles: patches 2u and 2u+1
    const int per = p.tiles_h * p.tiles_w;
    const int pwc = 2 * p.PW + 1, phc = 2 * p.PH + 1;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0 = smem_u32(&sh.full[0]), empty0 = smem_u32(&sh.empty[0]);
    const uint32_t b_res0 = smem_u32(b_res);
    const uint32_t half_rows = (uint32_t)p.Nt >> 1;

    if (warp == 0) {
        if (SPLIT) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PP_REGS_AUX_SPLIT)); else asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PP_REGS_AUX));
        if (lane == 0) {
            const uint32_t a_tx = (uint32_t)(pwc * phc) * 128u;
            const uint32_t b_tx = half_rows * 128u;
            const int brow = (int)rank * (int)half_rows;
            if (resident) {
                const uint32_t wb = smem_u32(&sh.wfull) & PEER_BIT_MASK;
                if (rank == 0) mbar_expect_tx_u32(wb, 2u * (uint32_t)nkb * b_tx);
                int tap = 0, c0 = 0;
                for (int kb = 0; kb < nkb; ++kb) {
                    tma_load_3d_u32<true>(b_res0 + (uint32_t)kb * (uint32_t)bsub_bytes, &map_b, wb, c0, tap, brow, 1u);
                    c0 += 64;
                    if (c0 >= p.Cin) { c0 = 0; ++tap; }
                }
            }
            const uint32_t tx = a_tx + (resident ? 0u : b_tx);
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            uint32_t ready = mbar_test_u32(empty0, 1);
            if (p.pdl_wait) grid_dependency_wait();                          // the kernel before this one has written the activations
            for (int u = unit; u < units && ok; u += nunits) {
                int t = 2 * u + (int)rank;
                if (t >= total) t = total - 1;                               // odd patch count: the peer repeats the last patch (same values stored twice)
                const int n = t / per, tt_ = t - n * per;
                const int th = tt_ / p.tiles_w, tw = tt_ - th * p.tiles_w;
                const int h0 = 2 * th * p.PH - 1 - p.pad, w0 = 2 * tw * p.PW - 1 - p.pad;   // stride 1
                int r = 0, q = 0, tap = 0, c0 = 0;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ready && !mbar_wait_slow_u32(empty0 + 8 * s, ph ^ 1, abort_flag)) {
                        if (!*abort_flag) report_timeout(p.status, 41, t);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    int s2 = s + 1;
                    uint32_t ph2 = ph;
                    if (s2 == stages) { s2 = 0; ph2 ^= 1; }
                    ready = mbar_test_u32(empty0 + 8 * s2, ph2 ^ 1);
                    const uint32_t a_dst = smem_base + (uint32_t)s * (uint32_t)stage_bytes;
                    const uint32_t fb = (full0 + 8 * s) & PEER_BIT_MASK;
                    if (rank == 0) mbar_expect_tx_u32(fb, 2u * tx);
                    tma_load_4d_tile_pair(a_dst, &map_a, fb, c0, w0 + q, h0 + r, n);
                    if (!resident) tma_load_3d_u32<true>(a_dst + P_A_BYTES, &map_b, fb, c0, tap, brow, 1u);
                    c0 += 64;
                    const bool wrap_c = c0 >= p.Cin;
                    c0 = wrap_c ? 0 : c0;
                    tap += wrap_c ? 1 : 0;
                    q += wrap_c ? 1 : 0;
                    const bool wrap_q = q == p.k;
                    q = wrap_q ? 0 : q;
                    r += wrap_q ? 1 : 0;
                    s = s2;
                    ph = ph2;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (SPLIT) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PP_REGS_AUX_SPLIT)); else asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PP_REGS_AUX));
        if (rank == 0) {
            // the whole warp walks the loop (addresses and descriptors are warp-uniform), lane 0 alone issues and commits:
            // measured faster than a loop run by one lane inside a divergent branch
            const uint32_t el = lane == 0 ? 1u : 0u;
            const uint32_t tfull0 = smem_u32(&sh.tfull[0]), tempty0 = smem_u32(&sh.tempty[0]);
            const int last_nk16 = ((p.Cin - ((cpb - 1) << 6)) + 15) >> 4;
            const uint32_t idesc = make_idesc_bf16(2 * TILE_M, p.Nt);
            int s = 0, it = 0;
            uint32_t ph = 0;
            bool ok = true;
            if (resident && !__all_sync(0xffffffffu, mbar_wait(&sh.wfull, 0, abort_flag))) {
                if (el && !*abort_flag) report_timeout(p.status, 45, 0);
                *abort_flag = 1;
                ok = false;
            }
            bool ready = __all_sync(0xffffffffu, mbar_test_u32(full0, 0) != 0);
            for (int u = unit; u < units && ok; u += nunits, ++it) {
                const int acc = it & 1, au = it >> 1;
                if (!__all_sync(0xffffffffu, mbar_wait_u32(tempty0 + 8 * acc, (au & 1) ^ 1, abort_flag))) {
                    if (el && !*abort_flag) report_timeout(p.status, 42, u);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d = tmem + (uint32_t)(acc * 256);
                uint32_t accum = 0;
                int cc = 0;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ready && !__all_sync(0xffffffffu, mbar_wait_slow_u32(full0 + 8 * s, ph, abort_flag))) {
                        if (el && !*abort_flag) report_timeout(p.status, 43, u);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    int s2 = s + 1;
                    uint32_t ph2 = ph;
                    if (s2 == stages) { s2 = 0; ph2 ^= 1; }
                    ready = __all_sync(0xffffffffu, mbar_test_u32(full0 + 8 * s2, ph2) != 0);
                    tc_fence_after();
                    const uint32_t a = smem_base + (uint32_t)s * (uint32_t)stage_bytes;
                    const uint32_t alo = sdesc_lo(a);
                    const uint32_t blo = sdesc_lo(resident ? b_res0 + (uint32_t)kb * (uint32_t)bsub_bytes : a + P_A_BYTES);
                    const int nk16 = (cc == cpb - 1) ? last_nk16 : 4;
                    cc = (cc + 1 == cpb) ? 0 : cc + 1;
                    umma_bf16_lo<true>(d, alo, blo, idesc, accum, el);
                    accum = 1;
                    umma_bf16_lo<true>(d, alo + 2, blo + 2, idesc, 1u, (nk16 > 1) & el);
                    umma_bf16_lo<true>(d, alo + 4, blo + 4, idesc, 1u, (nk16 > 2) & el);
                    umma_bf16_lo<true>(d, alo + 6, blo + 6, idesc, 1u, (nk16 > 3) & el);
                    if (el) umma_commit_u32<true>(empty0 + 8 * s);
                    s = s2;
                    ph = ph2;
                }
                if (ok && el) umma_commit_u32<true>(tfull0 + 8 * acc);
            }
        }
        __syncwarp();
    } else if (warp < 4) {
        if (SPLIT) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PP_REGS_AUX_SPLIT)); else asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PP_REGS_AUX));   // idle warps of the first group of four
    } else {
        // epilogue groups of four warps, as in conv_patch_tma_kernel; each CTA drains its own patch
        if (SPLIT) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(PP_REGS_EPI_SPLIT));
        else asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(PP_REGS_EPI));
        const int g = SPLIT ? (warp - 4) >> 3 : (warp - 4) >> 2;            // tile group
        const int part = SPLIT ? ((warp - 4) >> 2) & 1 : 0;                  // half of the channels (SPLIT)
        const int q = warp & 3;
        const int row = q * 32 + lane;
        if (g < groups) {
            for (int it = g;; it += groups) {
                const int u = unit + it * nunits;
                if (u >= units) break;
                int t = 2 * u + (int)rank;
                if (t >= total) t = total - 1;
                const int acc = it & 1, au = it >> 1;
                const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.tfull[acc], au & 1, abort_flag));
                if (!ok) {
                    if (!*abort_flag) report_timeout(p.status, 44, t);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                uint64_t* te = &sh.tempty[acc];
                const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * 256);
                auto release = [&]() {
                    __syncwarp();
                    if (lane == 0) mbar_arrive_leader(te);
                };
                if (SPLIT) fused_epilogue_split(p, t, taddr, fe_stage + g * fe_bytes, row, part, 1 + g, release);
                else fused_epilogue<true>(p, t, taddr, fe_stage + g * fe_bytes, row, 1 + 2 * g, release);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) {}
        __syncthreads();
    }
    cluster_sync_all();                                                      // neither CTA leaves while the other may still signal it
    if (warp == 1) tmem_dealloc_pair(tmem, 512);
}

// =====================================================================================
//                                     stem kernel
// =====================================================================================
constexpr int S_THREADS = 416;          // warps 0-3 producers, warp 4 MMA, warps 5-8 and 9-12: two epilogue groups
constexpr int S_KSLOTS = 24;            // K slots per tap-row (k * Cin = 21 used)
constexpr int S_SUBTILES = 3;           // K' = 192 = 3 x 64
constexpr int S_A_BYTES = S_SUBTILES * P_A_BYTES;          // one im2col tile: 48 KB
constexpr int S_B_BYTES = S_SUBTILES * 64 * 128;            // resident filters: 24 KB (64 filters)

struct StemShared {
    uint64_t afull[2], aempty[2], tfull[2], tempty[2];
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ void cp_async4_zfill(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 4 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}

// Layer fixed to k = 7, stride 2, pad 3, Cin = 3, Cout = 64 (host checks).
__global__ void __launch_bounds__(S_THREADS, 1) conv_stem_kernel(const ConvParams p, const int in_rows, const int in_words) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ StemShared sh;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* Bs = smem;                                   // [3][64 rows][128 B]
    uint8_t* As = Bs + S_B_BYTES;                         // 2 x [3][128 rows][128 B]
    uint8_t* fe_stage = As + 2 * S_A_BYTES;
    const int fe_bytes = fe_smem_bytes(p);
    uint32_t* inp = reinterpret_cast<uint32_t*>(fe_stage + 2 * fe_bytes);       // 2 x [in_rows][in_words] input patches
    const int patch_words = in_rows * in_words;

    if (tid == 0) {
        for (int a = 0; a < 2; ++a) {
            mbar_init(&sh.afull[a], 128); mbar_init(&sh.aempty[a], 1);
            mbar_init(&sh.tfull[a], 1); mbar_init(&sh.tempty[a], 4);
        }
        sh.abort = 0;
        fence_barrier_init();
    }
    if (warp == 4) { tmem_alloc(&sh.tmem_base, 128); tmem_relinquish(); }
    // resident filter tile in K' order, zero elsewhere; operand tiles start zeroed (their unused
    // K' slots must stay finite: they meet zero weights)
    for (int i = tid; i < (S_B_BYTES + 2 * S_A_BYTES) / 16; i += S_THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (int i = tid; i < 64 * 147; i += S_THREADS) {
        const int j = i / 147, e = i - j * 147;           // filter j, element (r, s, c) flattened
        const int r = e / 21, sc = e - r * 21;
        const int kp = r * S_KSLOTS + sc;                 // K' index
        const int sub = kp >> 6, within = kp & 63;
        const uint32_t off = (uint32_t)sub * (64 * 128) + swz128(j, within >> 3) + (within & 7) * 2;
        *reinterpret_cast<unsigned short*>(Bs + off) = (j < p.Cout) ? reinterpret_cast<const unsigned short*>(p.w)[(size_t)j * 147 + e] : (unsigned short)0;
    }
    fe_init(p, fe_stage, tid, S_THREADS);
    fe_init(p, fe_stage + fe_bytes, tid, S_THREADS);
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort;

    const int total = p.m_tiles;
    const int per = p.tiles_h * p.tiles_w;
    const int pwc = 2 * p.PW + 1, phc = 2 * p.PH + 1;

    if (warp < 4) {
        // ------------------------------------------------ producers: thread = patch row (conv pixel)
        const int pi = tid / pwc, pj = tid - pi * pwc;
        const bool row_used = pi < phc;
        // issue the cp.async loads of tile t's input patch into buffer b
        // each thread copies the same word slots of every patch: (row, 2*word) of slot k, fixed for the kernel
        constexpr int MAX_SLOTS = 12;
        int slot_rr[MAX_SLOTS], slot_e[MAX_SLOTS];
#pragma unroll
        for (int k = 0; k < MAX_SLOTS; ++k) {
            const int i = tid + 128 * k;
            slot_rr[k] = i < patch_words ? i / in_words : -1;
            slot_e[k] = i < patch_words ? 2 * (i - (i / in_words) * in_words) : 0;
        }
        const int row_elems = 3 * p.W;
        auto load_patch = [&](int t, int b) {
            const int n = t / per, tt_ = t - n * per;
            const int th = tt_ / p.tiles_w, tw = tt_ - th * p.tiles_w;
            const int hi0 = 2 * (2 * th * p.PH - 1) - 3;              // first input row of the patch
            const int e0 = 3 * (2 * (2 * tw * p.PW - 1) - 3 - 1);     // first element of a patch row: one pixel early, so even
            const unsigned short* ximg = reinterpret_cast<const unsigned short*>(p.x) + (size_t)n * p.H * p.W * 3;
            const uint32_t dst0 = smem_u32(inp + b * patch_words) + 4u * tid;
#pragma unroll
            for (int k = 0; k < MAX_SLOTS; ++k) {
                if (slot_rr[k] >= 0) {
                    const int hi = hi0 + slot_rr[k];
                    const int e = e0 + slot_e[k];                      // element index inside the image row (even)
                    const bool ok = hi >= 0 && hi < p.H && e >= 0 && e + 1 < row_elems;
                    const unsigned short* src = ximg + (ok ? hi * row_elems + e : 0);
                    cp_async4_zfill(dst0 + 512u * k, src, ok);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        int it = 0;
        if ((int)blockIdx.x < total) load_patch(blockIdx.x, 0);
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++it) {
            const int b = it & 1, u = it >> 1;
            const int tn = t + gridDim.x;
            if (tn < total) load_patch(tn, b ^ 1);
            else asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 1;" ::: "memory");       // this tile's patch has landed (for this thread)
            asm volatile("bar.sync 2, 128;" ::: "memory");             // ... and for the other producers
            bool ok = mbar_wait(&sh.aempty[b], (u & 1) ^ 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (!*abort_flag) report_timeout(p.status, 41, t);
                *abort_flag = 1;
                break;
            }
            if (row_used) {
                uint8_t* At = As + b * S_A_BYTES;
                const uint32_t* src = inp + b * patch_words;
#pragma unroll
                for (int r = 0; r < 7; ++r) {
                    // tap-row r of this pixel: 24 elements (12 words) starting at patch row 2*pi + r, element 6*pj + 3
                    // (+3: the patch starts one pixel early)
                    const uint32_t* s32 = src + (2 * pi + r) * in_words;
                    const int e0 = 6 * pj + 3;                         // odd element index -> words straddle: realign below
                    uint32_t wv[13];
#pragma unroll
                    for (int k = 0; k < 13; ++k) wv[k] = s32[(e0 >> 1) + k];
                    uint32_t ov[12];
#pragma unroll
                    for (int k = 0; k < 12; ++k) ov[k] = __funnelshift_r(wv[k], wv[k + 1], 16);   // drop the leading half word
#pragma unroll
                    for (int m = 0; m < 3; ++m) {
                        const int q = 3 * r + m;                       // 16-byte chunk index along K'
                        const uint32_t off = (uint32_t)(q >> 3) * P_A_BYTES + swz128(tid, q & 7);
                        *reinterpret_cast<uint4*>(At + off) = make_uint4(ov[4 * m], ov[4 * m + 1], ov[4 * m + 2], ov[4 * m + 3]);
                    }
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(&sh.afull[b]);
            asm volatile("bar.sync 2, 128;" ::: "memory");             // everyone is done reading this patch buffer
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else if (warp == 4) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(TILE_M, 64);
            const uint32_t b_lo = sdesc_lo(smem_u32(Bs));
            int it = 0;
            for (int t = blockIdx.x; t < total; t += gridDim.x, ++it) {
                const int b = it & 1, u = it >> 1;
                if (!mbar_wait(&sh.tempty[b], (u & 1) ^ 1, abort_flag) || !mbar_wait(&sh.afull[b], u & 1, abort_flag)) {
                    if (!*abort_flag) report_timeout(p.status, 42, t);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d = tmem + (uint32_t)(b * 64);
                const uint32_t a_lo = sdesc_lo(smem_u32(As + b * S_A_BYTES));
#pragma unroll
                for (int kk = 0; kk < 11; ++kk) {                      // K' = 176 of 192: the rest is zero weights
                    const uint32_t sub = kk >> 2, k4 = kk & 3;
                    umma_bf16_lo<false>(d, a_lo + sub * (P_A_BYTES >> 4) + 2 * k4, b_lo + sub * ((64 * 128) >> 4) + 2 * k4, idesc, kk > 0, 1u);
                }
                umma_commit(&sh.aempty[b]);
                umma_commit(&sh.tfull[b]);
            }
        }
        __syncwarp();
    } else {
        // two epilogue groups (warps 5-8 and 9-12; each covers the four TMEM lane quarters): group g takes
        // the tiles whose accumulator buffer is g
        const int g = (warp - 5) >> 2;
        const int q = warp & 3;
        const int row = q * 32 + lane;
        for (int t = blockIdx.x + g * gridDim.x, u = 0; t < total; t += 2 * gridDim.x, ++u) {
            const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.tfull[g], u & 1, abort_flag));
            if (!ok) {
                if (!*abort_flag) report_timeout(p.status, 44, t);
                *abort_flag = 1;
                break;
            }
            tc_fence_after();
            uint64_t* te = &sh.tempty[g];
            fused_epilogue<false>(p, t, tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g * 64), fe_stage + g * fe_bytes, row, 1 + 2 * g, [&]() {
                __syncwarp();
                if (lane == 0) mbar_arrive(te);
            });
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) {}
        __syncthreads();
    }
    if (warp == 4) tmem_dealloc(tmem, 128);
}

// ---- host --------------------------------------------------------------------------------
bool conv_patch_tma_supports(const ConvParams& p) {
    if (!p.patch || !fe_supports(p)) return false;
    if (p.stride != 1 || (p.Cin & 7) || p.Cin < 64 || p.k > 15) return false;
    const int stage_bytes = P_A_BYTES + ((p.Nt * 128 + 1023) & ~1023);
    return 2 * stage_bytes + fe_smem_bytes(p) + 2048 <= P_SMEM_MAX;
}

int conv_patch_tma_launch(const ConvParams& p, cudaStream_t stream) {
    if (!conv_patch_tma_supports(p)) return DR_ERR_UNSUPPORTED;
    static PerDeviceFlag attr_set;
    if (!attr_set.get()) {
        if (cudaFuncSetAttribute(conv_patch_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_MAX) != cudaSuccess) return DR_ERR_CUDA;
        attr_set.set();
    }
    alignas(64) CUtensorMap map_a, map_b;
    {
        const cuuint64_t dims[4] = {(cuuint64_t)p.Cin, (cuuint64_t)p.W, (cuuint64_t)p.H, (cuuint64_t)p.B};
        const cuuint64_t strides[3] = {(cuuint64_t)p.Cin * 2, (cuuint64_t)p.W * p.Cin * 2, (cuuint64_t)p.H * p.W * p.Cin * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)(2 * p.PW + 1), (cuuint32_t)(2 * p.PH + 1), 1};
        if (tmap_tiled(&map_a, 4, p.x, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B) != DR_OK) return DR_ERR_CUDA;
    }
    {
        const cuuint64_t dims[3] = {(cuuint64_t)p.Cin, (cuuint64_t)(p.k * p.k), (cuuint64_t)p.Cout};
        const cuuint64_t strides[2] = {(cuuint64_t)p.Cin * 2, (cuuint64_t)p.K * 2};
        const cuuint32_t box[3] = {64, 1, (cuuint32_t)p.Nt};
        if (tmap_tiled(&map_b, 3, p.w, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B) != DR_OK) return DR_ERR_CUDA;
    }
    if (p.m_tiles <= 0) return DR_OK;
    // CTA pairs with each CTA's half of the filter bank resident in shared memory (or, if that does not fit, streamed):
    // the filters are what this layer moves most of otherwise.  Measured on GoogLeNet conv2 at batch 256.
    if (tunable("DR_PATCH_PAIR", 1) != 0 && p.m_tiles >= 2 && (p.Nt & 31) == 0) {
        static PerDeviceFlag pair_attr;
        static int max_clusters_dev[64] = {};
        int& max_clusters = max_clusters_dev[PerDeviceFlag::dev()];
        const int nkb = p.k * p.k * ((p.Cin + 63) / 64);
        const int bsub = ((p.Nt / 2) * 128 + 1023) & ~1023;
        const int budget = P_SMEM_MAX - 2048;
        const int fe = fe_smem_bytes(p);
        int groups = 0, stages = 0, resident = 0, stage_bytes = 0;
        const int res_pref = tunable("DR_PATCH_RESIDENT", -1);
        // two epilogue groups first (the fused LRN / pooling epilogue is what bounds these layers: conv2 takes 336 us with
        // two groups and streamed half-filters, 433 us with one group and resident filters), then resident filters
        const int g_pref = tunable("DR_PATCH_PAIR_GROUPS", 0);
        for (int g = 2; g >= 1 && !groups; --g)
            for (int res = 1; res >= 0 && !groups; --res) {
                if (res_pref >= 0 && res != res_pref) continue;
                if (g_pref > 0 && g != g_pref) continue;
                const int sb = P_A_BYTES + (res ? 0 : bsub);
                const int left = budget - g * fe - (res ? nkb * bsub : 0);
                if (left / sb >= 3) { groups = g; resident = res; stage_bytes = sb; stages = left / sb; }
            }
        if (groups) {
            if (stages > P_MAX_STAGES) stages = P_MAX_STAGES;
            const int forced_stages = tunable("DR_PATCH_STAGES", 0);
            if (forced_stages >= 2 && forced_stages < stages) stages = forced_stages;
            cudaLaunchConfig_t cfg = {};
            cudaLaunchAttribute attr[2];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // used when p.pdl_wait: the producer waits before its first activation load
            attr[1].val.programmaticStreamSerializationAllowed = 1;
            // two warps per row for the drain where the LRN comes first (see the kernel's comment)
            const bool split = fe_split_supports(p) && tunable("DR_PATCH_SPLIT", 1) != 0;
            cfg.blockDim = dim3(split ? PP_THREADS_SPLIT : PP_THREADS); cfg.stream = stream; cfg.attrs = attr; cfg.numAttrs = 1;
            if (!pair_attr.get()) {
                if (cudaFuncSetAttribute(conv_patch_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_MAX) != cudaSuccess) return DR_ERR_CUDA;
                if (cudaFuncSetAttribute(conv_patch_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_MAX) != cudaSuccess) return DR_ERR_CUDA;
                int mc[2] = {0, 0};
                for (int v = 0; v < 2; ++v) {
                    cudaLaunchConfig_t q = cfg;
                    q.blockDim = dim3(v ? PP_THREADS_SPLIT : PP_THREADS);
                    q.gridDim = dim3(2 * num_sms());
                    q.dynamicSmemBytes = (size_t)P_SMEM_MAX;
                    const cudaError_t e = v ? cudaOccupancyMaxActiveClusters(&mc[v], conv_patch_pair_kernel<true>, &q)
                                            : cudaOccupancyMaxActiveClusters(&mc[v], conv_patch_pair_kernel<false>, &q);
                    if (e != cudaSuccess || mc[v] < 1) return DR_ERR_CUDA;
                }
                max_clusters = mc[0] < mc[1] ? mc[0] : mc[1];
                pair_attr.set();
            }
            alignas(64) CUtensorMap map_bh;
            const cuuint64_t dims[3] = {(cuuint64_t)p.Cin, (cuuint64_t)(p.k * p.k), (cuuint64_t)p.Cout};
            const cuuint64_t strides[2] = {(cuuint64_t)p.Cin * 2, (cuuint64_t)p.K * 2};
            const cuuint32_t box[3] = {64, 1, (cuuint32_t)(p.Nt / 2)};      // each CTA of a pair holds half of the filters
            if (tmap_tiled(&map_bh, 3, p.w, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B) != DR_OK) return DR_ERR_CUDA;
            int smem_bytes = stages * stage_bytes + (resident ? nkb * bsub : 0) + groups * fe + 1024;
            if (smem_bytes < 120 * 1024) smem_bytes = 120 * 1024;
            const int units = (p.m_tiles + 1) / 2;
            const int pairs = units < max_clusters ? units : max_clusters;
            cfg.gridDim = dim3(2 * pairs);
            cfg.dynamicSmemBytes = (size_t)smem_bytes;
            cfg.numAttrs = p.pdl_wait ? 2 : 1;
            const cudaError_t le = split ? cudaLaunchKernelEx(&cfg, conv_patch_pair_kernel<true>, p, map_a, map_bh, stages, stage_bytes, groups, resident, bsub)
                                         : cudaLaunchKernelEx(&cfg, conv_patch_pair_kernel<false>, p, map_a, map_bh, stages, stage_bytes, groups, resident, bsub);
            if (le != cudaSuccess) return DR_ERR_CUDA;
            count_launch();
            return launch_status();
        }
    }
    const int stage_bytes = P_A_BYTES + ((p.Nt * 128 + 1023) & ~1023);
    // two epilogue groups when that still leaves three pipeline stages, else one group and the extra stages
    // (conv2 of GoogLeNet: 350 us with 2 groups / 3 stages, 361 us with 1 group / 4 stages)
    int groups = (P_SMEM_MAX - 2048 - 2 * fe_smem_bytes(p)) / stage_bytes >= 3 ? 2 : 1;
    if (getenv("DR_PATCH_GROUPS")) groups = atoi(getenv("DR_PATCH_GROUPS")) == 2 ? 2 : 1;
    if (groups == 2 && (P_SMEM_MAX - 2048 - 2 * fe_smem_bytes(p)) / stage_bytes < 2) groups = 1;
    int stages = (P_SMEM_MAX - 2048 - groups * fe_smem_bytes(p)) / stage_bytes;
    if (stages > P_MAX_STAGES) stages = P_MAX_STAGES;
    int smem_bytes = stages * stage_bytes + groups * fe_smem_bytes(p) + 1024;
    if (smem_bytes < 120 * 1024) smem_bytes = 120 * 1024;     // one CTA per SM: each CTA takes all of TMEM
    const int grid = p.m_tiles < num_sms() ? p.m_tiles : num_sms();
    conv_patch_tma_kernel<<<grid, P_THREADS, smem_bytes, stream>>>(p, map_a, map_b, stages, stage_bytes, groups);
    count_launch();
    return launch_status();
}

static void stem_patch_dims(const ConvParams& p, int* rows, int* words) {
    *rows = 2 * (2 * p.PH + 1) + 5;                                   // input rows under the conv patch
    const int pixels = 2 * (2 * p.PW + 1) + 5 + 1 + 1;                // + one early pixel (alignment) + one late (13th word)
    *words = (3 * pixels + 1) / 2 + 1;
}

bool conv_stem_supports(const ConvParams& p) {
    if (!p.patch || !fe_supports(p)) return false;
    if (p.k != 7 || p.stride != 2 || p.pad != 3 || p.Cin != 3 || p.Cout != 64 || (p.W & 1)) return false;
    int rows, words;
    stem_patch_dims(p, &rows, &words);
    if (rows * words > 12 * 128) return false;                         // word slots per producer thread
    return S_B_BYTES + 2 * S_A_BYTES + 2 * fe_smem_bytes(p) + 2 * rows * words * 4 + 2048 <= P_SMEM_MAX;
}

int conv_stem_launch(const ConvParams& p, cudaStream_t stream) {
    if (!conv_stem_supports(p)) return DR_ERR_UNSUPPORTED;
    static PerDeviceFlag attr_set;
    if (!attr_set.get()) {
        if (cudaFuncSetAttribute(conv_stem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_MAX) != cudaSuccess) return DR_ERR_CUDA;
        attr_set.set();
    }
    if (p.m_tiles <= 0) return DR_OK;
    int rows, words;
    stem_patch_dims(p, &rows, &words);
    const int smem_bytes = S_B_BYTES + 2 * S_A_BYTES + 2 * fe_smem_bytes(p) + 2 * rows * words * 4 + 1024;
    const int grid = p.m_tiles < num_sms() ? p.m_tiles : num_sms();
    conv_stem_kernel<<<grid, S_THREADS, smem_bytes, stream>>>(p, rows, words);
    count_launch();
    return launch_status();
}

}  // namespace dr
