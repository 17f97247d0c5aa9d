// Split-K implicit-GEMM convolution for layers with few output tiles (single-image inference, the
// regime the paper times: one forward pass of one image, Section 4.1).
//
// At batch 1 the 14x14 and 7x7 stages of GoogLeNet have 196 and 49 output pixels: one or two
// 128-row tiles.  The persistent kernel of conv_umma.cu would run such a layer on a handful of SMs,
// each walking the whole K = k*k*Cin (up to 20800) alone while the layer's weights (up to 27 MB)
// trickle in through one SM's load path.  Here the K range of every output tile is cut into
// `splits` slices, one CTA per (tile, n-block, slice), so that the whole GPU streams the weights:
//
//   1. each CTA multiplies its K slice (TMA im2col / tiled loads -> shared memory -> tcgen05.mma,
//      accumulator in tensor memory) exactly like the persistent kernel does;
//   2. it writes its float32 partial tile to scratch memory and arrives on the tile's counter;
//   3. it waits until all slices of the tile have arrived (the grid is launched cooperatively, i.e.
//      every CTA is resident, so the wait ends; it is bounded all the same);
//   4. it sums 1/splits of the tile over all partials, each element in slice order 0..splits-1 — a fixed order, so
//      the result does not depend on timing — applies bias / ReLU / residual and stores bf16 or f32.
//
// Scratch memory: `counters` (one int per output tile, zero on entry, back at zero when the kernel has finished) and `scratch`
// (tiles x splits x Nt/4 x 128 float4, contents irrelevant on entry).
//
// Cluster form of steps 2-4 (the short jobs of an inception module, where the hand-over is most of the time): the
// slices of a tile are the CTAs of one thread-block cluster; each keeps its partial tile in its own shared memory,
// a cluster barrier replaces the counter, and every CTA sums its share over the cluster's shared memories
// (distributed shared memory) in slice order: no trip through L2, the same fixed summation order.
#include <map>
#include <mutex>
#include <utility>

#include "conv_common.cuh"
#include "umma_ptx.cuh"

namespace dr {
using namespace ptx;

constexpr int SK_A_BYTES = TILE_M * 128;        // 128 pixels x 64 bf16
constexpr int SK_MAX_STAGES = 12;
constexpr int SK_THREADS = 192;                 // warp 0: TMA producer, warp 1: MMA issue + TMEM owner, warps 2-5: drain; all: reduction
constexpr int SK_SMEM_MAX = 227 * 1024 - 2048;  // dynamic part
constexpr int SK_MAX_TILES = DR_CONV_WS_COUNTER_BYTES / 4;

struct SkShared {
    uint64_t full[SK_MAX_STAGES], empty[SK_MAX_STAGES], accum;
    uint32_t tmem_base;
    int abort;
};

struct SkPlan {
    int nt, n_blocks, splits, kps, nkb, stages, sub_bytes;
    int cluster;              // slices of a tile = ranks of a cluster of `splits` CTAs
    int own_ctas;             // (job 2 of a group) runs on CTAs of its own rather than behind job 1
    uint32_t tmem_cols;
    size_t scratch_bytes;
};

__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// One job = one convolution layer cut into (tile, n-block, slice) work items.  A launch carries up to three jobs
// of one inception module: CTAs [0, small_begin) work on job 0 (the merged 5x5 branch); the remaining "small group"
// works on job 1 (the 1x1 reducer, which reads the same input as job 0) and then, once every CTA of job 1 has
// stored its output, on job 2 (the 3x3 convolution that reads the reducer's output).
struct alignas(64) SkJob {
    CUtensorMap map_a, map_b;
    ConvParams p;
    int a_mode, stages, sub_bytes, splits, kps;
    int cluster;              // 1: the slices of a tile are the ranks of a cluster (splits = cluster size); partials in shared memory
    int ctas;                 // work items of this job = tiles x slices
    uint32_t tmem_cols;
    float* scratch;
    int* counters;
};
struct SkJobs {
    SkJob j[3];
    int n;                    // 1, 2 or 3 jobs
    int cs;                   // cluster size of the launch (1: no clusters)
    int small_begin;          // first CTA of the small group (n >= 2)
    int c_begin;              // n == 3: first CTA of job 2; == small_begin when jobs 1 and 2 share their CTAs, beyond job 1's otherwise
    int* dep;                 // n == 3: counter on which job 2 waits for job 1
};

__device__ __forceinline__ void red_inc_gpu(int* p, unsigned wrap) {
    asm volatile("red.relaxed.gpu.global.inc.u32 [%0], %1;" ::"l"(p), "r"(wrap) : "memory");
}

// The whole CTA runs work item `bid` of job J.  `first`: this is the CTA's first job (wait for the previous kernel
// of the stream after the filter prefetch).  `dep_wait` >= 0: before reading its input, wait until *dep has
// reached dep_wait (the producing job's CTA count).  `dep_wrap` > 0: announce on *dep when this CTA is done with
// the job (producers: after their stores; consumers: after the wait), the counter wrapping to 0 at dep_wrap.
__device__ __forceinline__ void sk_run_job(const SkJob* const J, const int bid, SkShared& sh, uint8_t* smem, const uint32_t tmem,
                                           const bool first, int* dep, const int dep_wait, const bool dep_signal, const unsigned dep_wrap) {
    const ConvParams& p = J->p;
    const CUtensorMap& map_a = J->map_a;
    const CUtensorMap& map_b = J->map_b;
    const int a_mode = J->a_mode, stages = J->stages, sub_bytes = J->sub_bytes, splits = J->splits, kps = J->kps;
    float* __restrict__ scratch = J->scratch;
    int* __restrict__ counters = J->counters;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // work item of this CTA: K slice `split` of output tile (mt, nb); in the cluster form the slice is the cluster rank
    // (the job's first CTA starts a cluster) and trailing slices may be empty (they contribute zeros)
    const bool clustered = J->cluster != 0;
    const int split = bid % splits, tile = bid / splits;
    const int nb = tile / p.m_tiles, mt = tile - nb * p.m_tiles;
    const int n0 = nb * p.Nt;
    const int cout16 = (p.Cout + 15) & ~15;
    const int Nj = min(p.Nt, cout16 - n0);
    const int cpb = (p.Cin + 63) >> 6;
    const int nkb = p.k * p.k * cpb;
    const int kb0 = min(nkb, split * kps), kb1 = min(nkb, kb0 + kps);

    volatile int* abort_flag = &sh.abort;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full0 = smem_u32(&sh.full[0]), empty0 = smem_u32(&sh.empty[0]);

    if (warp == 0) {
        if (lane == 0) {
            // -------------------------------------------- TMA producer
            const uint32_t tx = SK_A_BYTES + (uint32_t)p.Nt * 128;
            const long long m0 = (long long)mt * TILE_M;
            const int hw = p.Ho * p.Wo;
            const int img = (int)(m0 / hw);
            const int rem = (int)(m0 - (long long)img * hw);
            const int ho = rem / p.Wo, wo = rem - ho * p.Wo;
            const int hb = ho * p.stride - p.pad, wb = wo * p.stride - p.pad;
            int tap = kb0 / cpb;
            int c0 = (kb0 - tap * cpb) << 6;
            int r = tap / p.k, tt = tap - r * p.k;
            // The filters do not depend on the layer before this one: their loads for the first round of pipeline
            // stages go out before the wait for that layer, so the weights stream in while it finishes.
            const int npre = min(stages, kb1 - kb0);
            {
                int tap_b = tap, c0_b = c0;
                for (int i = 0; i < npre; ++i) {
                    const uint32_t fb = full0 + 8 * i;
                    mbar_expect_tx_u32(fb, tx);
                    tma_load_3d_u32<false>(smem_base + (uint32_t)i * (uint32_t)sub_bytes + SK_A_BYTES, &map_b, fb, c0_b, tap_b, n0, 1u);
                    c0_b += 64;
                    if (c0_b >= p.Cin) { c0_b = 0; ++tap_b; }
                }
            }
            if (first) grid_dependency_wait();
            if (dep_wait >= 0) {
                // the input of this job is written by another job of this launch
                const long long t0 = clock64();
                while (ld_acquire_gpu(dep) < dep_wait) {
                    if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
                        if (!*abort_flag) report_timeout(p.status, 25, tile);
                        *abort_flag = 1;
                        break;
                    }
                }
                fence_proxy_async_all();      // those writes went through the generic proxy; the loads below are TMA's
                red_inc_gpu(dep, dep_wrap);   // consumers count too, so that the last of them wraps the counter to zero
            }
            int s = 0;
            uint32_t ph = 0;
            for (int kb = kb0; kb < kb1; ++kb) {
                const int i = kb - kb0;
                if (i >= stages && !mbar_wait_u32(empty0 + 8 * s, ph ^ 1, abort_flag)) {
                    if (!*abort_flag) report_timeout(p.status, 21, tile);
                    *abort_flag = 1;
                    break;
                }
                const uint32_t dst = smem_base + (uint32_t)s * (uint32_t)sub_bytes;
                const uint32_t fb = full0 + 8 * s;
                if (i >= npre) mbar_expect_tx_u32(fb, tx);
                if (a_mode == 0) tma_load_2d_u32<false>(dst, &map_a, fb, c0, (int)m0, 1u);
                else tma_load_im2col_4d_u32<false>(dst, &map_a, fb, c0, wb, hb, img, (uint16_t)tt, (uint16_t)r, 1u);
                if (i >= npre) tma_load_3d_u32<false>(dst + SK_A_BYTES, &map_b, fb, c0, tap, n0, 1u);
                c0 += 64;
                if (c0 >= p.Cin) {
                    c0 = 0; ++tap; ++tt;
                    if (tt == p.k) { tt = 0; ++r; }
                }
                if (++s == stages) { s = 0; ph ^= 1; }
            }
        }
        __syncwarp();
        if (first && lane != 0) grid_dependency_wait();
    } else if (warp == 1) {
        if (lane == 0) {
            // -------------------------------------------- MMA issue
            const uint32_t idesc = make_idesc_bf16(TILE_M, Nj);
            const int last_nk16 = ((p.Cin - ((cpb - 1) << 6)) + 15) >> 4;
            int cc = kb0 % cpb;
            int s = 0;
            uint32_t ph = 0, accum = 0;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!mbar_wait_u32(full0 + 8 * s, ph, abort_flag)) {
                    if (!*abort_flag) report_timeout(p.status, 22, tile);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t a = smem_base + (uint32_t)s * (uint32_t)sub_bytes;
                const uint32_t alo = sdesc_lo(a), blo = sdesc_lo(a + SK_A_BYTES);
                const int nk16 = (cc == cpb - 1) ? last_nk16 : 4;
                cc = (cc + 1 == cpb) ? 0 : cc + 1;
                umma_bf16_lo<false>(tmem, alo, blo, idesc, accum, 1u);
                accum = 1;
                umma_bf16_lo<false>(tmem, alo + 2, blo + 2, idesc, 1u, nk16 > 1);
                umma_bf16_lo<false>(tmem, alo + 4, blo + 4, idesc, 1u, nk16 > 2);
                umma_bf16_lo<false>(tmem, alo + 6, blo + 6, idesc, 1u, nk16 > 3);
                umma_commit_u32<false>(empty0 + 8 * s);
                if (++s == stages) { s = 0; ph ^= 1; }
            }
            umma_commit_u32<false>(smem_u32(&sh.accum));   // also on a timeout: fires once whatever was issued has finished
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ drain: float32 partial tile -> scratch.  TMEM lane quarter = warp % 4.
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.accum, 0, abort_flag));
        if (!ok) {
            if (!*abort_flag) report_timeout(p.status, 23, tile);
            *abort_flag = 1;
        } else if (!*abort_flag) {
            tc_fence_after();
            const long long m = (long long)mt * TILE_M + row;
            const bool row_ok = m < p.M;
            const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16);
            // partial tile layout [column quad][row]: the 32 rows of a warp are 512 contiguous bytes per store
            // (cluster form: in this CTA's shared memory, where the pipeline stages were)
            float4* dst = (clustered ? reinterpret_cast<float4*>(smem) : reinterpret_cast<float4*>(scratch + ((size_t)tile * splits + split) * TILE_M * p.Nt)) + row;
            const bool empty = kb1 <= kb0;                 // no k-block in this slice: the accumulator was never written
            int c = 0;
            for (; c + 32 <= Nj; c += 32) {
                uint32_t v[32];
                tmem_ld_x32(taddr + c, v);
                tmem_ld_wait();
                if (empty) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        dst[((c >> 2) + j) * TILE_M] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                                        __uint_as_float(v[4 * j + 3]));
                }
            }
            if (c < Nj) {   // 16-column tail
                uint32_t v[16];
                tmem_ld_x16(taddr + c, v);
                tmem_ld_wait();
                if (empty) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0u;
                }
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        dst[((c >> 2) + j) * TILE_M] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                                        __uint_as_float(v[4 * j + 3]));
                }
            }
        }
    }

    // ---------------------------------------------------- all slices of the tile meet here
    // This CTA's share of the tile: elements [f0, f1) of the Nj/4 x valid_rows float4 values (column quad major, so
    // that consecutive threads read consecutive rows of the partial tiles).  A thread owns up to four elements
    // (e, e + 192, ...) and sums their slices in order 0..splits-1, sixteen loads in flight.
    const long long mrem = p.M - (long long)mt * TILE_M;
    const int valid_rows = mrem < TILE_M ? (int)mrem : TILE_M;
    const int nq = Nj >> 2;
    const int total = valid_rows * nq;
    const int per = (total + splits - 1) / splits;
    const int f0 = split * per, f1 = min(total, f0 + per);
    tc_fence_before();
    __syncthreads();                     // the whole partial tile has been written (by this CTA's threads, in CTA order)
    if (clustered) cluster_sync_all();   // ... and so have the partial tiles of the other slices (every thread of the cluster arrives)
    if (!clustered && tid == 0) {
        __threadfence();                 // ... and is visible device-wide before the arrival is (cumulative over the barrier)
        // the counter runs 0 .. 2*splits-1 and wraps to zero: first arrivals take it to `splits`, second ones back to 0
        const unsigned old = atomicInc(reinterpret_cast<unsigned*>(&counters[tile]), 2u * (unsigned)splits - 1u);
        if ((int)old + 1 < splits) {     // arrives even after a timeout above, so that the other slices do not wait for nothing
            const long long t0 = clock64();
            while (ld_acquire_gpu(&counters[tile]) < splits) {
                if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
                    if (!*abort_flag) report_timeout(p.status, 24, tile);
                    *abort_flag = 1;
                    break;
                }
            }
        }
        __threadfence();
    }
    __syncthreads();

    if (!*abort_flag) {
        const size_t slice4 = (size_t)TILE_M * (p.Nt >> 2);      // float4 per partial tile
        const float4* part = reinterpret_cast<const float4*>(scratch) + (size_t)tile * splits * slice4;
        const bool f32 = p.flags & DR_OUT_F32;
        for (int base = f0 + tid; base < f1; base += 4 * SK_THREADS) {
            int row[4], col[4];
            const float4* src[4];
            uint32_t soff[4];
            float4 acc[4], bias[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int e = min(base + q * SK_THREADS, f1 - 1);          // clamped: the extra sums are not stored
                const int cq = e / valid_rows;
                row[q] = e - cq * valid_rows;
                col[q] = n0 + 4 * cq;
                src[q] = part + (size_t)cq * TILE_M + row[q];
                soff[q] = (uint32_t)(cq * TILE_M + row[q]) * 16u;
                acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                bias[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                if ((p.flags & DR_BIAS) && col[q] < p.Cout)
                    bias[q] = make_float4(__ldg(p.bias + col[q]), __ldg(p.bias + col[q] + 1), __ldg(p.bias + col[q] + 2), __ldg(p.bias + col[q] + 3));
            }
#pragma unroll 4
            for (int sp = 0; sp < splits; ++sp) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float4 v = clustered ? ld_shared_cluster_f4(mapa_shared(smem_base, (uint32_t)sp) + soff[q]) : __ldcg(src[q] + (size_t)sp * slice4);
                    acc[q].x += v.x; acc[q].y += v.y; acc[q].z += v.z; acc[q].w += v.w;
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (base + q * SK_THREADS >= f1 || col[q] >= p.Cout) continue;
                float4 a = acc[q];
                const long long m = (long long)mt * TILE_M + row[q];
                a.x += bias[q].x; a.y += bias[q].y; a.z += bias[q].z; a.w += bias[q].w;
                if (p.flags & DR_RELU) { a.x = fmaxf(a.x, 0.f); a.y = fmaxf(a.y, 0.f); a.z = fmaxf(a.z, 0.f); a.w = fmaxf(a.w, 0.f); }
                if (p.flags & DR_RESIDUAL) {
                    const uint2 u = __ldg(reinterpret_cast<const uint2*>(p.residual + m * p.Cout + col[q]));
                    a.x += bf16_lo(u.x); a.y += bf16_hi(u.x); a.z += bf16_lo(u.y); a.w += bf16_hi(u.y);
                    if (p.flags & DR_RELU_AFTER_RESIDUAL) { a.x = fmaxf(a.x, 0.f); a.y = fmaxf(a.y, 0.f); a.z = fmaxf(a.z, 0.f); a.w = fmaxf(a.w, 0.f); }
                }
                if (f32) {
                    *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.y) + m * p.ldc + p.coff + col[q]) = a;
                } else {
                    uint2 o;
                    o.x = pack_bf16(a.x, a.y);
                    o.y = pack_bf16(a.z, a.w);
                    *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.y) + m * p.ldc + p.coff + col[q]) = o;
                }
            }
        }
    }

    __syncthreads();                     // every thread of this CTA has finished reading the partials and has stored its outputs
    if (tid == 0) {
        // second arrival, not waited for: the last of them wraps the counter back to zero
        if (!clustered) red_inc_gpu(&counters[tile], 2u * (unsigned)splits - 1u);
        if (dep_signal) {                // this CTA's share of the job's output is in memory: tell the job that reads it
            __threadfence();
            red_inc_gpu(dep, dep_wrap);
        }
    }
    if (clustered) cluster_sync_all();   // no CTA of the cluster reads this one's shared memory any more (it may be refilled, or the CTA may exit)
}

__global__ void __launch_bounds__(SK_THREADS, 1) conv_splitk_kernel(const __grid_constant__ SkJobs jobs) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ SkShared sh;
    const int tid = threadIdx.x, warp = tid >> 5;
    const bool small = jobs.n >= 2 && (int)blockIdx.x >= jobs.small_begin;
    // job 2 on CTAs of its own (they request their filters at once and wait for job 1 with nothing else to do), or behind
    // job 1 on the same CTAs
    const bool own_c = jobs.n == 3 && jobs.c_begin > jobs.small_begin && (int)blockIdx.x >= jobs.c_begin;
    const int bid = own_c ? (int)blockIdx.x - jobs.c_begin : small ? (int)blockIdx.x - jobs.small_begin : (int)blockIdx.x;
    const int j0 = own_c ? 2 : small ? 1 : 0;                   // first job of this CTA
    const int j1 = (small && jobs.n == 3 && jobs.c_begin == jobs.small_begin) ? 2 : j0;   // last job of this CTA
    uint32_t tmem_cols = 32;
    for (int j = j0; j <= j1; ++j) tmem_cols = max(tmem_cols, jobs.j[j].tmem_cols);

    if (tid == 0) {
        for (int s = 0; s < SK_MAX_STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        sh.abort = 0;
        fence_barrier_init();
        // the descriptors of every job this CTA will run, ahead of their first use
        for (int j = j0; j <= j1; ++j) { prefetch_tensormap(&jobs.j[j].map_a); prefetch_tensormap(&jobs.j[j].map_b); }
    }
    if (warp == 1) { tmem_alloc(&sh.tmem_base, tmem_cols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    // The next kernel in the stream may be scheduled from here on (it waits for this one to finish before it
    // touches anything this one writes).  Every warp but the producer's waits for the previous kernel right away; the
    // producer's warp as a whole waits after the filter prefetch (lanes parked in the wait would hold lane 0 back).
    grid_launch_dependents();
    if (warp != 0) grid_dependency_wait();

    const unsigned dep_wrap = jobs.n == 3 ? (unsigned)(jobs.j[1].ctas + jobs.j[2].ctas - 1) : 0u;
    for (int j = j0; j <= j1; ++j) {
        if (j != j0) {
            // same CTA, next job: barriers start over (their phases depend on how many k-blocks the last job had)
            __syncthreads();
            if (tid == 0) {
                for (int s = 0; s < SK_MAX_STAGES; ++s) {
                    mbar_inval(&sh.full[s]); mbar_inval(&sh.empty[s]);
                    mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1);
                }
                mbar_inval(&sh.accum);
                mbar_init(&sh.accum, 1);
                fence_barrier_init();
            }
            tc_fence_before();
            __syncthreads();
            tc_fence_after();
        }
        const bool has_work = bid < jobs.j[j].ctas;
        // one call site per job: inside each, the job's fields are kernel parameters at fixed offsets (constant-bank
        // operands); a job picked by a run-time index would be read through generic loads again and again
        if (has_work) {
            if (j == 0) sk_run_job(&jobs.j[0], bid, sh, smem, tmem, true, nullptr, -1, false, 0u);
            else if (j == 1) sk_run_job(&jobs.j[1], bid, sh, smem, tmem, true, jobs.dep, -1, jobs.n == 3, dep_wrap);
            else sk_run_job(&jobs.j[2], bid, sh, smem, tmem, j == j0, jobs.dep, jobs.j[1].ctas, false, dep_wrap);
        } else if (j == j0 && warp == 0) {
            grid_dependency_wait();
        }
    }
    __syncthreads();
    if (sh.abort) {   // give copies and MMAs still in flight time to land before shared memory and TMEM go away
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) {}
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem, tmem_cols);
}

// ---- host ---------------------------------------------------------------------------------
static bool splitk_shape_ok(const ConvParams& p) {
    if (p.flags & (DR_POOL | DR_LRN)) return false;
    if (p.patch) return false;
    if ((p.Cin & 7) || p.Cin < 64) return false;
    if ((p.Cout & 3) || (p.ldc & 3) || (p.coff & 3)) return false;
    if (p.k > 255 || p.M <= 0 || p.M > 0x7fffffffLL) return false;
    return true;
}

// Choice of n-block width and slice count for a layer that may use `budget` CTAs.  Measured on B200 (batch 1,
// GoogLeNet's inception layers): n-blocks of about 80 columns and at most 32 slices are within a microsecond of
// the best plan of every layer; a slice has at least two k-blocks unless `single` allows plans without splitting.
static bool splitk_plan_budget(const ConvParams& p, int budget, bool single, SkPlan* out, int s_cap = 0) {
    if (!splitk_shape_ok(p)) return false;
    const int cpb = (p.Cin + 63) >> 6;
    const int nkb = p.k * p.k * cpb;
    const int cout16 = (p.Cout + 15) & ~15;
    const int nb_min = (cout16 + 255) / 256;
    int nb = tunable("DR_SPLITK_NB", 0);
    if (nb <= 0) nb = (cout16 + 40) / 80;
    if (nb < nb_min) nb = nb_min;
    while (nb > nb_min && (long long)p.m_tiles * nb * (single ? 1 : 2) > budget) --nb;
    int nt = ((cout16 + nb - 1) / nb + 15) / 16 * 16;
    while ((long long)nt * (nb - 1) >= cout16 && nb > 1) { --nb; nt = ((cout16 + nb - 1) / nb + 15) / 16 * 16; }   // no empty block
    const long long tiles = (long long)p.m_tiles * nb;
    if (tiles > SK_MAX_TILES || tiles > budget) return false;
    int S = (int)(budget / tiles);
    if (S > nkb / 2) S = nkb / 2;
    int s_max = tunable("DR_SPLITK_S", 0);
    if (s_max <= 0) s_max = 32;
    if (S > s_max) S = s_max;
    if (s_cap > 0 && S > s_cap) S = s_cap;
    if (S < 1) S = 1;
    if (S < 2 && !single) return false;
    SkPlan b{};
    b.kps = (nkb + S - 1) / S;
    b.splits = (nkb + b.kps - 1) / b.kps;                               // no empty slice
    b.nt = nt; b.n_blocks = nb; b.nkb = nkb;
    b.sub_bytes = SK_A_BYTES + ((b.nt * 128 + 1023) & ~1023);
    int st = (tunable("DR_SPLITK_SMEM_KB", 200) * 1024 - 1024) / b.sub_bytes;
    if (st > SK_MAX_STAGES) st = SK_MAX_STAGES;
    if (st > b.kps) st = b.kps;
    b.stages = st;
    b.tmem_cols = 32;
    while ((int)b.tmem_cols < b.nt) b.tmem_cols <<= 1;
    b.scratch_bytes = ((size_t)p.m_tiles * b.n_blocks * b.splits * TILE_M * b.nt * sizeof(float) + 255) / 256 * 256;
    *out = b;
    return true;
}

// Cluster form of a short job: exactly `cs` slices per tile (trailing ones may be empty), n-blocks of about 80 columns,
// fewer if the job would not fit `budget` CTAs.
static bool splitk_plan_cluster(const ConvParams& p, int budget, int cs, SkPlan* out) {
    if (!splitk_shape_ok(p)) return false;
    const int cpb = (p.Cin + 63) >> 6;
    const int nkb = p.k * p.k * cpb;
    if (nkb < 2) return false;
    const int cout16 = (p.Cout + 15) & ~15;
    const int nb_min = (cout16 + 255) / 256;
    int nb = (cout16 + 40) / 80;
    if (nb < nb_min) nb = nb_min;
    while (nb > nb_min && (long long)p.m_tiles * nb * cs > budget) --nb;
    int nt = ((cout16 + nb - 1) / nb + 15) / 16 * 16;
    while ((long long)nt * (nb - 1) >= cout16 && nb > 1) { --nb; nt = ((cout16 + nb - 1) / nb + 15) / 16 * 16; }
    const long long tiles = (long long)p.m_tiles * nb;
    if (tiles > SK_MAX_TILES || tiles * cs > budget) return false;
    SkPlan b{};
    b.kps = (nkb + cs - 1) / cs;
    b.splits = cs;
    b.cluster = 1;
    b.nt = nt; b.n_blocks = nb; b.nkb = nkb;
    b.sub_bytes = SK_A_BYTES + ((b.nt * 128 + 1023) & ~1023);
    int st = (tunable("DR_SPLITK_SMEM_KB", 200) * 1024 - 1024) / b.sub_bytes;
    if (st > SK_MAX_STAGES) st = SK_MAX_STAGES;
    if (st > b.kps) st = b.kps;
    b.stages = st;
    b.tmem_cols = 32;
    while ((int)b.tmem_cols < b.nt) b.tmem_cols <<= 1;
    b.scratch_bytes = 0;                                  // partial tiles stay in shared memory
    *out = b;
    return true;
}

// A layer on its own: worth splitting when the persistent kernel would leave most of the GPU idle AND walk a long K
// per CTA.  Measured: from about 24 k-blocks on (16 when the layer has only one or two output tiles); below that
// the hand-over between the slices costs more than the shorter loop saves (the 1x1 reducers stay where they were).
static bool splitk_plan(const ConvParams& p, SkPlan* out) {
    if (!splitk_shape_ok(p)) return false;
    const int sms = num_sms();
    const int force = tunable("DR_SPLITK", -1);            // 0: never, 1: whenever the shape allows
    if (force == 0) return false;
    const int nkb = p.k * p.k * ((p.Cin + 63) >> 6);
    if (force != 1) {
        if ((long long)p.m_tiles * p.n_blocks * 2 > sms) return false;
        if (nkb < 16 || (nkb < 24 && p.m_tiles > 2)) return false;
    }
    if (nkb < 4) return false;
    return splitk_plan_budget(p, sms, false, out);
}

size_t conv_splitk_scratch_bytes(const ConvParams& p) {
    SkPlan pl;
    if (!splitk_plan(p, &pl)) return 0;
    return pl.scratch_bytes;
}

bool conv_splitk_supports(const ConvParams& p) {
    if (!p.sk_counters || !p.sk_scratch || ((uintptr_t)p.sk_scratch & 15)) return false;
    SkPlan pl;
    if (!splitk_plan(p, &pl)) return false;
    return p.sk_scratch_bytes >= pl.scratch_bytes;
}

// Layers of one inception module in one launch: `a` (the long one, job 0), `b` (a short one reading the same input:
// the 1x1 reducer, job 1) and optionally `c` (the convolution that reads b's output, job 2).  b and c share a small
// group of CTAs, a takes the rest.  Scratch: a's, then b's, then c's; counters: a's tiles, b's, c's, then the
// counter on which c waits for b.
static int group_smem_bytes(const SkPlan& pa, const SkPlan& pb, const SkPlan* pc) {
    int smem = pa.stages * pa.sub_bytes;
    const SkPlan* small[2] = {&pb, pc};
    for (const SkPlan* q : small) {
        if (!q) continue;
        if (q->stages * q->sub_bytes > smem) smem = q->stages * q->sub_bytes;
        if (q->cluster && q->nt * 512 > smem) smem = q->nt * 512;       // the partial tile of a cluster job lives where the stages were
    }
    return smem + 1024;
}

static int max_active_clusters(int cs, int smem_bytes);

static bool splitk_group_plan(const ConvParams& a, const ConvParams& b, const ConvParams* c, SkPlan* pa, SkPlan* pb, SkPlan* pc) {
    if (tunable("DR_SPLITK_PAIR", 1) == 0) return false;
    if (a.x != b.x || a.B != b.B || a.H != b.H || a.W != b.W || a.Cin != b.Cin) return false;
    const int small = tunable("DR_SPLITK_SMALL_CTAS", 48);
    // Cluster form for the two short jobs of a three-job launch (the chain reducer -> 3x3 is the critical path of a
    // module at batch 1); the long job keeps the hand-over through L2.  Every CTA of the launch must be resident at once.
    const int cs = tunable("DR_SPLITK_CLUSTER", 4);      // measured: 4 beats 8 (the device holds 33 clusters of 4, 15 of 8) and 2
    if (cs > 1 && cs <= 8 && c && c->x == b.y && c->Cin == b.Cout && b.ldc == b.Cout && b.coff == 0 && !(b.flags & DR_OUT_F32)) {
        SkPlan qb, qc, qa, alone;
        if (splitk_plan_cluster(b, small, cs, &qb) && splitk_plan_cluster(*c, small, cs, &qc) && splitk_plan(a, &alone)) {
            const int used_b = b.m_tiles * qb.n_blocks * cs, used_c = c->m_tiles * qc.n_blocks * cs;
            // CTAs of its own for the 3x3 where the long job keeps at least half of the device: a CTA that ran the reducer
            // first starts its 3x3 slice about 3 us after the others (barriers set up again, filters requested late)
            const bool own = tunable("DR_SPLITK_OWN_CTAS", 1) != 0 && used_b + used_c <= num_sms() / 2;
            const int used = own ? used_b + used_c : (used_b > used_c ? used_b : used_c);
            qc.own_ctas = own ? 1 : 0;
            // the device holds fewer CTAs in clusters than singly (a cluster sits inside one GPC): plan against that number
            const int smem_cap = tunable("DR_SPLITK_SMEM_KB", 200) * 1024 + 1024;
            int cap = max_active_clusters(cs, smem_cap) * cs;
            if (cap > num_sms()) cap = num_sms();
            const int budget_a = (cap - used) / cs * cs;
            if (budget_a >= 2 * cs && splitk_plan_budget(a, budget_a, false, &qa)) {
                const int ctas_a = (a.m_tiles * qa.n_blocks * qa.splits + cs - 1) / cs * cs;
                const long long tiles = (long long)a.m_tiles * qa.n_blocks + (long long)b.m_tiles * qb.n_blocks + (long long)c->m_tiles * qc.n_blocks + 1;
                if (tiles <= SK_MAX_TILES && group_smem_bytes(qa, qb, &qc) <= smem_cap && (ctas_a + used) <= cap) {
                    *pa = qa; *pb = qb; *pc = qc;
                    return true;
                }
            }
        }
    }
    if (!splitk_plan_budget(b, small, true, pb, tunable("DR_SPLITK_B_S", 0))) return false;
    int used = b.m_tiles * pb->n_blocks * pb->splits;
    long long tiles = (long long)b.m_tiles * pb->n_blocks;
    if (c) {
        if (c->x != b.y || c->Cin != b.Cout || b.ldc != b.Cout || b.coff != 0 || (b.flags & DR_OUT_F32)) return false;   // c reads b's dense output
        if (!splitk_plan_budget(*c, small, true, pc, tunable("DR_SPLITK_C_S", 0))) return false;
        const int used_c = c->m_tiles * pc->n_blocks * pc->splits;
        if (tunable("DR_SPLITK_OWN_CTAS", 1) != 0 && used + used_c <= num_sms() / 2) { used += used_c; pc->own_ctas = 1; }   // as in the cluster form
        else if (used_c > used) used = used_c;
        tiles += (long long)c->m_tiles * pc->n_blocks + 1;
    }
    SkPlan alone;
    if (!splitk_plan(a, &alone)) return false;                         // a must be a split-K layer in its own right
    if (!splitk_plan_budget(a, num_sms() - used, false, pa)) return false;
    if ((long long)a.m_tiles * pa->n_blocks + tiles > SK_MAX_TILES) return false;
    return true;
}

size_t conv_splitk_group_scratch_bytes(const ConvParams& a, const ConvParams& b, const ConvParams* c) {
    SkPlan pa, pb, pc{};
    if (!splitk_group_plan(a, b, c, &pa, &pb, &pc)) return 0;
    return pa.scratch_bytes + pb.scratch_bytes + (c ? pc.scratch_bytes : 0);
}

bool conv_splitk_group_supports(const ConvParams& a, const ConvParams& b, const ConvParams* c) {
    if (!a.sk_counters || !a.sk_scratch || ((uintptr_t)a.sk_scratch & 255)) return false;
    SkPlan pa, pb, pc{};
    if (!splitk_group_plan(a, b, c, &pa, &pb, &pc)) return false;
    return a.sk_scratch_bytes >= pa.scratch_bytes + pb.scratch_bytes + (c ? pc.scratch_bytes : 0);
}

static int fill_job(const ConvParams& p0, const SkPlan& pl, float* scratch, int* counters, SkJob* j) {
    j->p = p0;
    j->p.Nt = pl.nt;
    j->p.n_blocks = pl.n_blocks;
    const int est = encode_conv_maps(j->p, pl.nt, &j->map_a, &j->map_b, &j->a_mode);
    if (est != DR_OK) return est;
    j->stages = pl.stages; j->sub_bytes = pl.sub_bytes; j->splits = pl.splits; j->kps = pl.kps; j->tmem_cols = pl.tmem_cols;
    j->cluster = pl.cluster;
    j->scratch = scratch; j->counters = counters;
    j->ctas = p0.m_tiles * pl.n_blocks * pl.splits;
    return DR_OK;
}

static int launch_jobs(const SkJobs& jobs, int ctas, int smem_bytes, cudaStream_t stream) {
    static PerDeviceFlag attr_set;
    if (!attr_set.get()) {
        if (cudaFuncSetAttribute(conv_splitk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SK_SMEM_MAX) != cudaSuccess) return DR_ERR_CUDA;
        attr_set.set();
    }
    // Launch mode.  Programmatic (default): the kernel may start while the previous kernel of the stream drains, and
    // prefetches its filters meanwhile; the grid never exceeds the SM count, and the kernel before it never waits on
    // this one, so every slice becomes resident.  DR_SPLITK_PDL=0: a cooperative launch (residency checked by the
    // runtime), no overlap.
    const bool pdl = tunable("DR_SPLITK_PDL", 1) != 0 || jobs.cs > 1;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    if (pdl) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
    } else {
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
    }
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(SK_THREADS);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (jobs.cs > 1) {                   // residency of every cluster was checked when the plan was made
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)jobs.cs; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    if (cudaLaunchKernelEx(&cfg, conv_splitk_kernel, jobs) != cudaSuccess) {
        (void)cudaGetLastError();
        return DR_ERR_CUDA;
    }
    count_launch();
    return launch_status();
}

// How many clusters of `cs` CTAs with `smem_bytes` of dynamic shared memory the device holds at once (memoised).
static int max_active_clusters(int cs, int smem_bytes) {
    static std::mutex mu;
    static std::map<std::pair<int, int>, int> memo;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    const std::pair<int, int> key(dev * 16 + cs, smem_bytes);
    std::lock_guard<std::mutex> lock(mu);
    auto it = memo.find(key);
    if (it != memo.end()) return it->second;
    int n = 0;
    if (cudaFuncSetAttribute(conv_splitk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SK_SMEM_MAX) == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.gridDim = dim3((unsigned)(num_sms() / cs * cs));
        cfg.blockDim = dim3(SK_THREADS);
        cfg.dynamicSmemBytes = (size_t)smem_bytes;
        cfg.attrs = attr; cfg.numAttrs = 1;
        if (cudaOccupancyMaxActiveClusters(&n, conv_splitk_kernel, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    }
    memo[key] = n;
    return n;
}

int conv_splitk_launch(const ConvParams& p, cudaStream_t stream) {
    SkPlan pl;
    if (!conv_splitk_supports(p) || !splitk_plan(p, &pl)) return DR_ERR_UNSUPPORTED;
    SkJobs jobs{};
    const int st = fill_job(p, pl, p.sk_scratch, p.sk_counters, &jobs.j[0]);
    if (st != DR_OK) return st;
    jobs.n = 1;
    // as many stages as the slice has k-blocks, up to 200 KB: short slices leave room for a CTA of the next layer
    // beside one of this layer on the same SM (at most 256 TMEM columns each)
    return launch_jobs(jobs, jobs.j[0].ctas, pl.stages * pl.sub_bytes + 1024, stream);
}

int conv_splitk_group_launch(const ConvParams& a, const ConvParams& b, const ConvParams* c, cudaStream_t stream) {
    SkPlan pa, pb, pc{};
    if (!conv_splitk_group_supports(a, b, c) || !splitk_group_plan(a, b, c, &pa, &pb, &pc)) return DR_ERR_UNSUPPORTED;
    SkJobs jobs{};
    int st = fill_job(a, pa, a.sk_scratch, a.sk_counters, &jobs.j[0]);
    if (st != DR_OK) return st;
    char* scratch = reinterpret_cast<char*>(a.sk_scratch) + pa.scratch_bytes;
    int* counters = a.sk_counters + a.m_tiles * pa.n_blocks;
    st = fill_job(b, pb, reinterpret_cast<float*>(scratch), counters, &jobs.j[1]);
    if (st != DR_OK) return st;
    const int cs = (c && pb.cluster && pc.cluster) ? pb.splits : 1;
    int small = jobs.j[1].ctas;
    jobs.n = 2;
    jobs.cs = cs;
    if (c) {
        scratch += pb.scratch_bytes;
        counters += b.m_tiles * pb.n_blocks;
        st = fill_job(*c, pc, reinterpret_cast<float*>(scratch), counters, &jobs.j[2]);
        if (st != DR_OK) return st;
        jobs.dep = counters + c->m_tiles * pc.n_blocks;
        if (jobs.j[2].ctas > small) small = jobs.j[2].ctas;
        jobs.n = 3;
    }
    jobs.small_begin = (jobs.j[0].ctas + cs - 1) / cs * cs;              // the small group starts a cluster
    jobs.c_begin = jobs.small_begin;
    if (c && pc.own_ctas) {
        jobs.c_begin = jobs.small_begin + jobs.j[1].ctas;                // a multiple of the cluster size
        small = jobs.j[1].ctas + jobs.j[2].ctas;
    }
    return launch_jobs(jobs, jobs.small_begin + small, group_smem_bytes(pa, pb, c ? &pc : nullptr), stream);
}

}  // namespace dr
