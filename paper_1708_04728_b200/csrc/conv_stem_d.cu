// The 7x7 / stride-2 / 3-channel stem with fused ReLU -> 3x3/2 max-pool [-> LRN]: "operands in place".
//
// No im2col tile is ever built.  An input row lives in shared memory as 16-byte slots, one slot per
// PAIR of pixels: [p0c0 p0c1 p0c2 p1c0 p1c1 p1c2 0 0], slot sigma = pair + 2 (two zero slots in front
// and one behind are the horizontal padding).  The seven taps of output column wo in filter row r
// cover pixels 2wo-3 .. 2wo+3, which is inside pairs wo-2 .. wo+1 = slots wo .. wo+3: a 64-byte window
// that starts 16 bytes after the window of column wo-1.  In the tensor core's K-major no-swizzle
// operand layout a matrix row is 16 bytes per 8-element K chunk, rows 16 bytes apart inside an 8-row
// group, groups SBO apart, K chunks LBO apart.  With SBO = 128 and LBO = 16 the operand "row n,
// K chunk j" is simply slot n + j of the row buffer: the overlapping windows are described to the
// MMA in place, and the copy of the input that shared memory holds is the only one.
//
// The GEMM is transposed (D[channel][column]): A = filters, B = image row.  M = 128 stacks two output
// rows of a pair (2i, 2i+1): A rows 0-63 hold the filters against K blocks 0..6 (input rows 4i-3 ..
// 4i+3), A rows 64-127 hold the same filters against K blocks 2..8 (input rows 4i-1 .. 4i+5); K = 9
// blocks x 32.  One tile = one pair of output rows of one image = 18 MMAs of 128 x 128 x 16.
//
// In tensor memory a lane is a channel of one of the two rows and a column is wo, so the horizontal
// 3-window max is register arithmetic on the columns a thread loads.  The vertical max needs rows
// 2i-1, 2i, 2i+1: the row-(2i+1) threads keep their previous tile's result as a register carry, fold
// it in and pass the partial max through shared memory to the row-2i threads, which finish the pool,
// add bias, clamp, and transpose through shared memory for the cross-channel LRN and the NHWC store.
//
// Work split: all row pairs of the batch, in (image, pair) order, are cut into one contiguous range
// per stream; two independent streams per CTA.  A stream is a pipeline of one loader warp (a 24-row
// ring of input rows filled by cp.async three tiles ahead), one MMA warp (two accumulators), four
// pooling warps (tensor memory -> pooled, biased, clamped values in the transpose buffer) and four
// LRN/store warps that drain the transpose buffer half a row at a time.  A range that starts inside
// an image first computes the pair above it for the carry only.  Registers are re-split at kernel
// start: the pooling warps hold a row of maxima each and take 144, the others give theirs up.
#include <cstdlib>

#include "conv_common.cuh"
#include "conv_fused_epilogue.cuh"
#include "umma_ptx.cuh"

namespace dr {
using namespace ptx;

constexpr int SD_THREADS = 640;          // warps 0-3 / 4-7: pooling of stream 0 / 1; 8-11 / 12-15: LRN + store; 16, 17: MMA; 18, 19: loaders
constexpr int SD_REGS_POOL = 144, SD_REGS_LRN = 64, SD_REGS_AUX = 64;     // per thread after the re-split
static_assert(256 * SD_REGS_POOL + 256 * SD_REGS_LRN + 128 * SD_REGS_AUX <= SD_THREADS * 96, "register split exceeds the launch allocation");
constexpr int SD_NQ = 6;                 // ring depth in quads (4 input rows = what one tile adds)
constexpr int SD_NR = 4 * SD_NQ;         // ring rows
constexpr int SD_WT_BYTES = 36 * 2048;   // filters: 36 K chunks x 128 rows x 16 B
constexpr int SD_LB_PITCH = 76;          // floats per pooled pixel in the transpose buffer: 4 halo + 64 + 4 halo + 4 (bank spread)
constexpr int SD_SMEM_MAX = 227 * 1024 - 512;     // dynamic part; the static part holds the barriers

struct SdShared {
    uint64_t qfull[2][SD_NQ], qempty[2][SD_NQ], tfull[2][2], tempty[2][2];
    uint64_t lfull[2][2], lempty[2][2];      // halves of the transpose buffer: pooling warps -> LRN warps and back
    uint32_t tmem_base;
    int abort;
};

struct SdGeom {
    int pitch;        // bytes of one ring row: (W/2 + 4) slots
    int NP;           // row pairs per image
    int sa_pitch;     // floats per channel in the partial-max buffer
    long long total;  // row pairs in the batch
};

// K-major, no swizzle: start address, leading (K chunk) and stride (8-row group) offsets in bytes
__device__ __forceinline__ uint64_t sd_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | ((uint64_t)1 << 46);
}

__device__ __forceinline__ void sd_cp_async4(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 4 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}

// tcgen05.wait::ld that also names the destination registers, so no use of them is scheduled above it
__device__ __forceinline__ void sd_ld_wait(uint32_t* r) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]),
                   "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]),
                   "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]),
                   "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :
                 : "memory");
}

__device__ __forceinline__ bool sd_bar_and(int id, bool ok) {     // AND over the 128 threads of an epilogue group
    uint32_t out;
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.u32 p, %1, 0;\n"
        "bar.red.and.pred q, %2, 128, p;\n"
        "selp.u32 %0, 1, 0, q;\n"
        "}\n"
        : "=r"(out)
        : "r"((uint32_t)ok), "r"(id)
        : "memory");
    return out != 0;
}

__device__ __forceinline__ float sd_max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// The stream's range of row pairs, one image segment at a time.
struct SdSegments {
    long long cur, end;
    int NP;
    __device__ SdSegments(long long total, int streams, int s, int np) : NP(np) {
        cur = total * s / streams;
        end = total * (s + 1) / streams;
    }
    // n: image; j0: first pair computed (the carry-only pair when halo); T: tiles
    __device__ bool next(int& n, int& j0, int& T, bool& halo) {
        if (cur >= end) return false;
        n = (int)(cur / NP);
        const int is = (int)(cur - (long long)n * NP);
        const long long img_end = (long long)(n + 1) * NP;
        const long long e = end < img_end ? end : img_end;
        halo = is > 0;
        j0 = is - (halo ? 1 : 0);
        T = (int)(e - cur) + (halo ? 1 : 0);
        cur = e;
        return true;
    }
};

// Horizontal 3-window max (columns 2pw-1, 2pw, 2pw+1) of one accumulator row; emit(pw, value) for pw = 0..63,
// in order, with compile-time pw.  Columns at or beyond Wo count as -inf.
template <class Emit>
__device__ __forceinline__ void sd_hpool(uint32_t taddr, int Wo, Emit emit) {
    const float NEG = __uint_as_float(0xff800000u);
    float prev = NEG;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        if (32 * k < Wo) {
            uint32_t x[32];
            tmem_ld_x32(taddr + 32 * k, x);
            sd_ld_wait(x);
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(x[j]);
            if (32 * k + 32 > Wo) {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (32 * k + j >= Wo) v[j] = NEG;
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float a = j == 0 ? prev : v[2 * j - 1];
                emit(16 * k + j, sd_max3(a, v[2 * j], v[2 * j + 1]));
            }
            prev = v[31];
        }
    }
}

// Layer fixed to k = 7, stride 2, pad 3, Cin = 3, Cout = 64, pool 3x3/2 pad 1 after the ReLU (host checks).
// WO: the output width when it is known at compile time (the width guards fold away), 0 for any width.
template <int WO>
__global__ void __launch_bounds__(SD_THREADS, 1) conv_stem_d_kernel(const ConvParams p, const SdGeom gm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ SdShared sh;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ring_bytes = SD_NR * gm.pitch + 256;                        // + the run-over of junk columns past the last row
    const int sa_bytes = 64 * gm.sa_pitch * 4;
    const int lb_bytes = 4 * (WO ? (WO + 1) / 2 : p.Wy) * SD_LB_PITCH;
    uint8_t* Wt = smem;
    uint8_t* ring0 = Wt + SD_WT_BYTES;
    uint8_t* sa0 = ring0 + 2 * ring_bytes;
    uint8_t* lb0 = sa0 + 2 * sa_bytes;
    const int total_bytes = SD_WT_BYTES + 2 * ring_bytes + 2 * sa_bytes + 2 * lb_bytes;

    if (tid == 0) {
        for (int g = 0; g < 2; ++g) {
            for (int q = 0; q < SD_NQ; ++q) { mbar_init(&sh.qfull[g][q], 32); mbar_init(&sh.qempty[g][q], 1); }
            for (int b = 0; b < 2; ++b) {
                mbar_init(&sh.tfull[g][b], 1); mbar_init(&sh.tempty[g][b], 4);
                mbar_init(&sh.lfull[g][b], 64); mbar_init(&sh.lempty[g][b], 4);
            }
        }
        sh.abort = 0;
        fence_barrier_init();
    }
    if (warp == 16) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
    // everything starts at zero: padding slots, the two spare elements of every slot, unused filter slots, LRN halos
    for (int i = tid; i < total_bytes / 16; i += SD_THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    grid_launch_dependents();            // the layer behind this one may set up on free SMs (it waits for this kernel before it reads)
    // filters.  K = block*32 + j*8 + e: slot j of the window, element e = pixel-in-pair*3 + channel; tap s = 2j + pixel - 1
    for (int i = tid; i < 64 * 147; i += SD_THREADS) {
        const int c = i / 147, e0 = i - c * 147;
        const int r = e0 / 21, sc = e0 - r * 21;
        const int s = sc / 3, ch = sc - s * 3;
        const int j = (s + 1) >> 1, pe = (s + 1) & 1;
        const unsigned short val = reinterpret_cast<const unsigned short*>(p.w)[i];
        const int el = pe * 3 + ch;
        // row c against block r; row 64 + c against block r + 2
        *reinterpret_cast<unsigned short*>(Wt + (4 * r + j) * 2048 + c * 16 + el * 2) = val;
        *reinterpret_cast<unsigned short*>(Wt + (4 * (r + 2) + j) * 2048 + (64 + c) * 16 + el * 2) = val;
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort;
    const int streams = 2 * gridDim.x;

    if (warp >= 18) {
        // ------------------------------------------------------------- loader of stream g
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(SD_REGS_AUX));
        const int g = warp - 18;
        SdSegments seg(gm.total, streams, 2 * blockIdx.x + g, gm.NP);
        const uint32_t ring = smem_u32(ring0 + g * ring_bytes);
        const int pairs = p.W >> 1;
        const size_t row_elems = (size_t)p.W * 3;
        long long Ql = 0;
        bool dead = false;
        int n, j0, T;
        bool halo;
        while (!dead && seg.next(n, j0, T, halo)) {
            const int y_first = 4 * j0 - 3;
            const unsigned short* ximg = reinterpret_cast<const unsigned short*>(p.x) + (size_t)n * p.H * row_elems;
            for (int q = 0; q < T + 2; ++q, ++Ql) {
                const int slot = (int)(Ql % SD_NQ);
                const uint32_t use = (uint32_t)(Ql / SD_NQ);
                const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.qempty[g][slot], (use & 1) ^ 1, abort_flag));
                if (!ok) {
                    if (!*abort_flag) report_timeout(p.status, 61, (int)Ql);
                    *abort_flag = 1;
                    dead = true;
                    break;
                }
#pragma unroll
                for (int rr = 0; rr < 4; ++rr) {
                    const int y = y_first + 4 * q + rr;
                    const bool yin = y >= 0 && y < p.H;
                    const unsigned short* xrow = ximg + (yin ? (size_t)y * row_elems : 0);
                    const uint32_t drow = ring + (uint32_t)(slot * 4 + rr) * gm.pitch + 32u;
                    for (int pr = lane; pr < pairs; pr += 32) {
                        const unsigned short* src = xrow + (yin ? pr * 6 : 0);
                        const uint32_t dst = drow + 16u * pr;
                        sd_cp_async4(dst, src, yin);
                        sd_cp_async4(dst + 4, src + 2, yin);
                        sd_cp_async4(dst + 8, src + 4, yin);
                    }
                }
                // this lane's arrival on the quad's barrier fires when its copies above have landed
                asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&sh.qfull[g][slot])) : "memory");
            }
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    } else if (warp >= 16) {
        // ------------------------------------------------------------- MMA issue of stream g
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(SD_REGS_AUX));
        const int g = warp - 16;
        {
            // The whole warp walks the loop (every value below is warp-uniform) and lane 0 alone issues the MMAs and the
            // commits: a lone lane inside a divergent branch issues one MMA per 120-210 cycles, a converged warp with a
            // predicated MMA one per 64, which is what the 18 MMAs of a tile need.
            const uint32_t el = lane == 0 ? 1u : 0u;
            SdSegments seg(gm.total, streams, 2 * blockIdx.x + g, gm.NP);
            const uint32_t ring = smem_u32(ring0 + g * ring_bytes);
            const uint32_t wt = smem_u32(Wt);
            const uint32_t idesc = make_idesc_bf16(128, 128);
            const uint64_t a0 = sd_desc(wt, 2048u, 128u);                  // filters: K chunk (2r + h) is 4096 bytes = 256 descriptor units further
            const uint64_t bhi = sd_desc(0u, 16u, 128u);                   // image row: everything but the start address
            long long Qb = 0, qready = 0;
            uint32_t tcount = 0;
            bool dead = false;
            int n, j0, T;
            bool halo;
            while (!dead && seg.next(n, j0, T, halo)) {
                for (int t = 0; t < T; ++t, ++tcount) {
                    bool ok = true;
                    while (ok && qready <= Qb + t + 2) {
                        ok = __all_sync(0xffffffffu, mbar_wait(&sh.qfull[g][(int)(qready % SD_NQ)], (uint32_t)(qready / SD_NQ) & 1, abort_flag));
                        ++qready;
                    }
                    const uint32_t buf = tcount & 1;
                    ok = ok && __all_sync(0xffffffffu, mbar_wait(&sh.tempty[g][buf], ((tcount >> 1) & 1) ^ 1, abort_flag));
                    if (!ok) {
                        if (el && !*abort_flag) report_timeout(p.status, 62, (int)tcount);
                        *abort_flag = 1;
                        dead = true;
                        break;
                    }
                    tc_fence_after();
                    fence_proxy_async_smem();                              // the loader's copies, seen through the barrier, before the MMA reads them
                    const uint32_t d = tmem + (uint32_t)(g * 256) + buf * 128u;
                    const int row0 = (int)((4 * (Qb + t)) % SD_NR);
#pragma unroll
                    for (int r = 0; r < 9; ++r) {
                        int R = row0 + r;
                        if (R >= SD_NR) R -= SD_NR;
                        const uint32_t brow = ring + (uint32_t)R * gm.pitch;
                        const uint64_t b0 = bhi | (uint64_t)((brow & 0x3FFFFu) >> 4);
#pragma unroll
                        for (int h = 0; h < 2; ++h)
                            umma_bf16_pred(d, a0 + (uint64_t)((2 * r + h) * 256), b0 + (uint64_t)(2 * h), idesc, (r | h) != 0, el);
                    }
                    if (el) {
                        umma_commit(&sh.tfull[g][buf]);
                        umma_commit(&sh.qempty[g][(int)((Qb + t) % SD_NQ)]);
                    }
                    __syncwarp();
                }
                if (!dead && el) {
                    umma_commit(&sh.qempty[g][(int)((Qb + T) % SD_NQ)]);
                    umma_commit(&sh.qempty[g][(int)((Qb + T + 1) % SD_NQ)]);
                }
                __syncwarp();
                Qb += T + 2;
            }
        }
        __syncwarp();
    } else if (warp >= 8) {
        // ------------------------------------------------------------- LRN + store of stream g
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(SD_REGS_LRN));
        const int g = (warp - 8) >> 2;
        const int L = ((warp - 8) & 3) * 32 + lane;
        const int Wy = WO ? (WO + 1) / 2 : p.Wy;
        const int hs = ((Wy + 1) / 2 + 3) & ~3;                            // columns in the first half of the transpose buffer
        const float* lb = reinterpret_cast<const float*>(lb0 + g * lb_bytes);
        const bool lrn = p.flags & DR_LRN;
        __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(p.y);
        SdSegments seg(gm.total, streams, 2 * blockIdx.x + g, gm.NP);
        uint32_t lc = 0;                                                   // output tiles so far
        bool dead = false;
        int n, j0, T;
        bool halo;
        while (!dead && seg.next(n, j0, T, halo)) {
            for (int t = halo ? 1 : 0; t < T && !dead; ++t, ++lc) {
                const long long qrow = ((long long)n * p.Hy + (j0 + t)) * Wy;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.lfull[g][h], lc & 1, abort_flag));
                    if (!ok) {
                        if (!*abort_flag) report_timeout(p.status, 64, (int)lc);
                        *abort_flag = 1;
                        dead = true;
                        break;
                    }
                    const int pw0 = h ? hs : 0;
                    const int items = ((h ? Wy : hs) - pw0) * 8;           // item = (pooled column, group of 8 channels)
                    for (int it = L; (it & ~31) < items; it += 128) {      // whole warps leave together (warp votes inside)
                        const bool active = it < items;
                        const int pw = pw0 + (active ? it >> 3 : 0), c8 = it & 7;
                        const float4* s4 = reinterpret_cast<const float4*>(lb + pw * SD_LB_PITCH + (c8 << 3));   // x[c-4 .. c+11]
                        float w16[16];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float4 f = s4[j];
                            w16[4 * j] = f.x; w16[4 * j + 1] = f.y; w16[4 * j + 2] = f.z; w16[4 * j + 3] = f.w;
                        }
                        uint4 u;
                        if (lrn) {
                            float v[12], sq[12], ss[8], sc[8];
#pragma unroll
                            for (int j = 0; j < 12; ++j) { v[j] = w16[j + 2]; sq[j] = v[j] * v[j]; }          // v[0] = x[c-2]
#pragma unroll
                            for (int j = 0; j < 8; ++j) ss[j] = (sq[j] + sq[j + 1]) + (sq[j + 2] + sq[j + 3]) + sq[j + 4];
                            fe_lrn_scale<8>(p, ss, sc);
                            u.x = pack_bf16(v[2] * sc[0], v[3] * sc[1]); u.y = pack_bf16(v[4] * sc[2], v[5] * sc[3]);
                            u.z = pack_bf16(v[6] * sc[4], v[7] * sc[5]); u.w = pack_bf16(v[8] * sc[6], v[9] * sc[7]);
                        } else {
                            u.x = pack_bf16(w16[4], w16[5]); u.y = pack_bf16(w16[6], w16[7]);
                            u.z = pack_bf16(w16[8], w16[9]); u.w = pack_bf16(w16[10], w16[11]);
                        }
                        if (active) *reinterpret_cast<uint4*>(y + (qrow + pw) * p.ldc + p.coff + (c8 << 3)) = u;
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.lempty[g][h]);
                }
            }
        }
    } else {
        // ------------------------------------------------------------- pooling of stream g
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(SD_REGS_POOL));
        const int g = warp >> 2, q = warp & 3;
        const int L = q * 32 + lane, c = L & 63;
        const bool phb = L >= 64;                                         // this thread's lane is a channel of row 2i+1
        const int Wo = WO ? WO : p.Wo, Wy = WO ? (WO + 1) / 2 : p.Wy, sp = gm.sa_pitch;
        const int hs = ((Wy + 1) / 2 + 3) & ~3;
        float* sa = reinterpret_cast<float*>(sa0 + g * sa_bytes) + c * sp;   // this channel's partial maxima
        float* lb = reinterpret_cast<float*>(lb0 + g * lb_bytes);           // [pw][4 | 64 | 4 (+4)]
        const float bias = (p.flags & DR_BIAS) ? p.bias[c] : 0.f;
        const bool relu = p.flags & DR_RELU;
        const float NEG = __uint_as_float(0xff800000u);
        const int bar0 = 1 + 3 * g;
        SdSegments seg(gm.total, streams, 2 * blockIdx.x + g, gm.NP);
        uint32_t tcount = 0, lc = 0;
        bool dead = false, fail = false;
        int n, j0, T;
        bool halo;
        float keep[64];                       // row 2i threads: this tile's horizontal maxima; row 2i+1 threads: the carry
        while (!dead && seg.next(n, j0, T, halo)) {
#pragma unroll
            for (int j = 0; j < 64; ++j) keep[j] = NEG;
            for (int t = 0; t < T; ++t, ++tcount) {
                const uint32_t buf = tcount & 1;
                bool ok = mbar_wait(&sh.tfull[g][buf], (tcount >> 1) & 1, abort_flag) && !fail;
                ok = sd_bar_and(bar0, ok);
                if (!ok) {
                    if (!*abort_flag) report_timeout(p.status, 63, (int)tcount);
                    *abort_flag = 1;
                    dead = true;
                    break;
                }
                tc_fence_after();
                const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g * 256) + buf * 128u;
                const int i = j0 + t;                                      // row pair = pooled row
                const bool carry_only = halo && t == 0;
                const bool b_valid = 2 * i + 1 < p.Ho;
                if (phb) {
                    // partial max with the row above, kept for the row-2i threads; the new carry is this row
                    float4 m4;
                    sd_hpool(taddr, Wo, [&](int pw, float v) {
                        if (!b_valid) v = NEG;
                        const float m = fmaxf(v, keep[pw]);
                        keep[pw] = v;
                        if ((pw & 3) == 0) m4.x = m;
                        else if ((pw & 3) == 1) m4.y = m;
                        else if ((pw & 3) == 2) m4.z = m;
                        else {
                            m4.w = m;
                            if (!carry_only && pw - 3 < Wy) *reinterpret_cast<float4*>(sa + pw - 3) = m4;
                        }
                    });
                } else if (!carry_only) {
                    sd_hpool(taddr, Wo, [&](int pw, float v) { keep[pw] = v; });
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.tempty[g][buf]);
                if (carry_only) continue;
                asm volatile("bar.sync %0, 128;" ::"r"(bar0 + 1) : "memory");
                if (!phb) {
#pragma unroll
                    for (int f = 0; f < 16; ++f) {
                        if (4 * f < Wy) {
                            const float4 m4 = *reinterpret_cast<const float4*>(sa + 4 * f);
                            keep[4 * f] = fmaxf(keep[4 * f], m4.x); keep[4 * f + 1] = fmaxf(keep[4 * f + 1], m4.y);
                            keep[4 * f + 2] = fmaxf(keep[4 * f + 2], m4.z); keep[4 * f + 3] = fmaxf(keep[4 * f + 3], m4.w);
                        }
                    }
                }
                asm volatile("bar.sync %0, 128;" ::"r"(bar0 + 2) : "memory");   // the partial maxima may be overwritten
                if (!phb) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (!mbar_wait(&sh.lempty[g][h], (lc & 1) ^ 1, abort_flag)) fail = true;   // reported at the next tile's vote
#pragma unroll
                        for (int f = 0; f < 16; ++f) {
                            if (4 * f < Wy && (4 * f >= hs) == (h == 1)) {
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    float v = keep[4 * f + e] + bias;
                                    if (relu) v = fmaxf(v, 0.f);
                                    if (4 * f + e < Wy) lb[(4 * f + e) * SD_LB_PITCH + 4 + c] = v;
                                }
                            }
                        }
                        mbar_arrive(&sh.lfull[g][h]);
                    }
                }
                ++lc;
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
    if (warp == 16) tmem_dealloc(tmem, 512);
}

// ---- host --------------------------------------------------------------------------------
static SdGeom sd_geom(const ConvParams& p) {
    SdGeom g;
    g.pitch = (p.W / 2 + 4) * 16;
    g.NP = (p.Ho + 1) / 2;
    int sp = (p.Wy + 3) / 4;          // float4s per channel; odd, so a quarter warp's float4 accesses spread over all banks
    if (!(sp & 1)) ++sp;
    g.sa_pitch = 4 * sp;
    g.total = (long long)p.B * g.NP;
    return g;
}
static int sd_smem_bytes(const ConvParams& p, const SdGeom& g) {
    return SD_WT_BYTES + 2 * (SD_NR * g.pitch + 256) + 2 * 64 * g.sa_pitch * 4 + 2 * 4 * p.Wy * SD_LB_PITCH;
}

bool conv_stem_d_supports(const ConvParams& p) {
    if (!p.patch || !fe_supports(p) || fe_lrn_first(p)) return false;
    if (p.argmax) return false;                                      // positions of the maxima: the im2col-building stem kernel returns them
    if (p.k != 7 || p.stride != 2 || p.pad != 3 || p.Cin != 3 || p.Cout != 64 || (p.W & 1)) return false;
    if (p.Wo > 124) return false;                                   // one output row per 128-column MMA
    return sd_smem_bytes(p, sd_geom(p)) + 1024 <= SD_SMEM_MAX;
}

int conv_stem_d_launch(const ConvParams& p, cudaStream_t stream) {
    if (!conv_stem_d_supports(p)) return DR_ERR_UNSUPPORTED;
    static PerDeviceFlag attr_set;
    if (!attr_set.get()) {
        if (cudaFuncSetAttribute(conv_stem_d_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SD_SMEM_MAX) != cudaSuccess) return DR_ERR_CUDA;
        if (cudaFuncSetAttribute(conv_stem_d_kernel<112>, cudaFuncAttributeMaxDynamicSharedMemorySize, SD_SMEM_MAX) != cudaSuccess) return DR_ERR_CUDA;
        attr_set.set();
    }
    const SdGeom g = sd_geom(p);
    if (g.total <= 0) return DR_OK;
    int smem_bytes = sd_smem_bytes(p, g) + 1024;
    if (smem_bytes < 120 * 1024) smem_bytes = 120 * 1024;              // one CTA per SM: each CTA takes all of tensor memory
    const long long want = (g.total + 1) / 2;
    const int grid = want < num_sms() ? (int)want : num_sms();
    if (p.Wo == 112) conv_stem_d_kernel<112><<<grid, SD_THREADS, smem_bytes, stream>>>(p, g);
    else conv_stem_d_kernel<0><<<grid, SD_THREADS, smem_bytes, stream>>>(p, g);
    count_launch();
    return launch_status();
}

}  // namespace dr
