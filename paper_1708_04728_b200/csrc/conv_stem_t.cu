// The 7x7 / stride-2 / 3-channel stem with fused ReLU -> 3x3/2 max-pool [-> LRN], "channels on lanes".
//
// The GEMM is computed transposed, D[c][pixel] = sum_k W[c][k] * X[pixel][k]: the A operand is the
// (resident) filter matrix, 64 real rows padded to the MMA's M = 128, and the B operand is the im2col
// tile of a (2*PH+1) x 15 patch of convolution outputs (PH <= 5) stored with a row pitch of 16, N = 176.  In tensor memory a
// lane is then an output CHANNEL and a column is a PIXEL of the patch, so an epilogue thread owns
// one channel of the whole patch: the 3x3/2 max is plain register arithmetic on columns it loads
// itself (no shared-memory staging, no barriers), and the LRN window runs across neighbouring lanes
// with warp shuffles; only the two channels on either side of the lane-31/32 boundary cross between
// the two warps of a group, through a few hundred bytes of shared memory.
//
// Producers (six warps, thread = patch pixel) build the im2col tile exactly as conv_stem_kernel does:
// the input patch arrives by 4-byte cp.async one tile ahead, K is laid out as 7 tap-rows x 24 slots so
// that every tap-row is a 48-byte run (see conv_patch.cu).
#include <cstdlib>

#include "conv_common.cuh"
#include "conv_fused_epilogue.cuh"
#include "umma_ptx.cuh"

namespace dr {
using namespace ptx;

constexpr int ST_PW = 7, ST_PWC = 2 * ST_PW + 1;      // pooled / conv patch width (compile time: register indexing)
constexpr int ST_PITCH = 16;                           // GEMM columns per patch row: TMEM loads of a row start 16-aligned
constexpr int ST_MAX_PH = 5;
constexpr int ST_N = (2 * ST_MAX_PH + 1) * ST_PITCH;   // MMA N = 176 GEMM columns (11 x 15 = 165 real pixels)
constexpr int ST_THREADS = 512;                        // warps 0-5 producers, 6 MMA, 8-11 and 12-15: two epilogue groups
constexpr int ST_W_SUB = 128 * 128;                    // bytes of one K sub-tile of the filter operand (128 rows)
constexpr int ST_X_SUB = ST_N * 128;                   // ... of the im2col operand (176 rows)
constexpr int ST_W_BYTES = 3 * ST_W_SUB;               // 48 KB
constexpr int ST_X_BYTES = 3 * ST_X_SUB;               // 66 KB per buffer
constexpr int ST_SMEM_MAX = 227 * 1024 - 4096;          // dynamic part (the static part holds barriers, bias, LRN edge exchange)

struct StemTShared {
    uint64_t xfull[2], xempty[2], tfull[2], tempty[2];
    uint32_t tmem_base;
    int abort;
    float bias[64];
    float edge[2][2][2][ST_MAX_PH * ST_PW][2];         // [group][tile parity][warp half][pooled pixel][2 channels]
};

__device__ __forceinline__ uint32_t st_swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ void st_cp_async4(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 4 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}

__global__ void __launch_bounds__(ST_THREADS, 1) conv_stem_t_kernel(const ConvParams p, const int in_rows, const int in_words) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ StemTShared sh;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* Wt = smem;                                   // [3][128 rows][128 B]   filters (A operand)
    uint8_t* Xt = Wt + ST_W_BYTES;                        // 2 x [3][176 rows][128 B] im2col (B operand)
    uint32_t* inp = reinterpret_cast<uint32_t*>(Xt + 2 * ST_X_BYTES);   // 2 x [in_rows][in_words] input patches
    const int patch_words = in_rows * in_words;

    if (tid == 0) {
        for (int a = 0; a < 2; ++a) {
            mbar_init(&sh.xfull[a], 192); mbar_init(&sh.xempty[a], 1);
            mbar_init(&sh.tfull[a], 1); mbar_init(&sh.tempty[a], 4);
        }
        sh.abort = 0;
        fence_barrier_init();
    }
    if (warp == 6) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
    if (tid < 64) sh.bias[tid] = (p.flags & DR_BIAS) ? p.bias[tid] : 0.f;
    // operands start zeroed: rows 64..127 of the filter tile, the unused K slots and unused pixel rows
    // must stay finite (they meet zeros on the other side)
    for (int i = tid; i < (ST_W_BYTES + 2 * ST_X_BYTES) / 16; i += ST_THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (int i = tid; i < 64 * 147; i += ST_THREADS) {
        const int j = i / 147, e = i - j * 147;           // filter j, element (r, s, c) flattened
        const int r = e / 21, sc = e - r * 21;
        const int kp = r * 24 + sc;                       // K' index: 24 slots per tap-row
        const int sub = kp >> 6, within = kp & 63;
        const uint32_t off = (uint32_t)sub * ST_W_SUB + st_swz(j, within >> 3) + (within & 7) * 2;
        const unsigned short wv = reinterpret_cast<const unsigned short*>(p.w)[(size_t)j * 147 + e];
        *reinterpret_cast<unsigned short*>(Wt + off) = wv;
        // rows 64..127 repeat the filters: TMEM lanes 64..127 then hold the same channels again, which lets the
        // warps of lane quarters 2 and 3 share the epilogue of a tile with quarters 0 and 1
        const uint32_t off2 = (uint32_t)sub * ST_W_SUB + st_swz(j + 64, within >> 3) + (within & 7) * 2;
        *reinterpret_cast<unsigned short*>(Wt + off2) = wv;
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort;

    const int total = p.m_tiles;
    const int per = p.tiles_h * p.tiles_w;
    const int PH = p.PH, phc = 2 * PH + 1;

    if (warp < 6) {
        // ------------------------------------------------ producers: thread = patch pixel (GEMM column)
        const int pi = tid / ST_PITCH, pj = tid - pi * ST_PITCH;
        const bool row_used = pi < phc && pj < ST_PWC;
        constexpr int MAX_SLOTS = 10;                     // word slots of a patch per producer thread
        int slot_rr[MAX_SLOTS], slot_e[MAX_SLOTS];
#pragma unroll
        for (int k = 0; k < MAX_SLOTS; ++k) {
            const int i = tid + 192 * k;
            slot_rr[k] = i < patch_words ? i / in_words : -1;
            slot_e[k] = i < patch_words ? 2 * (i - (i / in_words) * in_words) : 0;
        }
        const int row_elems = 3 * p.W;
        auto load_patch = [&](int t, int b) {
            const int n = t / per, tt_ = t - n * per;
            const int th = tt_ / p.tiles_w, tw = tt_ - th * p.tiles_w;
            const int hi0 = 2 * (2 * th * PH - 1) - 3;                // first input row of the patch
            const int e0 = 3 * (2 * (2 * tw * ST_PW - 1) - 3 - 1);    // first element of a patch row: one pixel early, so even
            const unsigned short* ximg = reinterpret_cast<const unsigned short*>(p.x) + (size_t)n * p.H * p.W * 3;
            const uint32_t dst0 = smem_u32(inp + b * patch_words) + 4u * tid;
#pragma unroll
            for (int k = 0; k < MAX_SLOTS; ++k) {
                if (slot_rr[k] >= 0) {
                    const int hi = hi0 + slot_rr[k];
                    const int e = e0 + slot_e[k];
                    const bool ok = hi >= 0 && hi < p.H && e >= 0 && e + 1 < row_elems;
                    st_cp_async4(dst0 + 768u * k, ximg + (ok ? hi * row_elems + e : 0), ok);
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
            asm volatile("bar.sync 2, 192;" ::: "memory");             // ... and for the other producers
            bool ok = mbar_wait(&sh.xempty[b], (u & 1) ^ 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (!*abort_flag) report_timeout(p.status, 51, t);
                *abort_flag = 1;
                break;
            }
            if (row_used) {
                uint8_t* Xb = Xt + b * ST_X_BYTES;
                const uint32_t* src = inp + b * patch_words;
#pragma unroll
                for (int r = 0; r < 7; ++r) {
                    // tap-row r of this pixel: 24 elements from patch row 2*pi + r, element 6*pj + 3 (odd: realign by 16 bits)
                    const uint32_t* s32 = src + (2 * pi + r) * in_words + 3 * pj + 1;
                    uint32_t wv[13];
#pragma unroll
                    for (int k = 0; k < 13; ++k) wv[k] = s32[k];
                    uint32_t ov[12];
#pragma unroll
                    for (int k = 0; k < 12; ++k) ov[k] = __funnelshift_r(wv[k], wv[k + 1], 16);
#pragma unroll
                    for (int m = 0; m < 3; ++m) {
                        const int q = 3 * r + m;                       // 16-byte chunk index along K'
                        const uint32_t off = (uint32_t)(q >> 3) * ST_X_SUB + st_swz(tid, q & 7);
                        *reinterpret_cast<uint4*>(Xb + off) = make_uint4(ov[4 * m], ov[4 * m + 1], ov[4 * m + 2], ov[4 * m + 3]);
                    }
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(&sh.xfull[b]);
            asm volatile("bar.sync 2, 192;" ::: "memory");             // everyone is done reading this patch buffer
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else if (warp == 6) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(128, ST_N);
            const uint32_t w_lo = sdesc_lo(smem_u32(Wt));
            int it = 0;
            for (int t = blockIdx.x; t < total; t += gridDim.x, ++it) {
                const int b = it & 1, u = it >> 1;
                if (!mbar_wait(&sh.tempty[b], (u & 1) ^ 1, abort_flag) || !mbar_wait(&sh.xfull[b], u & 1, abort_flag)) {
                    if (!*abort_flag) report_timeout(p.status, 52, t);
                    *abort_flag = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d = tmem + (uint32_t)(b * 256);
                const uint32_t x_lo = sdesc_lo(smem_u32(Xt + b * ST_X_BYTES));
#pragma unroll
                for (int kk = 0; kk < 11; ++kk) {                      // K' = 176 of 192: the rest is zero weights
                    const uint32_t sub = kk >> 2, k4 = kk & 3;
                    umma_bf16_lo<false>(d, w_lo + sub * (ST_W_SUB >> 4) + 2 * k4, x_lo + sub * (ST_X_SUB >> 4) + 2 * k4, idesc, kk > 0, 1u);
                }
                umma_commit(&sh.xempty[b]);
                umma_commit(&sh.tfull[b]);
            }
        }
        __syncwarp();
    } else if (warp >= 8) {
        // ------------------------------------------------ epilogue: lane = channel, column = patch pixel.
        // A group is four warps (TMEM lane quarters 0-3): quarters q and q+2 hold the same 32 channels and
        // take alternate pooled rows of the tile.
        const int g = warp >= 12 ? 1 : 0;                              // warps 8-11 -> group 0; 12-15 -> group 1
        const int quarter = warp & 3;
        const int half = quarter & 1;                                  // channels 0-31 / 32-63
        const int rowset = quarter >> 1;                               // pooled rows of parity `rowset`
        const int c = half * 32 + lane;
        const bool lrn = p.flags & DR_LRN;
        const bool relu = p.flags & DR_RELU;
        const float bias_c = sh.bias[c];
        const float NEG_INF = __int_as_float(0xff800000);
        __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(p.y);
        int u = 0;
        for (int t = blockIdx.x + g * gridDim.x; t < total; t += 2 * gridDim.x, ++u) {
            const bool ok = __all_sync(0xffffffffu, mbar_wait(&sh.tfull[g], u & 1, abort_flag));
            if (!ok) {
                if (!*abort_flag) report_timeout(p.status, 54, t);
                *abort_flag = 1;
                break;
            }
            tc_fence_after();
            const int n = t / per, tt_ = t - n * per;
            const int th = tt_ / p.tiles_w, tw = tt_ - th * p.tiles_w;
            const int ho0 = 2 * th * PH - 1, wo0 = 2 * tw * ST_PW - 1;  // conv pixel of patch position (0,0)
            const bool col_edge = wo0 < 0 || wo0 + ST_PWC > p.Wo;       // some patch columns lie outside the conv plane
            const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(g * 256);
            float pooled[ST_MAX_PH][ST_PW];
#pragma unroll
            for (int ppi = 0; ppi < ST_MAX_PH; ++ppi) {
                if (ppi < PH && (ppi & 1) == rowset) {
                    // conv rows 2*ppi .. 2*ppi+2 of the patch: 48 consecutive columns starting at 32*ppi
                    uint32_t r[48];
                    const uint32_t col = (uint32_t)(2 * ppi * ST_PITCH);
                    tmem_ld_x32(taddr + col, r);
                    tmem_ld_x16(taddr + col + 32, r + 32);
                    tmem_ld_wait();
                    float v[48];
#pragma unroll
                    for (int k = 0; k < 48; ++k) v[k] = __uint_as_float(r[k]);
                    // rows / columns outside the conv plane never win
#pragma unroll
                    for (int dr_ = 0; dr_ < 3; ++dr_) {
                        const int ho = ho0 + 2 * ppi + dr_;
                        if (ho < 0 || ho >= p.Ho) {
#pragma unroll
                            for (int k = 0; k < ST_PWC; ++k) v[dr_ * ST_PITCH + k] = NEG_INF;
                        }
                    }
                    if (col_edge) {
#pragma unroll
                        for (int k = 0; k < ST_PWC; ++k) {
                            const int wo = wo0 + k;
                            if (wo < 0 || wo >= p.Wo) { v[k] = NEG_INF; v[ST_PITCH + k] = NEG_INF; v[2 * ST_PITCH + k] = NEG_INF; }
                        }
                    }
#pragma unroll
                    for (int ppj = 0; ppj < ST_PW; ++ppj) {
                        float m = v[2 * ppj];
#pragma unroll
                        for (int dd = 1; dd < 9; ++dd) m = fmaxf(m, v[(dd / 3) * ST_PITCH + 2 * ppj + (dd % 3)]);
                        m += bias_c;                                    // bias and ReLU commute with the max
                        pooled[ppi][ppj] = relu ? fmaxf(m, 0.f) : m;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.tempty[g]);                  // accumulator no longer needed

            if (lrn) {
                // channels c-2..c+2: neighbouring lanes; the lane 31|32 boundary crosses to the other warp via smem
                float (*mine)[2] = sh.edge[g][u & 1][half];
                if ((half == 0 && lane >= 30) || (half == 1 && lane < 2)) {
#pragma unroll
                    for (int ppi = 0; ppi < ST_MAX_PH; ++ppi)
#pragma unroll
                        for (int ppj = 0; ppj < ST_PW; ++ppj)
                            if (ppi < PH && (ppi & 1) == rowset) mine[ppi * ST_PW + ppj][lane & 1] = pooled[ppi][ppj];
                }
                asm volatile("bar.sync %0, 128;" ::"r"(4 + g) : "memory");
            }
#pragma unroll
            for (int ppi = 0; ppi < ST_MAX_PH; ++ppi) {
                if (ppi < PH && (ppi & 1) == rowset) {
                    const int ph = th * PH + ppi;
                    float out[ST_PW];
                    if (lrn) {
                        const float (*other)[2] = sh.edge[g][u & 1][half ^ 1];
                        float ss[ST_PW], sc[ST_PW];
#pragma unroll
                        for (int ppj = 0; ppj < ST_PW; ++ppj) {
                            const float x = pooled[ppi][ppj];
                            float m1 = __shfl_up_sync(0xffffffffu, x, 1), m2 = __shfl_up_sync(0xffffffffu, x, 2);
                            float p1 = __shfl_down_sync(0xffffffffu, x, 1), p2 = __shfl_down_sync(0xffffffffu, x, 2);
                            const float o0 = other[ppi * ST_PW + ppj][0], o1 = other[ppi * ST_PW + ppj][1];
                            if (half == 0) {            // channels 0..31: below channel 0 nothing; above lane 31 the other warp's 32, 33
                                if (lane < 1) m1 = 0.f;
                                if (lane < 2) m2 = 0.f;
                                if (lane == 31) { p1 = o0; p2 = o1; }
                                if (lane == 30) p2 = o0;
                            } else {                    // channels 32..63: below lane 0 the other warp's 30, 31; above channel 63 nothing
                                if (lane == 0) { m1 = o1; m2 = o0; }
                                if (lane == 1) m2 = o1;
                                if (lane > 30) p1 = 0.f;
                                if (lane > 29) p2 = 0.f;
                            }
                            ss[ppj] = (m2 * m2 + m1 * m1) + (x * x + p1 * p1) + p2 * p2;
                        }
                        fe_lrn_scale<ST_PW>(p, ss, sc);
#pragma unroll
                        for (int ppj = 0; ppj < ST_PW; ++ppj) out[ppj] = pooled[ppi][ppj] * sc[ppj];
                    } else {
#pragma unroll
                        for (int ppj = 0; ppj < ST_PW; ++ppj) out[ppj] = pooled[ppi][ppj];
                    }
                    if (ph < p.Hy) {
#pragma unroll
                        for (int ppj = 0; ppj < ST_PW; ++ppj) {
                            const int pw = tw * ST_PW + ppj;
                            if (pw < p.Wy) y[(((long long)n * p.Hy + ph) * p.Wy + pw) * p.ldc + p.coff + c] = __float2bfloat16_rn(out[ppj]);
                        }
                    }
                }
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
    if (warp == 6) tmem_dealloc(tmem, 512);
}

static void stem_t_geometry(const ConvParams& p, ConvParams* q, int* rows, int* words) {
    *q = p;
    q->PW = ST_PW;
    q->PH = p.Hy < ST_MAX_PH ? p.Hy : ST_MAX_PH;
    q->tiles_h = (p.Hy + q->PH - 1) / q->PH;
    q->tiles_w = (p.Wy + ST_PW - 1) / ST_PW;
    q->m_tiles = p.B * q->tiles_h * q->tiles_w;
    *rows = 2 * (2 * q->PH + 1) + 5;
    const int pixels = 2 * ST_PWC + 5 + 2;                 // + one early pixel (alignment) + one late (13th word)
    *words = (3 * pixels + 1) / 2 + 1;
}

bool conv_stem_t_supports(const ConvParams& p) {
    if (!(p.flags & DR_POOL) || p.argmax || !p.patch) return false;
    if ((p.flags & DR_LRN) && ((p.flags & DR_LRN_BEFORE_POOL) || p.lrn_half != 2 || p.lrn_k <= 0.f || p.lrn_alpha_n < 0.f)) return false;
    if (p.flags & (DR_RESIDUAL | DR_OUT_F32)) return false;
    if (p.k != 7 || p.stride != 2 || p.pad != 3 || p.Cin != 3 || p.Cout != 64 || (p.W & 1)) return false;
    if ((long long)p.B * ((p.Hy + ST_MAX_PH - 1) / ST_MAX_PH) * ((p.Wy + ST_PW - 1) / ST_PW) > 0x7fffffffLL) return false;
    ConvParams q;
    int rows, words;
    stem_t_geometry(p, &q, &rows, &words);
    if (rows * words > 10 * 192) return false;
    return ST_W_BYTES + 2 * ST_X_BYTES + 2 * rows * words * 4 + 2048 <= ST_SMEM_MAX;
}

int conv_stem_t_launch(const ConvParams& p, cudaStream_t stream) {
    if (!conv_stem_t_supports(p)) return DR_ERR_UNSUPPORTED;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(conv_stem_t_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ST_SMEM_MAX) != cudaSuccess) return DR_ERR_CUDA;
        attr_set = true;
    }
    ConvParams q;
    int rows, words;
    stem_t_geometry(p, &q, &rows, &words);
    if (q.m_tiles <= 0) return DR_OK;
    const int smem_bytes = ST_W_BYTES + 2 * ST_X_BYTES + 2 * rows * words * 4 + 1024;
    const int grid = q.m_tiles < num_sms() ? q.m_tiles : num_sms();
    conv_stem_t_kernel<<<grid, ST_THREADS, smem_bytes, stream>>>(q, rows, words);
    count_launch();
    return launch_status();
}

}  // namespace dr
