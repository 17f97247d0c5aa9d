// Stand-alone non-tensor layers (ReLU, max-pool, LRN, BatchNorm/Scale, add, concat, global
// average pool) and the offline parameter kernels (BN fold, filter embedding).
//
// These are the layers Section 2 of the paper calls "non-tensor": no weights, one pass over
// the activations each.  On this hardware they are bound by HBM bandwidth, so every kernel
// moves 128 bits per thread per access, coalesced along the channel axis of NHWC, with a grid
// sized to a few waves of the SMs.
#include <cmath>

#include "common.cuh"

namespace dr {

std::atomic<long long> g_launches{0};
__device__ int g_dev_status[4] = {0, 0, 0, 0};

int* dev_status_ptr() {
    static int* ptr[64] = {nullptr};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return nullptr;
    if (!ptr[dev] && cudaGetSymbolAddress((void**)&ptr[dev], g_dev_status) != cudaSuccess) ptr[dev] = nullptr;
    return ptr[dev];
}

static std::atomic<int> g_num_sms[64];
int num_sms() {
    int dev = 0;
    (void)cudaGetDevice(&dev);
    std::atomic<int>& slot = g_num_sms[dev & 63];
    int n = slot.load(std::memory_order_relaxed);
    if (!n) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { (void)cudaGetLastError(); n = 148; }
        slot.store(n, std::memory_order_relaxed);
    }
    return n;
}

static inline int grid_for(size_t work_items, int threads) {
    size_t blocks = (work_items + threads - 1) / threads;
    size_t cap = (size_t)num_sms() * 16;           // grid-stride beyond 16 blocks per SM
    if (blocks > cap) {
        // every thread the same number of items: a grid of `cap` blocks over 1.2 x cap blocks' worth of work would run a
        // second, mostly idle round
        const size_t iters = (blocks + cap - 1) / cap;
        blocks = (blocks + iters - 1) / iters;
    }
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

// ---------------------------------------------------------------- ReLU / add: 8 bf16 per thread
__global__ void relu_kernel(size_t n8, size_t n, const uint4* __restrict__ x, uint4* __restrict__ y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += stride) {
        uint4 v = __ldg(x + i);
        uint32_t* u = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
        for (int j = 0; j < 4; ++j) u[j] = pack_bf16(fmaxf(bf16_lo(u[j]), 0.f), fmaxf(bf16_hi(u[j]), 0.f));
        y[i] = v;
    }
    // tail (n not a multiple of 8), handled by the first threads
    const __nv_bfloat16* xs = reinterpret_cast<const __nv_bfloat16*>(x);
    __nv_bfloat16* ys = reinterpret_cast<__nv_bfloat16*>(y);
    for (size_t i = n8 * 8 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        ys[i] = __float2bfloat16_rn(fmaxf(__bfloat162float(xs[i]), 0.f));
}

__global__ void add_kernel(size_t n8, size_t n, const uint4* __restrict__ a, const uint4* __restrict__ b,
                           uint4* __restrict__ y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += stride) {
        uint4 va = __ldg(a + i), vb = __ldg(b + i), vo;
        const uint32_t* ua = reinterpret_cast<const uint32_t*>(&va);
        const uint32_t* ub = reinterpret_cast<const uint32_t*>(&vb);
        uint32_t* uo = reinterpret_cast<uint32_t*>(&vo);
#pragma unroll
        for (int j = 0; j < 4; ++j)
            uo[j] = pack_bf16(bf16_lo(ua[j]) + bf16_lo(ub[j]), bf16_hi(ua[j]) + bf16_hi(ub[j]));
        y[i] = vo;
    }
    const __nv_bfloat16* as = reinterpret_cast<const __nv_bfloat16*>(a);
    const __nv_bfloat16* bs = reinterpret_cast<const __nv_bfloat16*>(b);
    __nv_bfloat16* ys = reinterpret_cast<__nv_bfloat16*>(y);
    for (size_t i = n8 * 8 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        ys[i] = __float2bfloat16_rn(__bfloat162float(as[i]) + __bfloat162float(bs[i]));
}

// ---------------------------------------------------------------- BatchNorm (+ Scale)
// y = (x - mean/m) * g/sqrt(var/m+eps) + beta (g=1, beta=0 without Scale; mean == nullptr: Scale only).
// One thread per 8 consecutive channels of one pixel; C must be a multiple of 8 for the
// vector path, otherwise the scalar kernel runs.
__global__ void bn_kernel(size_t nvec, int C8, const uint4* __restrict__ x, const float* __restrict__ mean,
                          const float* __restrict__ var, float inv_m, float eps, const float* __restrict__ gamma,
                          const float* __restrict__ beta, uint4* __restrict__ y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    int c8 = (int)(i0 % C8);                              // the channel group advances by a fixed step: one division per thread
    const int step = (int)(stride % C8);
    for (size_t i = i0; i < nvec; i += stride, c8 = c8 + step >= C8 ? c8 + step - C8 : c8 + step) {
        const int c0 = c8 * 8;
        uint4 v = __ldg(x + i);
        uint32_t* u = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float r[2] = {bf16_lo(u[j]), bf16_hi(u[j])};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = c0 + 2 * j + h;
                const float a = (gamma ? __ldg(gamma + c) : 1.f) * (mean ? rsqrtf(__ldg(var + c) * inv_m + eps) : 1.f);
                r[h] = (r[h] - (mean ? __ldg(mean + c) * inv_m : 0.f)) * a + (gamma ? __ldg(beta + c) : 0.f);
            }
            u[j] = pack_bf16(r[0], r[1]);
        }
        y[i] = v;
    }
}
// The same with the per-channel constants folded to y = a x + b' (a = gamma / sqrt(var/m + eps), b' = beta - a mean/m)
// and computed once per block into shared memory (C <= 4096).  A thread's channel group advances by a fixed step from
// one vector to its next; when that step is zero (the grid stride is a multiple of the channel groups, the usual case)
// the sixteen constants stay in registers for the whole loop, otherwise they are four 16-byte shared loads per vector
// (read per vector, the three-constant form asked more of shared memory than the loads and stores of the data).
__global__ void bn_smem_kernel(size_t nvec, int C8, const uint4* __restrict__ x, const float* __restrict__ mean,
                               const float* __restrict__ var, float inv_m, float eps, const float* __restrict__ gamma,
                               const float* __restrict__ beta, uint4* __restrict__ y) {
    extern __shared__ float bn_s[];                       // [2][C]: a, b'
    const int C = C8 * 8;
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        const float a = (gamma ? __ldg(gamma + c) : 1.f) * (mean ? rsqrtf(__ldg(var + c) * inv_m + eps) : 1.f);
        bn_s[c] = a;
        bn_s[C + c] = (gamma ? __ldg(beta + c) : 0.f) - a * (mean ? __ldg(mean + c) * inv_m : 0.f);
    }
    __syncthreads();
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    int c8 = (int)(i0 % C8);
    const int step = (int)(stride % C8);
    float a[8], b[8];
    auto load_consts = [&](int c0) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            *reinterpret_cast<float4*>(a + 4 * h) = *reinterpret_cast<const float4*>(bn_s + c0 + 4 * h);
            *reinterpret_cast<float4*>(b + 4 * h) = *reinterpret_cast<const float4*>(bn_s + C + c0 + 4 * h);
        }
    };
    load_consts(c8 * 8);
    for (size_t i = i0; i < nvec; i += stride) {
        uint4 v = __ldg(x + i);
        uint32_t* u = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
        for (int j = 0; j < 4; ++j)
            u[j] = pack_bf16(fmaf(bf16_lo(u[j]), a[2 * j], b[2 * j]), fmaf(bf16_hi(u[j]), a[2 * j + 1], b[2 * j + 1]));
        y[i] = v;
        if (step) {
            c8 = c8 + step >= C8 ? c8 + step - C8 : c8 + step;
            load_consts(c8 * 8);
        }
    }
}
__global__ void bn_scalar_kernel(size_t n, int C, const __nv_bfloat16* __restrict__ x, const float* __restrict__ mean,
                                 const float* __restrict__ var, float inv_m, float eps,
                                 const float* __restrict__ gamma, const float* __restrict__ beta,
                                 __nv_bfloat16* __restrict__ y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const int c = (int)(i % C);
        const float a = (gamma ? gamma[c] : 1.f) * (mean ? rsqrtf(var[c] * inv_m + eps) : 1.f);
        y[i] = __float2bfloat16_rn((__bfloat162float(x[i]) - (mean ? mean[c] * inv_m : 0.f)) * a + (gamma ? beta[c] : 0.f));
    }
}

// ---------------------------------------------------------------- max-pool
// One thread per (output pixel, 8 channels).  First maximum in row-major window order wins.
__global__ void maxpool_kernel(int B, int H, int W, int C8, int Ho, int Wo, int k, int s, int p,
                               const uint4* __restrict__ x, uint4* __restrict__ y, int32_t* __restrict__ argmax) {
    // a kernel launched behind this one with programmatic serialization (the split-K convolution) may start its
    // prologue and filter prefetch now; it waits for this kernel's completion before it reads y
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const size_t total = (size_t)B * Ho * Wo * C8;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int c8 = (int)(i % C8);
        size_t q = i / C8;
        const int wo = (int)(q % Wo); q /= Wo;
        const int ho = (int)(q % Ho);
        const int n = (int)(q / Ho);
        float best[8];
        int where[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) { best[j] = 0.f; where[j] = -1; }
        for (int r = 0; r < k; ++r) {
            const int hi = ho * s - p + r;
            if (hi < 0 || hi >= H) continue;
            for (int t = 0; t < k; ++t) {
                const int wi = wo * s - p + t;
                if (wi < 0 || wi >= W) continue;
                const uint4 v = __ldg(x + (((size_t)n * H + hi) * W + wi) * C8 + c8);
                const uint32_t* u = reinterpret_cast<const uint32_t*>(&v);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float lo = bf16_lo(u[j]), hi2 = bf16_hi(u[j]);
                    if (where[2 * j] < 0 || lo > best[2 * j]) { best[2 * j] = lo; where[2 * j] = hi * W + wi; }
                    if (where[2 * j + 1] < 0 || hi2 > best[2 * j + 1]) { best[2 * j + 1] = hi2; where[2 * j + 1] = hi * W + wi; }
                }
            }
        }
        uint4 o;
        uint32_t* uo = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
        for (int j = 0; j < 4; ++j) uo[j] = pack_bf16(best[2 * j], best[2 * j + 1]);
        y[i] = o;
        if (argmax) {
            int4* a = reinterpret_cast<int4*>(argmax + i * 8);
            a[0] = make_int4(where[0], where[1], where[2], where[3]);
            a[1] = make_int4(where[4], where[5], where[6], where[7]);
        }
    }
}
// Without argmax the maximum is taken on packed bf16 pairs (4 instructions per tap and 8 channels).
__global__ void maxpool_noarg_kernel(int B, int H, int W, int C8, int Ho, int Wo, int k, int s, int p,
                                     const uint4* __restrict__ x, uint4* __restrict__ y) {
    const size_t total = (size_t)B * Ho * Wo * C8;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int c8 = (int)(i % C8);
        size_t q = i / C8;
        const int wo = (int)(q % Wo); q /= Wo;
        const int ho = (int)(q % Ho);
        const int n = (int)(q / Ho);
        uint4 m = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);   // -inf: padding never wins
        __nv_bfloat162* mm = reinterpret_cast<__nv_bfloat162*>(&m);
        for (int r = 0; r < k; ++r) {
            const int hi = ho * s - p + r;
            if (hi < 0 || hi >= H) continue;
            for (int t = 0; t < k; ++t) {
                const int wi = wo * s - p + t;
                if (wi < 0 || wi >= W) continue;
                const uint4 v = __ldg(x + (((size_t)n * H + hi) * W + wi) * C8 + c8);
                const __nv_bfloat162* vv = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
                for (int j = 0; j < 4; ++j) mm[j] = __hmax2(mm[j], vv[j]);
            }
        }
        y[i] = m;
    }
}
// The 3x3 window unrolled: the nine loads go out together (taps outside the plane load a clamped, valid address and
// are replaced by -inf afterwards), then the maxima.
__global__ void maxpool3_noarg_kernel(int B, int H, int W, int C8, int Ho, int Wo, int s, int p, const uint4* __restrict__ x,
                                      uint4* __restrict__ y) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // see maxpool_noarg_kernel
    const size_t total = (size_t)B * Ho * Wo * C8;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        // the index is split with 32-bit divisions where it fits (a 64-bit division costs several times the rest of the body)
        int c8, wo, ho;
        size_t n;
        if (total <= 0xffffffffull) {
            const unsigned iu = (unsigned)i, q1 = iu / (unsigned)C8, q2 = q1 / (unsigned)Wo, q3 = q2 / (unsigned)Ho;
            c8 = (int)(iu - q1 * (unsigned)C8); wo = (int)(q1 - q2 * (unsigned)Wo); ho = (int)(q2 - q3 * (unsigned)Ho); n = q3;
        } else {
            c8 = (int)(i % C8);
            size_t q = i / C8;
            wo = (int)(q % Wo); q /= Wo;
            ho = (int)(q % Ho);
            n = q / Ho;
        }
        const int h0 = ho * s - p, w0 = wo * s - p;
        uint4 v[9];
        bool ok[9];
#pragma unroll
        for (int r = 0; r < 3; ++r)
#pragma unroll
            for (int t = 0; t < 3; ++t) {
                const int hi = h0 + r, wi = w0 + t;
                ok[3 * r + t] = hi >= 0 && hi < H && wi >= 0 && wi < W;
                const int hc = min(max(hi, 0), H - 1), wc = min(max(wi, 0), W - 1);     // clamped: always a valid address
                v[3 * r + t] = __ldg(x + ((n * H + hc) * W + wc) * C8 + c8);
            }
        uint4 m = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);       // -inf: padding never wins
        __nv_bfloat162* mm = reinterpret_cast<__nv_bfloat162*>(&m);
#pragma unroll
        for (int d = 0; d < 9; ++d) {
            const uint4 u = ok[d] ? v[d] : make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
            const __nv_bfloat162* uu = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
            for (int j = 0; j < 4; ++j) mm[j] = __hmax2(mm[j], uu[j]);
        }
        y[i] = m;
    }
}
thread_local bool g_pool_pdl = false;
// An ordinary launch, or one with programmatic stream serialization when the network executor asks for it (the
// kernels that take this path execute griddepcontrol.wait before their first load).
template <class... KArgs, class... Args>
static void launch_maybe_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = 0; cfg.stream = stream;
    cfg.attrs = attr; cfg.numAttrs = g_pool_pdl ? 1 : 0;
    (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// 3x3 / stride 2: a thread takes a 2 x 2 block of pooled positions (8 channels), whose windows cover 5 x 5 inputs:
// 25 loads for four outputs instead of 36, all issued before the first maximum.  Taps outside the plane load a clamped,
// valid address and are replaced by -inf.
__global__ void __launch_bounds__(256) maxpool3s2_quad_kernel(int B, int H, int W, int C8, int Ho, int Wo, int p, const uint4* __restrict__ x,
                                                              uint4* __restrict__ y) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // see maxpool_kernel
    asm volatile("griddepcontrol.wait;" ::: "memory");                // no-op unless launched with programmatic serialization
    const unsigned Ho2 = (unsigned)(Ho + 1) >> 1, Wo2 = (unsigned)(Wo + 1) >> 1;
    const unsigned total = (unsigned)B * Ho2 * Wo2 * (unsigned)C8;     // the host keeps this below 2^32
    const unsigned stride = gridDim.x * blockDim.x;
    const uint4 NEG = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);   // -inf: padding never wins
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const unsigned q1 = i / (unsigned)C8, q2 = q1 / Wo2, n = q2 / Ho2;
        const int c8 = (int)(i - q1 * (unsigned)C8), wo = 2 * (int)(q1 - q2 * Wo2), ho = 2 * (int)(q2 - n * Ho2);
        const int h0 = 2 * ho - p, w0 = 2 * wo - p;
        const uint4* img = x + (size_t)n * H * W * C8 + c8;
        uint4 v[25];
#pragma unroll
        for (int r = 0; r < 5; ++r)
#pragma unroll
            for (int t = 0; t < 5; ++t) {
                const int hi = h0 + r, wi = w0 + t;
                const int hc = min(max(hi, 0), H - 1), wc = min(max(wi, 0), W - 1);
                const uint4 u = __ldg(img + ((size_t)hc * W + wc) * C8);
                v[5 * r + t] = (hi == hc && wi == wc) ? u : NEG;
            }
        // column-wise maxima of the three rows each pooled row needs, then across columns
#pragma unroll
        for (int a = 0; a < 2; ++a) {
            uint4 colmax[5];
#pragma unroll
            for (int t = 0; t < 5; ++t) {
                uint4 m = v[5 * (2 * a) + t];
                __nv_bfloat162* mm = reinterpret_cast<__nv_bfloat162*>(&m);
#pragma unroll
                for (int r = 1; r < 3; ++r) {
                    const __nv_bfloat162* uu = reinterpret_cast<const __nv_bfloat162*>(&v[5 * (2 * a + r) + t]);
#pragma unroll
                    for (int k = 0; k < 4; ++k) mm[k] = __hmax2(mm[k], uu[k]);
                }
                colmax[t] = m;
            }
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                uint4 m = colmax[2 * b];
                __nv_bfloat162* mm = reinterpret_cast<__nv_bfloat162*>(&m);
#pragma unroll
                for (int t = 1; t < 3; ++t) {
                    const __nv_bfloat162* uu = reinterpret_cast<const __nv_bfloat162*>(&colmax[2 * b + t]);
#pragma unroll
                    for (int k = 0; k < 4; ++k) mm[k] = __hmax2(mm[k], uu[k]);
                }
                if (ho + a < Ho && wo + b < Wo) y[(((size_t)n * Ho + ho + a) * Wo + wo + b) * C8 + c8] = m;
            }
        }
    }
}
__global__ void maxpool_scalar_kernel(int B, int H, int W, int C, int Ho, int Wo, int k, int s, int p,
                                      const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ y,
                                      int32_t* __restrict__ argmax) {
    const size_t total = (size_t)B * Ho * Wo * C;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int c = (int)(i % C);
        size_t q = i / C;
        const int wo = (int)(q % Wo); q /= Wo;
        const int ho = (int)(q % Ho);
        const int n = (int)(q / Ho);
        float best = 0.f; int where = -1;
        for (int r = 0; r < k; ++r) {
            const int hi = ho * s - p + r;
            if (hi < 0 || hi >= H) continue;
            for (int t = 0; t < k; ++t) {
                const int wi = wo * s - p + t;
                if (wi < 0 || wi >= W) continue;
                const float v = __bfloat162float(x[(((size_t)n * H + hi) * W + wi) * C + c]);
                if (where < 0 || v > best) { best = v; where = hi * W + wi; }
            }
        }
        y[i] = __float2bfloat16_rn(best);
        if (argmax) argmax[i] = where;
    }
}

// ---------------------------------------------------------------- LRN across channels
// One thread per (pixel, 8 channels).  It loads its own 16 bytes and the 16-byte groups on either
// side (served by L1: the neighbouring threads load them as their own), so HBM sees the tensor
// once.  Window half-width up to 8.
__device__ __forceinline__ void unpack8(const uint4& q, float* v) {
    const uint32_t* u = reinterpret_cast<const uint32_t*>(&q);
#pragma unroll
    for (int j = 0; j < 4; ++j) { v[2 * j] = bf16_lo(u[j]); v[2 * j + 1] = bf16_hi(u[j]); }
}
// MAXH: largest half-window this instantiation handles (2 for the usual window of five: two predicated steps
// instead of eight)
// The scale (kappa + alpha_n ss)^(-beta) = kappa^(-beta) (1 + u)^(-beta), u = alpha_n ss / kappa: while u < 1/256 for all
// eight sums of every lane of the warp, its series to the u^2 term is exact to float32 resolution (the next term is below
// 4e-8) and needs no special-function unit; ser = {kappa^(-beta), c1 alpha_n / kappa ..., c2 (alpha_n / kappa)^2 ..., the ss limit}.
template <int MAXH>
__global__ void lrn_kernel(size_t nvec, int C8, int half, float alpha_n, float beta, float kappa, float4 ser,
                           const uint4* __restrict__ x, uint4* __restrict__ y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    int c8 = (int)(i0 % C8);                              // advances by a fixed step: one division per thread
    const int step = (int)(stride % C8);
    for (size_t i = i0; i < nvec; i += stride, c8 = c8 + step >= C8 ? c8 + step - C8 : c8 + step) {
        float v[24];
        unpack8(__ldg(x + i), v + 8);
        if (c8 > 0) unpack8(__ldg(x + i - 1), v);
        else {
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = 0.f;
        }
        if (c8 + 1 < C8) unpack8(__ldg(x + i + 1), v + 16);
        else {
#pragma unroll
            for (int j = 0; j < 8; ++j) v[16 + j] = 0.f;
        }
        float sq[24];
#pragma unroll
        for (int j = 0; j < 24; ++j) sq[j] = v[j] * v[j];
        float r[8], ssv[8], smax = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float ss = sq[8 + j];
#pragma unroll
            for (int d = 1; d <= MAXH; ++d)
                if (d <= half) ss += sq[8 + j - d] + sq[8 + j + d];
            ssv[j] = ss;
            smax = fmaxf(smax, ss);
        }
        if (__all_sync(__activemask(), smax < ser.w)) {
#pragma unroll
            for (int j = 0; j < 8; ++j) r[j] = v[8 + j] * fmaf(ssv[j], fmaf(ssv[j], ser.z, ser.y), ser.x);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) r[j] = v[8 + j] * lrn_pow(kappa + alpha_n * ssv[j], beta);
        }
        uint4 o;
        uint32_t* uo = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
        for (int j = 0; j < 4; ++j) uo[j] = pack_bf16(r[2 * j], r[2 * j + 1]);
        y[i] = o;
    }
}
__global__ void lrn_scalar_kernel(size_t n, int C, int half, float alpha_n, float beta, float kappa,
                                  const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const int c = (int)(i % C);
        float ss = 0.f;
        for (int d = -half; d <= half; ++d)
            if (c + d >= 0 && c + d < C) { const float t = __bfloat162float(x[i + d]); ss += t * t; }
        y[i] = __float2bfloat16_rn(__bfloat162float(x[i]) * lrn_pow(kappa + alpha_n * ss, beta));
    }
}

// ---------------------------------------------------------------- concat: strided channel copy
__global__ void concat_kernel(size_t nvec, int C8, int ldc8, int coff8, const uint4* __restrict__ x,
                              uint4* __restrict__ y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += stride) {
        const size_t pix = i / C8;
        const int c8 = (int)(i % C8);
        y[pix * ldc8 + coff8 + c8] = __ldg(x + i);
    }
}
__global__ void concat_scalar_kernel(size_t n, int C, int ldc, int coff, const __nv_bfloat16* __restrict__ x,
                                     __nv_bfloat16* __restrict__ y) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        y[(i / C) * ldc + coff + (i % C)] = x[i];
}

// ---------------------------------------------------------------- global average pool
// One block per (image, 64-channel slab): threads split the plane, partial sums meet in shared
// memory in a fixed order (deterministic).  blockDim = (64 channels / 2, PIXSPLIT).
// For C a multiple of 8: one block per (image, slab of 64 channels), blockDim = (8 channel groups, 32 pixel lanes): a
// thread sums every 32nd position of its 8 channels (16-byte loads, all of them in flight at once for planes up to 64
// pixels); the 32 partial sums of a channel meet in shared memory and are added in lane order (deterministic).
__global__ void __launch_bounds__(256) avgpool8_kernel(int HW, int C8, const uint4* __restrict__ x, uint4* __restrict__ y) {
    __shared__ float part[32][8][9];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // see maxpool_kernel
    asm volatile("griddepcontrol.wait;" ::: "memory");                // no-op unless launched with programmatic serialization
    const int n = blockIdx.y, c8 = blockIdx.x * 8 + threadIdx.x, py = threadIdx.y;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (c8 < C8) {
        const uint4* src = x + (size_t)n * HW * C8 + c8;
        for (int q0 = py; q0 < HW; q0 += 64) {
            const bool two = q0 + 32 < HW;
            const uint4 v = __ldg(src + (size_t)q0 * C8);
            const uint4 u = two ? __ldg(src + (size_t)(q0 + 32) * C8) : make_uint4(0, 0, 0, 0);
            acc[0] += bf16_lo(v.x); acc[1] += bf16_hi(v.x); acc[2] += bf16_lo(v.y); acc[3] += bf16_hi(v.y);
            acc[4] += bf16_lo(v.z); acc[5] += bf16_hi(v.z); acc[6] += bf16_lo(v.w); acc[7] += bf16_hi(v.w);
            acc[0] += bf16_lo(u.x); acc[1] += bf16_hi(u.x); acc[2] += bf16_lo(u.y); acc[3] += bf16_hi(u.y);
            acc[4] += bf16_lo(u.z); acc[5] += bf16_hi(u.z); acc[6] += bf16_lo(u.w); acc[7] += bf16_hi(u.w);
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) part[py][threadIdx.x][j] = acc[j];
    __syncthreads();
    const int t = py * 8 + threadIdx.x;                  // 64 threads finish: (channel group, channel)
    if (t < 64) {
        const int g = t >> 3, j = t & 7;
        float sum = 0.f;
#pragma unroll
        for (int k = 0; k < 32; ++k) sum += part[k][g][j];
        part[0][g][j] = sum / (float)HW;
    }
    __syncthreads();
    if (py == 0 && c8 < C8) {
        const float* r = part[0][threadIdx.x];
        y[(size_t)n * C8 + c8] = make_uint4(pack_bf16(r[0], r[1]), pack_bf16(r[2], r[3]), pack_bf16(r[4], r[5]), pack_bf16(r[6], r[7]));
    }
}

constexpr int AVG_SPLIT = 8;
__global__ void avgpool_kernel(int HW, int C, const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ y) {
    __shared__ float part[AVG_SPLIT][64];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // see maxpool_noarg_kernel
    const int n = blockIdx.y, c = blockIdx.x * 64 + threadIdx.x * 2;
    float s0 = 0.f, s1 = 0.f;
    if (c < C) {
        for (int q = threadIdx.y; q < HW; q += AVG_SPLIT) {
            const __nv_bfloat16* p = x + ((size_t)n * HW + q) * C + c;
            if (c + 1 < C) {
                const uint32_t u = *reinterpret_cast<const uint32_t*>(p);
                s0 += bf16_lo(u); s1 += bf16_hi(u);
            } else {
                s0 += __bfloat162float(p[0]);
            }
        }
    }
    part[threadIdx.y][threadIdx.x * 2] = s0;
    part[threadIdx.y][threadIdx.x * 2 + 1] = s1;
    __syncthreads();
    if (threadIdx.y == 0) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float s = 0.f;
#pragma unroll
            for (int k = 0; k < AVG_SPLIT; ++k) s += part[k][threadIdx.x * 2 + h];
            if (c + h < C) y[(size_t)n * C + c + h] = __float2bfloat16_rn(s / (float)HW);
        }
    }
}

// ---------------------------------------------------------------- Lemma 2: BN/Scale fold
// One block per output channel j; eta_j computed once per thread, weights streamed.
__global__ void fold_bn_kernel(int K, const __nv_bfloat16* __restrict__ w_in, const float* __restrict__ b_in,
                               const float* __restrict__ mean, const float* __restrict__ var, float inv_m, float eps,
                               const float* __restrict__ gamma, const float* __restrict__ beta,
                               __nv_bfloat16* __restrict__ w_out, float* __restrict__ b_out) {
    const int j = blockIdx.x;
    const float eta = gamma[j] / sqrtf(var[j] * inv_m + eps);
    for (int i = threadIdx.x; i < K; i += blockDim.x)
        w_out[(size_t)j * K + i] = __float2bfloat16_rn(eta * __bfloat162float(w_in[(size_t)j * K + i]));
    if (threadIdx.x == 0) b_out[j] = eta * (b_in ? b_in[j] : 0.f) + beta[j] - eta * mean[j] * inv_m;
}

// ---------------------------------------------------------------- zero-embedding of a small filter
__global__ void embed_filter_kernel(int Cin, int ks, int kb, const __nv_bfloat16* __restrict__ w_small, int joff,
                                    __nv_bfloat16* __restrict__ w_big) {
    const int j = blockIdx.x, o = (kb - ks) / 2;
    const int per = kb * kb * Cin;
    for (int i = threadIdx.x; i < per; i += blockDim.x) {
        const int c = i % Cin, t = i / Cin, s = t % kb - o, r = t / kb - o;
        __nv_bfloat16 v = __float2bfloat16_rn(0.f);
        if (r >= 0 && r < ks && s >= 0 && s < ks) v = w_small[(((size_t)j * ks + r) * ks + s) * Cin + c];
        w_big[(size_t)(joff + j) * per + i] = v;
    }
}

// ---------------------------------------------------------------- grouped filters as block-diagonal dense filters
// w_grouped [Cout][k][k][Cin_g] -> w_dense [Cout][k][k][Cin_g * groups]: filter j keeps its values at the input
// channels of its own group (j / (Cout / groups)) and is zero elsewhere.
__global__ void embed_groups_kernel(int Cout, int Cin_g, int kk, int groups, const __nv_bfloat16* __restrict__ w_grouped,
                                    __nv_bfloat16* __restrict__ w_dense) {
    const int j = blockIdx.x, g = j / (Cout / groups);
    const int Cin = Cin_g * groups, per = kk * Cin;
    for (int i = threadIdx.x; i < per; i += blockDim.x) {
        const int c = i % Cin, t = i / Cin, cg = c - g * Cin_g;
        __nv_bfloat16 v = __float2bfloat16_rn(0.f);
        if (cg >= 0 && cg < Cin_g) v = w_grouped[((size_t)j * kk + t) * Cin_g + cg];
        w_dense[(size_t)j * per + i] = v;
    }
}

// ---------------------------------------------------------------- space-to-depth form of a strided few-channel convolution
// y[n][R][S][(ah*s + aw)*C + c] = x[n][R*s + ah - pad][S*s + aw - pad][c] (zero outside the image and for channels
// >= s*s*C); one thread per 8 output channels.
__global__ void s2d_kernel(size_t total8, int H, int W, int C, int s, int pad, int Hs, int Ws, int Cp, const unsigned short* __restrict__ x,
                           uint4* __restrict__ y) {
    const int c8n = Cp >> 3;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total8; i += (size_t)gridDim.x * blockDim.x) {
        const int c8 = (int)(i % c8n);
        size_t pix = i / c8n;
        const int S = (int)(pix % Ws); pix /= Ws;
        const int R = (int)(pix % Hs);
        const size_t n = pix / Hs;
        unsigned short e[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int ch = c8 * 8 + j;
            unsigned short v = 0;
            if (ch < s * s * C) {
                const int a = ch / C, c = ch - a * C;
                const int ah = a / s, aw = a - ah * s;
                const int h = R * s + ah - pad, w = S * s + aw - pad;
                if (h >= 0 && h < H && w >= 0 && w < W) v = __ldg(x + ((n * H + h) * W + w) * C + c);
            }
            e[j] = v;
        }
        uint4 o;
        o.x = e[0] | ((uint32_t)e[1] << 16); o.y = e[2] | ((uint32_t)e[3] << 16);
        o.z = e[4] | ((uint32_t)e[5] << 16); o.w = e[6] | ((uint32_t)e[7] << 16);
        y[i] = o;
    }
}

// The same copy for s*C a multiple of 4 (e.g. stride 4 over 3 channels): one thread per (output pixel, ah) moves the
// s*C contiguous input elements of image row R*s + ah - pad, columns S*s - pad .. S*s - pad + s - 1, to output
// channels [ah*s*C, (ah+1)*s*C) with 8-byte stores; the thread with ah = 0 also clears channels [s*s*C, Cp).
__global__ void s2d_rows_kernel(size_t total, int H, int W, int C, int s, int pad, int Hs, int Ws, int Cp, const unsigned short* __restrict__ x,
                                unsigned short* __restrict__ y) {
    const int run = s * C;                                   // elements per (pixel, ah); multiple of 4
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int ah = (int)(i % s);
        size_t pix = i / s;
        const int S = (int)(pix % Ws);
        const size_t nr = pix / Ws;                          // n * Hs + R
        const int R = (int)(nr % Hs);
        const size_t n = nr / Hs;
        const int h = R * s + ah - pad, w0 = S * s - pad;
        const bool row_ok = h >= 0 && h < H;
        const unsigned short* src = x + ((n * H + (row_ok ? h : 0)) * W) * C;
        uint2* dst = reinterpret_cast<uint2*>(y + pix * Cp + (size_t)ah * run);
        for (int e = 0; e < run; e += 4) {
            unsigned short v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int idx = e + j, w = w0 + idx / C;     // element idx of the run = (aw, c)
                v[j] = (row_ok && w >= 0 && w < W) ? __ldg(src + ((long long)w0 * C + idx)) : (unsigned short)0;
            }
            dst[e >> 2] = make_uint2(v[0] | ((uint32_t)v[1] << 16), v[2] | ((uint32_t)v[3] << 16));
        }
        if (ah == 0) {
            uint2* z = reinterpret_cast<uint2*>(y + pix * Cp + (size_t)s * run);
            for (int e = 0; e < Cp - s * run; e += 4) z[e >> 2] = make_uint2(0u, 0u);
        }
    }
}

// w [Cout][k][k][C] -> w_out [Cout][kp][kp][Cp], kp = ceil(k/s): tap (R*s + ah, S*s + aw) of the original filter
// becomes channel (ah*s + aw)*C + c of tap (R, S); taps past k and channels past s*s*C are zero.
__global__ void s2d_filter_kernel(int k, int C, int s, int kp, int Cp, const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ w_out) {
    const int j = blockIdx.x, per = kp * kp * Cp;
    for (int i = threadIdx.x; i < per; i += blockDim.x) {
        const int ch = i % Cp, t = i / Cp, S = t % kp, R = t / kp;
        __nv_bfloat16 v = __float2bfloat16_rn(0.f);
        if (ch < s * s * C) {
            const int a = ch / C, c = ch - a * C;
            const int r = R * s + a / s, q = S * s + a % s;
            if (r < k && q < k) v = w[(((size_t)j * k + r) * k + q) * C + c];
        }
        w_out[(size_t)j * per + i] = v;
    }
}

// The inverse gather, for gradients: dw [Cout][k][k][C] (float32) takes each element from the one place of
// dw_s2d [Cout][kp][kp][Cp] that s2d_filter_kernel copies it to; the places that hold structural zeros are not read.
__global__ void s2d_filter_grad_kernel(int k, int C, int s, int kp, int Cp, const float* __restrict__ dw_s2d, float* __restrict__ dw) {
    const int j = blockIdx.x, per = k * k * C;
    for (int i = threadIdx.x; i < per; i += blockDim.x) {
        const int c = i % C, t = i / C, q = t % k, r = t / k;
        const int R = r / s, S = q / s, a = (r - R * s) * s + (q - S * s);
        dw[(size_t)j * per + i] = dw_s2d[(((size_t)j * kp + R) * kp + S) * Cp + a * C + c];
    }
}

}  // namespace dr

// ================================================================ C ABI
using namespace dr;
#define DR_REQUIRE(cond, code) do { if (!(cond)) return (code); } while (0)

extern "C" {

const char* dr_strerror(int status) {
    switch (status) {
        case DR_OK: return "ok";
        case DR_ERR_INVALID_ARG: return "invalid argument";
        case DR_ERR_UNSUPPORTED: return "unsupported configuration";
        case DR_ERR_ALIGNMENT: return "pointer, channel stride or channel offset misaligned";
        case DR_ERR_WORKSPACE: return "workspace missing or too small, or net not prepared";
        case DR_ERR_CUDA: return "CUDA call failed";
        case DR_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
        default: return "unknown status";
    }
}

long long dr_launch_count(void) { return g_launches.load(); }

int dr_device_status(int info[4]) {
    int h[4] = {0, 0, 0, 0};
    if (cudaDeviceSynchronize() != cudaSuccess) return DR_ERR_CUDA;
    if (cudaMemcpyFromSymbol(h, g_dev_status, sizeof(h)) != cudaSuccess) return DR_ERR_CUDA;
    if (h[0] != 0) {
        int z[4] = {0, 0, 0, 0};
        if (cudaMemcpyToSymbol(g_dev_status, z, sizeof(z)) != cudaSuccess) return DR_ERR_CUDA;
    }
    if (info) for (int i = 0; i < 4; ++i) info[i] = h[i];
    return h[0] == 0 ? DR_OK : DR_ERR_DEVICE_TIMEOUT;
}

int dr_relu(size_t n, const void* x, void* y, void* stream) {
    DR_REQUIRE(x && y, DR_ERR_INVALID_ARG);
    if (n == 0) return DR_OK;
    DR_REQUIRE(aligned16(x) && aligned16(y), DR_ERR_ALIGNMENT);
    relu_kernel<<<grid_for((n + 7) / 8, 256), 256, 0, (cudaStream_t)stream>>>(n / 8, n, (const uint4*)x, (uint4*)y);
    count_launch();
    return launch_status();
}

int dr_add(size_t n, const void* a, const void* b, void* y, void* stream) {
    DR_REQUIRE(a && b && y, DR_ERR_INVALID_ARG);
    if (n == 0) return DR_OK;
    DR_REQUIRE(aligned16(a) && aligned16(b) && aligned16(y), DR_ERR_ALIGNMENT);
    add_kernel<<<grid_for((n + 7) / 8, 256), 256, 0, (cudaStream_t)stream>>>(n / 8, n, (const uint4*)a, (const uint4*)b, (uint4*)y);
    count_launch();
    return launch_status();
}

int dr_bn(int B, int H, int W, int C, const void* x, const float* mean, const float* var, float m, float eps,
          const float* gamma, const float* beta, void* y, void* stream) {
    DR_REQUIRE(x && y && mean && var, DR_ERR_INVALID_ARG);
    DR_REQUIRE(B >= 0 && H >= 0 && W >= 0 && C > 0 && m != 0.f && eps >= 0.f, DR_ERR_INVALID_ARG);
    DR_REQUIRE(gamma == nullptr || beta != nullptr, DR_ERR_INVALID_ARG);
    const size_t n = (size_t)B * H * W * C;
    if (n == 0) return DR_OK;
    DR_REQUIRE(aligned16(x) && aligned16(y), DR_ERR_ALIGNMENT);
    if (C % 8 == 0 && C <= 4096)
        bn_smem_kernel<<<grid_for(n / 8, 256), 256, 2 * C * sizeof(float), (cudaStream_t)stream>>>(n / 8, C / 8, (const uint4*)x, mean, var, 1.f / m, eps, gamma, beta, (uint4*)y);
    else if (C % 8 == 0)
        bn_kernel<<<grid_for(n / 8, 256), 256, 0, (cudaStream_t)stream>>>(n / 8, C / 8, (const uint4*)x, mean, var, 1.f / m, eps, gamma, beta, (uint4*)y);
    else
        bn_scalar_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(n, C, (const __nv_bfloat16*)x, mean, var, 1.f / m, eps, gamma, beta, (__nv_bfloat16*)y);
    count_launch();
    return launch_status();
}

int dr_scale(int B, int H, int W, int C, const void* x, const float* gamma, const float* beta, void* y, void* stream) {
    DR_REQUIRE(x && y && gamma && beta, DR_ERR_INVALID_ARG);
    DR_REQUIRE(B >= 0 && H >= 0 && W >= 0 && C > 0, DR_ERR_INVALID_ARG);
    const size_t n = (size_t)B * H * W * C;
    if (n == 0) return DR_OK;
    DR_REQUIRE(aligned16(x) && aligned16(y), DR_ERR_ALIGNMENT);
    if (C % 8 == 0 && C <= 4096)
        bn_smem_kernel<<<grid_for(n / 8, 256), 256, 2 * C * sizeof(float), (cudaStream_t)stream>>>(n / 8, C / 8, (const uint4*)x, nullptr, nullptr, 1.f, 0.f, gamma, beta, (uint4*)y);
    else if (C % 8 == 0)
        bn_kernel<<<grid_for(n / 8, 256), 256, 0, (cudaStream_t)stream>>>(n / 8, C / 8, (const uint4*)x, nullptr, nullptr, 1.f, 0.f, gamma, beta, (uint4*)y);
    else
        bn_scalar_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(n, C, (const __nv_bfloat16*)x, nullptr, nullptr, 1.f, 0.f, gamma, beta, (__nv_bfloat16*)y);
    count_launch();
    return launch_status();
}

int dr_maxpool(int B, int H, int W, int C, int k, int s, int p, const void* x, void* y, int32_t* argmax, void* stream) {
    DR_REQUIRE(x && y, DR_ERR_INVALID_ARG);
    DR_REQUIRE(B >= 0 && H > 0 && W > 0 && C > 0 && k > 0 && s > 0 && p >= 0 && 2 * p < k + 1 && p < k, DR_ERR_INVALID_ARG);
    DR_REQUIRE(H + 2 * p >= k && W + 2 * p >= k, DR_ERR_INVALID_ARG);
    const int Ho = (H + 2 * p - k) / s + 1, Wo = (W + 2 * p - k) / s + 1;
    const size_t n = (size_t)B * Ho * Wo * C;
    if (n == 0) return DR_OK;
    DR_REQUIRE(aligned16(x) && aligned16(y) && (!argmax || aligned16(argmax)), DR_ERR_ALIGNMENT);
    if (C % 8 == 0 && !argmax && k == 3 && s == 2 && (size_t)B * ((Ho + 1) / 2) * ((Wo + 1) / 2) * (C / 8) < 0xffffffffull)
        launch_maybe_pdl(maxpool3s2_quad_kernel, dim3(grid_for((size_t)B * ((Ho + 1) / 2) * ((Wo + 1) / 2) * (C / 8), 256)), dim3(256), (cudaStream_t)stream, B, H, W, C / 8, Ho, Wo,
                         p, (const uint4*)x, (uint4*)y);
    else if (C % 8 == 0 && !argmax && k == 3)
        maxpool3_noarg_kernel<<<grid_for(n / 8, 256), 256, 0, (cudaStream_t)stream>>>(B, H, W, C / 8, Ho, Wo, s, p, (const uint4*)x, (uint4*)y);
    else if (C % 8 == 0 && !argmax)
        maxpool_noarg_kernel<<<grid_for(n / 8, 256), 256, 0, (cudaStream_t)stream>>>(B, H, W, C / 8, Ho, Wo, k, s, p, (const uint4*)x, (uint4*)y);
    else if (C % 8 == 0)
        maxpool_kernel<<<grid_for(n / 8, 256), 256, 0, (cudaStream_t)stream>>>(B, H, W, C / 8, Ho, Wo, k, s, p, (const uint4*)x, (uint4*)y, argmax);
    else
        maxpool_scalar_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(B, H, W, C, Ho, Wo, k, s, p, (const __nv_bfloat16*)x, (__nv_bfloat16*)y, argmax);
    count_launch();
    return launch_status();
}

int dr_lrn(int B, int H, int W, int C, int size, float alpha, float beta, float k, const void* x, void* y, void* stream) {
    DR_REQUIRE(x && y, DR_ERR_INVALID_ARG);
    DR_REQUIRE(B >= 0 && H >= 0 && W >= 0 && C > 0 && size >= 1 && (size & 1) && size <= 15, DR_ERR_INVALID_ARG);
    const size_t n = (size_t)B * H * W * C;
    if (n == 0) return DR_OK;
    DR_REQUIRE(aligned16(x) && aligned16(y), DR_ERR_ALIGNMENT);
    float4 ser = make_float4(0.f, 0.f, 0.f, -1.f);          // no series unless kappa > 0 and alpha >= 0
    if (k > 0.f && alpha >= 0.f) {
        const double au = (double)(alpha / size) / k, kp = pow((double)k, -(double)beta), be = beta;
        ser = make_float4((float)kp, (float)(-be * kp * au), (float)(be * (be + 1) / 2 * kp * au * au), au > 0 ? (float)(0.00390625 / au) : 3.0e38f);
    }
    if (C % 8 == 0)
        if (size / 2 <= 2)
            lrn_kernel<2><<<grid_for(n / 8, 256), 256, 0, (cudaStream_t)stream>>>(n / 8, C / 8, size / 2, alpha / size, beta, k, ser, (const uint4*)x, (uint4*)y);
        else
            lrn_kernel<8><<<grid_for(n / 8, 256), 256, 0, (cudaStream_t)stream>>>(n / 8, C / 8, size / 2, alpha / size, beta, k, ser, (const uint4*)x, (uint4*)y);
    else
        lrn_scalar_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(n, C, size / 2, alpha / size, beta, k, (const __nv_bfloat16*)x, (__nv_bfloat16*)y);
    count_launch();
    return launch_status();
}

int dr_concat(size_t npix, int C, const void* x, int ldc, int coff, void* y, void* stream) {
    DR_REQUIRE(x && y && C > 0 && ldc >= C && coff >= 0 && coff + C <= ldc, DR_ERR_INVALID_ARG);
    if (npix == 0) return DR_OK;
    DR_REQUIRE(aligned16(x) && aligned16(y), DR_ERR_ALIGNMENT);
    const size_t n = npix * C;
    if (C % 8 == 0 && ldc % 8 == 0 && coff % 8 == 0)
        concat_kernel<<<grid_for(n / 8, 256), 256, 0, (cudaStream_t)stream>>>(n / 8, C / 8, ldc / 8, coff / 8, (const uint4*)x, (uint4*)y);
    else
        concat_scalar_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(n, C, ldc, coff, (const __nv_bfloat16*)x, (__nv_bfloat16*)y);
    count_launch();
    return launch_status();
}

int dr_avgpool_global(int B, int H, int W, int C, const void* x, void* y, void* stream) {
    DR_REQUIRE(x && y && B >= 0 && H > 0 && W > 0 && C > 0, DR_ERR_INVALID_ARG);
    if (B == 0) return DR_OK;
    DR_REQUIRE(aligned16(x) && aligned16(y), DR_ERR_ALIGNMENT);
    DR_REQUIRE(C % 2 == 0, DR_ERR_UNSUPPORTED);
    if (C % 8 == 0) {
        dim3 grid((C / 8 + 7) / 8, B), block(8, 32);
        launch_maybe_pdl(avgpool8_kernel, grid, block, (cudaStream_t)stream, H * W, C / 8, (const uint4*)x, (uint4*)y);
        count_launch();
        return launch_status();
    }
    dim3 grid((C + 63) / 64, B), block(32, AVG_SPLIT);
    avgpool_kernel<<<grid, block, 0, (cudaStream_t)stream>>>(H * W, C, (const __nv_bfloat16*)x, (__nv_bfloat16*)y);
    count_launch();
    return launch_status();
}

int dr_fold_bn(int Cout, int K, const void* w_in, const float* b_in, const float* mean, const float* var, float m,
               float eps, const float* gamma, const float* beta, void* w_out, float* b_out, void* stream) {
    DR_REQUIRE(w_in && mean && var && gamma && beta && w_out && b_out, DR_ERR_INVALID_ARG);
    DR_REQUIRE(Cout > 0 && K > 0 && m != 0.f && eps >= 0.f, DR_ERR_INVALID_ARG);
    fold_bn_kernel<<<Cout, 256, 0, (cudaStream_t)stream>>>(K, (const __nv_bfloat16*)w_in, b_in, mean, var, 1.f / m, eps, gamma, beta, (__nv_bfloat16*)w_out, b_out);
    count_launch();
    return launch_status();
}

int dr_embed_filter(int Cout, int Cin, int ks, int kb, const void* w_small, int joff, void* w_big, void* stream) {
    DR_REQUIRE(w_small && w_big, DR_ERR_INVALID_ARG);
    DR_REQUIRE(Cout > 0 && Cin > 0 && ks > 0 && kb >= ks && (ks & 1) && (kb & 1) && joff >= 0, DR_ERR_INVALID_ARG);
    embed_filter_kernel<<<Cout, 256, 0, (cudaStream_t)stream>>>(Cin, ks, kb, (const __nv_bfloat16*)w_small, joff, (__nv_bfloat16*)w_big);
    count_launch();
    return launch_status();
}

int dr_space_to_depth(int B, int H, int W, int C, int k, int s, int pad, int Cp, const void* x, void* y, void* stream) {
    DR_REQUIRE(x && y && B >= 0 && H > 0 && W > 0 && C > 0 && k > 0 && s > 0 && pad >= 0, DR_ERR_INVALID_ARG);
    DR_REQUIRE(H + 2 * pad >= k && W + 2 * pad >= k && Cp >= s * s * C && (Cp & 7) == 0, DR_ERR_INVALID_ARG);
    DR_REQUIRE(aligned16(x) && aligned16(y), DR_ERR_ALIGNMENT);
    const int kp = (k + s - 1) / s;
    const int Hs = (H + 2 * pad - k) / s + kp, Ws = (W + 2 * pad - k) / s + kp;     // Ho + kp - 1
    const size_t total8 = (size_t)B * Hs * Ws * (Cp / 8);
    if (total8 == 0) return DR_OK;
    if ((s * C) % 4 == 0 && (Cp - s * s * C) % 4 == 0) {
        const size_t total = (size_t)B * Hs * Ws * s;
        s2d_rows_kernel<<<grid_for(total, 256), 256, 0, (cudaStream_t)stream>>>(total, H, W, C, s, pad, Hs, Ws, Cp, (const unsigned short*)x,
                                                                                 (unsigned short*)y);
    } else {
        s2d_kernel<<<grid_for(total8, 256), 256, 0, (cudaStream_t)stream>>>(total8, H, W, C, s, pad, Hs, Ws, Cp, (const unsigned short*)x, (uint4*)y);
    }
    count_launch();
    return launch_status();
}

int dr_s2d_filter(int Cout, int k, int C, int s, int Cp, const void* w, void* w_out, void* stream) {
    DR_REQUIRE(w && w_out && Cout > 0 && k > 0 && C > 0 && s > 0 && Cp >= s * s * C, DR_ERR_INVALID_ARG);
    const int kp = (k + s - 1) / s;
    s2d_filter_kernel<<<Cout, 256, 0, (cudaStream_t)stream>>>(k, C, s, kp, Cp, (const __nv_bfloat16*)w, (__nv_bfloat16*)w_out);
    count_launch();
    return launch_status();
}

int dr_s2d_filter_grad(int Cout, int k, int C, int s, int Cp, const float* dw_s2d, float* dw, void* stream) {
    DR_REQUIRE(dw_s2d && dw && Cout > 0 && k > 0 && C > 0 && s > 0 && Cp >= s * s * C, DR_ERR_INVALID_ARG);
    const int kp = (k + s - 1) / s;
    s2d_filter_grad_kernel<<<Cout, 256, 0, (cudaStream_t)stream>>>(k, C, s, kp, Cp, dw_s2d, dw);
    count_launch();
    return launch_status();
}

int dr_embed_groups(int Cout, int Cin_g, int k, int groups, const void* w_grouped, void* w_dense, void* stream) {
    DR_REQUIRE(w_grouped && w_dense, DR_ERR_INVALID_ARG);
    DR_REQUIRE(Cout > 0 && Cin_g > 0 && k > 0 && groups > 0 && Cout % groups == 0, DR_ERR_INVALID_ARG);
    embed_groups_kernel<<<Cout, 256, 0, (cudaStream_t)stream>>>(Cout, Cin_g, k * k, groups, (const __nv_bfloat16*)w_grouped, (__nv_bfloat16*)w_dense);
    count_launch();
    return launch_status();
}

}  // extern "C"
