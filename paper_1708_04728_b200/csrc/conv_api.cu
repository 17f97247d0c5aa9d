// dr_conv_slim / dr_inception_slim: validation, tiling choice and kernel dispatch.
#include <cmath>

#include "conv_common.cuh"

namespace dr {

static std::atomic<int> g_forced_path{DR_PATH_AUTO};    // test hooks: process-wide, read and written atomically
static std::atomic<int> g_last_path{-1};

// Fill the derived fields of ConvParams from a descriptor.  Returns a status.
int conv_make_params(const dr_conv_desc* d, int B, int H, int W, const void* x, const void* w, const float* b,
                     const void* residual, void* y, int32_t* argmax, ConvParams* out) {
    if (!d || !x || !w || !y) return DR_ERR_INVALID_ARG;
    if (d->k <= 0 || d->stride <= 0 || d->pad < 0 || d->Cin <= 0 || d->Cout <= 0) return DR_ERR_INVALID_ARG;
    if (B < 0 || H <= 0 || W <= 0) return DR_ERR_INVALID_ARG;
    if (H + 2 * d->pad < d->k || W + 2 * d->pad < d->k) return DR_ERR_INVALID_ARG;
    const unsigned f = d->flags;
    if ((f & DR_BIAS) && !b) return DR_ERR_INVALID_ARG;
    if ((f & DR_RESIDUAL) && !residual) return DR_ERR_INVALID_ARG;
    if ((f & DR_RELU_AFTER_RESIDUAL) && !(f & DR_RESIDUAL)) return DR_ERR_INVALID_ARG;
    if ((f & DR_LRN_BEFORE_POOL) && !((f & DR_LRN) && (f & DR_POOL))) return DR_ERR_INVALID_ARG;
    if (argmax && !(f & DR_POOL)) return DR_ERR_INVALID_ARG;
    const bool staged = f & (DR_POOL | DR_LRN);
    if (staged && (f & (DR_RESIDUAL | DR_OUT_F32))) return DR_ERR_UNSUPPORTED;
    if (staged && (d->Cout > 256 || (d->Cout & 1))) return DR_ERR_UNSUPPORTED;
    if (f & DR_POOL) {
        if (d->pool_k != 3 || d->pool_stride != 2 || d->pool_pad != 1) return DR_ERR_UNSUPPORTED;
    }
    if (f & DR_LRN) {
        if (d->lrn_size < 1 || !(d->lrn_size & 1) || d->lrn_size > 15) return DR_ERR_INVALID_ARG;
    }
    const int ldc = d->y_ldc ? d->y_ldc : d->Cout;
    const int coff = d->y_coff;
    if (ldc < d->Cout || coff < 0 || coff + d->Cout > ldc) return DR_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || (residual && !aligned16(residual))) return DR_ERR_ALIGNMENT;
    if (d->y_ldc && ((ldc & 7) || (coff & 7))) return DR_ERR_ALIGNMENT;

    ConvParams p{};
    p.x = (const __nv_bfloat16*)x; p.w = (const __nv_bfloat16*)w; p.bias = b;
    p.residual = (const __nv_bfloat16*)residual; p.y = y; p.argmax = argmax;
    p.status = dev_status_ptr();
    p.B = B; p.H = H; p.W = W; p.Cin = d->Cin; p.Cout = d->Cout; p.k = d->k; p.stride = d->stride; p.pad = d->pad;
    p.Ho = (H + 2 * d->pad - d->k) / d->stride + 1;
    p.Wo = (W + 2 * d->pad - d->k) / d->stride + 1;
    p.Hy = p.Ho; p.Wy = p.Wo;
    if (f & DR_POOL) {
        if (p.Ho + 2 < 3 || p.Wo + 2 < 3) return DR_ERR_INVALID_ARG;
        p.Hy = (p.Ho + 2 - 3) / 2 + 1; p.Wy = (p.Wo + 2 - 3) / 2 + 1;
    }
    p.K = d->k * d->k * d->Cin;
    p.flags = f;
    p.lrn_half = (f & DR_LRN) ? d->lrn_size / 2 : 0;
    p.lrn_alpha_n = (f & DR_LRN) ? d->lrn_alpha / d->lrn_size : 0.f;
    p.lrn_beta = d->lrn_beta; p.lrn_k = d->lrn_k;
    if (f & DR_LRN) {
        const double be = d->lrn_beta, kk = d->lrn_k;
        p.lrn_inv_k = kk > 0 ? (float)(1.0 / kk) : 0.f;
        p.lrn_kpow = kk > 0 ? (float)pow(kk, -be) : 0.f;
        p.lrn_c1 = (float)(-be);
        p.lrn_c2 = (float)(be * (be + 1) / 2);
        p.lrn_c3 = (float)(-be * (be + 1) * (be + 2) / 6);
        p.lrn_c4 = (float)(be * (be + 1) * (be + 2) * (be + 3) / 24);
        const double au = kk > 0 ? (double)p.lrn_alpha_n / kk : 0.0, kp = kk > 0 ? pow(kk, -be) : 0.0;
        p.lrn_s1 = (float)(kp * p.lrn_c1 * au);
        p.lrn_s2 = (float)(kp * p.lrn_c2 * au * au);
        p.lrn_s3 = (float)(kp * p.lrn_c3 * au * au * au);
        p.lrn_s4 = (float)(kp * p.lrn_c4 * au * au * au * au);
        p.lrn_ss_max = au > 0 ? (float)(0.03125 / au) : 3.0e38f;
        p.lrn_ss_max2 = au > 0 ? (float)(0.00390625 / au) : 3.0e38f;
    }
    p.ldc = ldc; p.coff = coff;
    p.M = (long long)B * p.Ho * p.Wo;
    const int cout16 = (d->Cout + 15) / 16 * 16;
    if (staged) {
        p.Nt = cout16; p.n_blocks = 1;
    } else {
        // Split N into near-equal blocks of at most 256 columns.  Among the smallest block counts pick the one
        // with the lowest estimated time: rounds of the persistent grid (CTA pairs for long-K layers) times the
        // measured cost of a k-block, about 0.2 us of fixed hand-shake plus 1 ns per output column.
        const long long m_tiles = (p.M + TILE_M - 1) / TILE_M;
        const bool pairs = (p.K >= 1024 || (p.k > 1 && p.K >= 512)) && m_tiles >= 2;
        const long long capacity = pairs ? num_sms() / 2 : num_sms();
        const long long m_units = pairs ? (m_tiles + 1) / 2 : m_tiles;
        const int nb_min = (cout16 + 255) / 256;
        double best = -1.0;
        for (int nb = nb_min; nb <= nb_min + 2 && nb * 16 <= cout16; ++nb) {
            const int nt = ((cout16 + nb - 1) / nb + 15) / 16 * 16;
            if ((long long)nt * (nb - 1) >= cout16) continue;          // last block would be empty
            const long long rounds = (m_units * nb + capacity - 1) / capacity;
            const double cost = (double)rounds * (0.20 + 0.00094 * nt);
            if (best < 0 || cost < best * 0.97) { best = cost; p.n_blocks = nb; p.Nt = nt; }
        }
    }
    if (f & DR_POOL) {
        static const int cand[][2] = {{3, 8}, {4, 6}, {5, 5}, {2, 12}, {8, 3}, {6, 4}};
        long best = -1;
        for (auto& c : cand) {
            const long t = (long)((p.Hy + c[0] - 1) / c[0]) * ((p.Wy + c[1] - 1) / c[1]);
            if (best < 0 || t < best) { best = t; p.PH = c[0]; p.PW = c[1]; }
        }
        p.patch = 1;
        p.tiles_h = (p.Hy + p.PH - 1) / p.PH; p.tiles_w = (p.Wy + p.PW - 1) / p.PW;
        const long long mt = (long long)B * p.tiles_h * p.tiles_w;
        if (mt > 0x7fffffffLL) return DR_ERR_UNSUPPORTED;
        p.m_tiles = (int)mt;
    } else {
        const long long mt = (p.M + TILE_M - 1) / TILE_M;
        if (mt > 0x7fffffffLL) return DR_ERR_UNSUPPORTED;
        p.m_tiles = (int)mt;
    }
    *out = p;
    return DR_OK;
}

// The patch-reuse kernel against the im2col kernel.  Its tiles are whole padded image rows, so part of every tile's MMA
// rows is padding (28 x 28 planes: 12.5 %, 14 x 14: 23 %); in exchange the activations are loaded once per channel block
// instead of once per tap, and with at most 128 output channels two tiles per CTA run side by side on double-buffered
// accumulators.  Measured at batch 256 (us, patch-reuse / im2col): a gain for tiles of at most 128 channels on planes of
// 28 x 28 and more (3a merged 5x5 181 / 216, 3a 3x3 55 / 73; ResNet-50 stage 2 and 3 3x3 54 / 61 and 38 / 42), a loss
// where a tile's accumulator takes all its TMEM half or the layer runs on wide tiles (3b 3x3 117 / 90, 4c 3x3 47 / 37,
// 3b merged 5x5 549 / 481, 4a 324 / 248).  DR_QLIN = 0 / 1 overrides (never / wherever it can).
static bool qlin_preferred(const ConvParams& p) {
    const int pref = tunable("DR_QLIN", -1);
    if (pref == 0 || !conv_qlin_supports(p)) return false;
    if (pref > 0) return true;
    const int cout16 = (p.Cout + 15) / 16 * 16;
    return cout16 <= 128 && conv_qlin_fill(p) >= 0.8 && p.m_tiles >= 2 * num_sms();
}

int conv_pick_path(const ConvParams& p, int forced) {
    if (forced == DR_PATH_SIMT) return DR_PATH_SIMT;
    if (forced == DR_PATH_UMMA_GATHER) return conv_umma_gather_supports(p) ? DR_PATH_UMMA_GATHER : -1;
    if (forced == DR_PATH_UMMA_TMA) return conv_umma_tma_supports(p) ? DR_PATH_UMMA_TMA : -1;
    if (forced == DR_PATH_UMMA_PATCH) return conv_patch_tma_supports(p) ? DR_PATH_UMMA_PATCH : -1;
    if (forced == DR_PATH_UMMA_STEM) return conv_stem_supports(p) ? DR_PATH_UMMA_STEM : -1;
    if (forced == DR_PATH_RETIRED_6) return -1;                 // a retired kernel's number: nothing runs under it
    if (forced == DR_PATH_UMMA_STEM_D) return conv_stem_d_supports(p) ? DR_PATH_UMMA_STEM_D : -1;
    if (forced == DR_PATH_UMMA_SPLITK) return conv_splitk_supports(p) ? DR_PATH_UMMA_SPLITK : -1;
    if (forced == DR_PATH_UMMA_QLIN) return conv_qlin_supports(p) ? DR_PATH_UMMA_QLIN : -1;
    if (conv_stem_d_supports(p)) return DR_PATH_UMMA_STEM_D;
    if (conv_stem_supports(p)) return DR_PATH_UMMA_STEM;
    if (conv_patch_tma_supports(p)) return DR_PATH_UMMA_PATCH;
    if (conv_splitk_supports(p)) return DR_PATH_UMMA_SPLITK;   // few output tiles and scratch at hand
    if (qlin_preferred(p)) return DR_PATH_UMMA_QLIN;
    if (conv_umma_tma_supports(p)) return DR_PATH_UMMA_TMA;
    if (conv_umma_gather_supports(p)) return DR_PATH_UMMA_GATHER;
    return DR_PATH_SIMT;
}

int conv_launch_path(const ConvParams& p, int path, cudaStream_t stream) {
    switch (path) {
        case DR_PATH_SIMT: return conv_simt_launch(p, stream);
        case DR_PATH_UMMA_GATHER: return conv_umma_gather_launch(p, stream);
        case DR_PATH_UMMA_TMA: return conv_umma_tma_launch(p, stream);
        case DR_PATH_UMMA_PATCH: return conv_patch_tma_launch(p, stream);
        case DR_PATH_UMMA_STEM: return conv_stem_launch(p, stream);
        case DR_PATH_UMMA_STEM_D: return conv_stem_d_launch(p, stream);
        case DR_PATH_UMMA_SPLITK: return conv_splitk_launch(p, stream);
        case DR_PATH_UMMA_QLIN: return conv_qlin_launch(p, stream);
        default: return DR_ERR_UNSUPPORTED;
    }
}

int forced_conv_path() { return g_forced_path; }

}  // namespace dr

using namespace dr;

extern "C" {

int dr_set_conv_path(int path) {
    if (path < DR_PATH_AUTO || path > DR_PATH_UMMA_QLIN) return DR_ERR_INVALID_ARG;
    g_forced_path = path;
    return DR_OK;
}

int dr_last_conv_path(void) { return g_last_path; }

int dr_conv_slim(const dr_conv_desc* desc, int B, int H, int W, const void* x, const void* w, const float* b,
                 const void* residual, void* y, int32_t* argmax, void* stream) {
    ConvParams p;
    const int st = conv_make_params(desc, B, H, W, x, w, b, residual, y, argmax, &p);
    if (st != DR_OK) return st;
    if (p.M == 0) return DR_OK;
    const int path = conv_pick_path(p, g_forced_path);
    if (path < 0) return DR_ERR_UNSUPPORTED;
    g_last_path = path;
    return conv_launch_path(p, path, (cudaStream_t)stream);
}

int dr_conv_plan(const dr_conv_desc* desc, int B, int H, int W, size_t workspace_bytes, int plan[8]) {
    if (!plan) return DR_ERR_INVALID_ARG;
    ConvParams p;
    const void* dummy = reinterpret_cast<const void*>(uintptr_t(256));   // only alignment is looked at
    const int st = conv_make_params(desc, B, H, W, dummy, dummy, (const float*)dummy, dummy, (void*)dummy, nullptr, &p);
    if (st != DR_OK) return st;
    if (workspace_bytes > (size_t)DR_CONV_WS_COUNTER_BYTES) {
        p.sk_counters = reinterpret_cast<int*>(uintptr_t(256));
        p.sk_scratch = reinterpret_cast<float*>(uintptr_t(256) + DR_CONV_WS_COUNTER_BYTES);
        p.sk_scratch_bytes = workspace_bytes - DR_CONV_WS_COUNTER_BYTES;
    }
    for (int i = 0; i < 8; ++i) plan[i] = 0;
    const int path = p.M > 0 ? conv_pick_path(p, g_forced_path) : DR_PATH_AUTO;
    if (path < 0) return DR_ERR_UNSUPPORTED;
    plan[0] = path; plan[1] = p.Nt; plan[2] = p.n_blocks;
    if (path == DR_PATH_UMMA_TMA) {
        bool pair = false, wide = false;
        conv_umma_tma_shape(&p, &pair, &wide);
        plan[1] = p.Nt; plan[2] = p.n_blocks; plan[3] = pair; plan[4] = wide;
    } else if (path == DR_PATH_UMMA_QLIN) {
        plan[1] = conv_qlin_nt(p); plan[2] = 1; plan[3] = 1; plan[4] = ((p.Cout + 15) / 16 * 16) > 256;
    }
    return DR_OK;
}

int dr_conv_workspace_bytes(const dr_conv_desc* desc, int B, int H, int W, size_t* bytes) {
    if (!bytes) return DR_ERR_INVALID_ARG;
    ConvParams p;
    const void* dummy = reinterpret_cast<const void*>(uintptr_t(256));   // only alignment is looked at
    const int st = conv_make_params(desc, B, H, W, dummy, dummy, (const float*)dummy, dummy, (void*)dummy, nullptr, &p);
    if (st != DR_OK) return st;
    const size_t scratch = p.M > 0 ? conv_splitk_scratch_bytes(p) : 0;
    *bytes = scratch ? (size_t)DR_CONV_WS_COUNTER_BYTES + scratch : 0;
    return DR_OK;
}

int dr_conv_slim_ws(const dr_conv_desc* desc, int B, int H, int W, const void* x, const void* w, const float* b,
                    const void* residual, void* y, int32_t* argmax, void* workspace, size_t workspace_bytes, void* stream) {
    ConvParams p;
    const int st = conv_make_params(desc, B, H, W, x, w, b, residual, y, argmax, &p);
    if (st != DR_OK) return st;
    if (workspace && ((uintptr_t)workspace & 255)) return DR_ERR_ALIGNMENT;
    if (p.M == 0) return DR_OK;
    if (workspace && workspace_bytes > (size_t)DR_CONV_WS_COUNTER_BYTES) {
        p.sk_counters = reinterpret_cast<int*>(workspace);
        p.sk_scratch = reinterpret_cast<float*>(reinterpret_cast<char*>(workspace) + DR_CONV_WS_COUNTER_BYTES);
        p.sk_scratch_bytes = workspace_bytes - DR_CONV_WS_COUNTER_BYTES;
    }
    const int path = conv_pick_path(p, g_forced_path);
    if (path < 0) return DR_ERR_UNSUPPORTED;
    g_last_path = path;
    return conv_launch_path(p, path, (cudaStream_t)stream);
}

int dr_inception_workspace_bytes(const dr_inception_desc* d, int B, int H, int W, size_t* bytes) {
    if (!d || !bytes || B < 0 || H <= 0 || W <= 0 || d->c3r <= 0) return DR_ERR_INVALID_ARG;
    *bytes = ((size_t)B * H * W * d->c3r * 2 + 255) / 256 * 256;
    // pool_after: the module output before pooling lives in the workspace as well
    if (d->pool_after) *bytes += ((size_t)B * H * W * ((size_t)d->c3 + d->cm) * 2 + 255) / 256 * 256;
    return DR_OK;
}

int dr_inception_slim(const dr_inception_desc* d, int B, int H, int W, const void* x, const void* const w[3],
                      const float* const b[3], void* y, void* workspace, void* stream) {
    if (!d || !x || !w || !b || !y) return DR_ERR_INVALID_ARG;
    if (d->Cin <= 0 || d->c3r <= 0 || d->c3 <= 0 || d->cm <= 0) return DR_ERR_INVALID_ARG;
    if (!workspace) return DR_ERR_WORKSPACE;
    for (int i = 0; i < 3; ++i)
        if (!w[i] || !b[i]) return DR_ERR_INVALID_ARG;
    if ((d->c3 & 7) || (d->cm & 7)) return DR_ERR_ALIGNMENT;
    const int ldc = d->c3 + d->cm;
    // pool_after: both convolutions write the un-pooled module output into the workspace (behind the reducer's tensor) and a
    // 3x3 / 2, pad 1 max-pooling layer brings it to y.  (Pooling is per channel, so it commutes with the concatenation; it is
    // not absorbed into these convolutions' epilogues: their tiles are runs of 128 consecutive pixels, not 2-D patches.)
    void* y_out = y;
    if (d->pool_after) y = (char*)workspace + ((size_t)B * H * W * d->c3r * 2 + 255) / 256 * 256;
    dr_conv_desc c{};
    c.flags = DR_BIAS | DR_RELU;
    // 1x1 reducer of the 3x3 path -> workspace
    c.k = 1; c.stride = 1; c.pad = 0; c.Cin = d->Cin; c.Cout = d->c3r; c.y_ldc = 0; c.y_coff = 0;
    int st = dr_conv_slim(&c, B, H, W, x, w[0], b[0], nullptr, workspace, nullptr, stream);
    if (st != DR_OK) return st;
    // 3x3 -> channels [0, c3)
    c.k = 3; c.pad = 1; c.Cin = d->c3r; c.Cout = d->c3; c.y_ldc = ldc; c.y_coff = 0;
    st = dr_conv_slim(&c, B, H, W, workspace, w[1], b[1], nullptr, y, nullptr, stream);
    if (st != DR_OK) return st;
    // merged 5x5 on the module input -> channels [c3, c3+cm)
    c.k = 5; c.pad = 2; c.Cin = d->Cin; c.Cout = d->cm; c.y_ldc = ldc; c.y_coff = d->c3;
    st = dr_conv_slim(&c, B, H, W, x, w[2], b[2], nullptr, y, nullptr, stream);
    if (st != DR_OK || !d->pool_after) return st;
    return dr_maxpool(B, H, W, ldc, 3, 2, 1, y, y_out, nullptr, stream);
}

// ---- dr_inception_slim_static: the same module with its scratch tensor in a fixed device array ----
// Scratch for the 1x1 reducer's output.  File-scope device storage: every GPU that loads this
// library reserves these bytes from load until the process exits.  In host code the symbol is only
// a handle; the address kernels can use comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_inception_static_scratch[DR_INCEPTION_STATIC_SCRATCH_BYTES];

static void* inception_static_scratch_ptr(int* status) {
    static void* ptr[64] = {nullptr};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *status = DR_ERR_CUDA; return nullptr; }
    if (!ptr[dev]) {
        void* q = nullptr;
        if (cudaGetSymbolAddress(&q, g_inception_static_scratch) != cudaSuccess || !q) { *status = DR_ERR_CUDA; return nullptr; }
        ptr[dev] = q;
    }
    *status = DR_OK;
    return ptr[dev];
}

int dr_inception_slim_static(const dr_inception_desc* d, int B, int H, int W, const void* x, const void* const w[3],
                             const float* const b[3], void* y, void* stream) {
    size_t need = 0;
    const int st = dr_inception_workspace_bytes(d, B, H, W, &need);
    if (st != DR_OK) return st;
    if (need > (size_t)DR_INCEPTION_STATIC_SCRATCH_BYTES) return DR_ERR_WORKSPACE;   // too large for the fixed array
    int ps = DR_OK;
    void* scratch = inception_static_scratch_ptr(&ps);
    if (ps != DR_OK) return ps;
    // Nothing in the scratch has to start at zero: the reducer writes every element of its
    // [B,H,W,c3r] output before the 3x3 convolution reads it, so earlier contents never show.
    return dr_inception_slim(d, B, H, W, x, w, b, y, scratch, stream);
}

}  // extern "C"
