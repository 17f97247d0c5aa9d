// dr_net: the two evaluated networks as static layer lists, in slim and unslimmed form.
//
// Slim form (what the paper's method produces, Sections 3.1-3.2): one convolution launch per slim
// layer; BatchNorm/Scale folded into the filters (Lemma 2), ReLU / max-pool / LRN / residual add
// in the epilogue, inception branches merged into one 5x5 convolution writing its slice of the
// concatenated tensor.  Unslimmed form: the original layer sequence (Eq. f_map, Section 3.1),
// every tensor and non-tensor layer a launch of its own with its own round trip through HBM —
// the baseline of Tables 2 and 4.  Both take the same un-slimmed parameter list.
#include <cstring>
#include <string>
#include <vector>

#include "conv_common.cuh"

namespace dr {

int conv_make_params(const dr_conv_desc* d, int B, int H, int W, const void* x, const void* w, const float* b,
                     const void* residual, void* y, int32_t* argmax, ConvParams* out);
int conv_pick_path(const ConvParams& p, int forced);
int conv_launch_path(const ConvParams& p, int path, cudaStream_t stream);
int forced_conv_path();

enum OpKind { OP_CONV, OP_RELU, OP_MAXPOOL, OP_LRN, OP_BN, OP_SCALE, OP_ADD, OP_CONCAT, OP_AVGPOOL, OP_S2D };

struct Tensor {
    int B, H, W, C;
    int is_f32;
    size_t off;       // byte offset inside the activation arena; (size_t)-1: external (input / logits)
    size_t bytes;
};

// A parameter an op consumes: either a user-supplied raw parameter or a derived one that
// dr_net_prepare writes into the workspace.
struct PRef {
    int raw = -1;            // index into params
    size_t ws_off = (size_t)-1;
    const void* resolve(const std::vector<const void*>& raw_ptrs, const char* ws) const {
        if (raw >= 0) return raw_ptrs[raw];
        if (ws_off != (size_t)-1) return ws + ws_off;
        return nullptr;
    }
};

struct Op {
    OpKind kind;
    std::string name;
    int in0 = -2, in1 = -2;  // tensor ids (-1: network input)
    int out = -2, coff = 0;
    dr_conv_desc cd{};       // OP_CONV
    PRef w, b;               // OP_CONV
    PRef v0, v1;             // BN: mean, var; SCALE: gamma, beta
    float eps = 0.f;
    double flops = 0, bytes = 0;
    int path = -1;
    int conv_index = -1;     // OP_CONV: ordinal among the convolutions (its block of split-K counters)
    int pair = -1;           // OP_CONV: a later convolution reading the same input that may share this one's launch,
    int chain = -1;          //          and the convolution that reads this one's output (it may join them)
    int pool_pad = 1;        // OP_MAXPOOL: 3x3 / 2 with this padding
    int s2d_k = 0, s2d_s = 0, s2d_pad = 0;   // OP_S2D: the convolution whose input this op re-lays
    int group = 0;           // decided by dr_net_prepare: 0 own launch, 2 with `pair`, 3 with `pair` and `chain`
};

// Derivations done once by dr_net_prepare
struct FoldJob { int w, mean, var, gamma, beta; size_t w_off, b_off; int Cout, K; };
struct EmbedJob { int w_small; int Cout, Cin, ks, kb, joff; size_t w_off; };
struct CopyJob { int src; size_t dst_off; size_t bytes; };
struct S2dJob { int w; int Cout, k, C, s, Cp; size_t w_off; };
struct GroupJob { int w_grouped; int Cout, Cin_g, k, groups; size_t w_off; };
// Zero-padded copy of a parameter: `rows` rows of `row_bytes` placed `pitch` bytes apart in a zeroed block of `total`.
struct PadJob { int src; size_t dst_off, total, rows, row_bytes, pitch; };

}  // namespace dr

using namespace dr;

struct dr_net {
    int arch, mode, B, H, W;
    std::vector<dr_param_spec> specs;
    std::vector<const void*> raw;
    std::vector<Tensor> tensors;
    std::vector<Op> ops;
    std::vector<FoldJob> folds;
    std::vector<EmbedJob> embeds;
    std::vector<CopyJob> copies;
    std::vector<GroupJob> group_jobs;
    std::vector<S2dJob> s2d_jobs;
    std::vector<PadJob> pad_jobs;
    size_t param_bytes = 0, act_bytes = 0;
    size_t sk_scratch_bytes = 0;   // split-K scratch shared by all layers (they run one after another), after the arena
    int n_conv = 0;                // each convolution has its own block of tile counters after that
    int t_input = -1, t_logits = -1;
    void* prepared_ws = nullptr;
    bool timing = false;
    std::vector<char> done;        // per forward pass: layers that shared an earlier layer's launch
    std::vector<cudaEvent_t> ev;   // 2 per op
    float eps = 1e-5f;

    int param(const std::string& name, int d0, int d1, int d2, int d3, int is_f32) {
        for (size_t i = 0; i < specs.size(); ++i)
            if (name == specs[i].name) return (int)i;
        dr_param_spec s{};
        std::strncpy(s.name, name.c_str(), sizeof(s.name) - 1);
        s.dims[0] = d0; s.dims[1] = d1; s.dims[2] = d2; s.dims[3] = d3;
        s.is_f32 = is_f32;
        s.count = (size_t)d0 * d1 * d2 * d3;
        specs.push_back(s);
        raw.push_back(nullptr);
        return (int)specs.size() - 1;
    }
    int filt(const std::string& n, int cout, int k, int cin) { return param(n + ".w", cout, k, k, cin, 0); }
    int vec(const std::string& n, int c) { return param(n, c, 1, 1, 1, 1); }
    size_t ws_alloc(size_t bytes) {
        const size_t o = param_bytes;
        param_bytes += (bytes + 255) / 256 * 256;
        return o;
    }
    int tensor(int B_, int H_, int W_, int C_, int is_f32 = 0, bool external = false) {
        Tensor t{B_, H_, W_, C_, is_f32, (size_t)-1, (size_t)B_ * H_ * W_ * C_ * (is_f32 ? 4 : 2)};
        if (!external) { t.off = act_bytes; act_bytes += (t.bytes + 255) / 256 * 256; }
        tensors.push_back(t);
        return (int)tensors.size() - 1;
    }
    const Tensor& T(int id) const { return tensors[id]; }
};

namespace dr {

static int out_size(int n, int k, int s, int p) { return (n + 2 * p - k) / s + 1; }

// Append a convolution op reading tensor `in`; creates the output tensor unless `out` is given.
static int add_conv(dr_net* n, const std::string& name, int in, int k, int s, int p, int cout, unsigned flags, PRef w,
                    PRef b, int out = -2, int coff = 0, int residual = -2) {
    const Tensor ti = n->T(in);
    Op op;
    op.kind = OP_CONV; op.name = name; op.in0 = in; op.in1 = residual;
    op.cd.k = k; op.cd.stride = s; op.cd.pad = p; op.cd.Cin = ti.C; op.cd.Cout = cout; op.cd.flags = flags;
    op.cd.pool_k = 3; op.cd.pool_stride = 2; op.cd.pool_pad = 1;
    op.cd.lrn_size = 5; op.cd.lrn_alpha = 1e-4f; op.cd.lrn_beta = 0.75f; op.cd.lrn_k = 1.f;
    int Ho = out_size(ti.H, k, s, p), Wo = out_size(ti.W, k, s, p);
    const long long M = (long long)ti.B * Ho * Wo;
    op.flops = 2.0 * (double)M * cout * k * k * ti.C;
    const double xin = (k == 1 && s > 1) ? (double)M * ti.C * 2 : (double)ti.bytes;
    if (flags & DR_POOL) { Ho = out_size(Ho, 3, 2, 1); Wo = out_size(Wo, 3, 2, 1); }
    if (out == -2) out = n->tensor(ti.B, Ho, Wo, cout, (flags & DR_OUT_F32) ? 1 : 0, (flags & DR_OUT_F32) != 0);
    op.out = out; op.coff = coff;
    op.cd.y_ldc = n->T(out).C; op.cd.y_coff = coff;
    op.w = w; op.b = b;
    op.conv_index = n->n_conv++;
    op.bytes = xin + (double)cout * k * k * ti.C * 2 + (double)ti.B * Ho * Wo * cout * ((flags & DR_OUT_F32) ? 4 : 2) +
               ((flags & DR_RESIDUAL) ? (double)ti.B * Ho * Wo * cout * 2 : 0.0) + ((flags & DR_BIAS) ? cout * 4.0 : 0.0);
    n->ops.push_back(op);
    return out;
}

static int add_simple(dr_net* n, OpKind kind, const std::string& name, int in0, int in1 = -2, int pool_pad = 1) {
    const Tensor ti = n->T(in0);
    Op op;
    op.kind = kind; op.name = name; op.in0 = in0; op.in1 = in1; op.pool_pad = pool_pad;
    int H = ti.H, W = ti.W;
    if (kind == OP_MAXPOOL) { H = out_size(H, 3, 2, pool_pad); W = out_size(W, 3, 2, pool_pad); }
    if (kind == OP_AVGPOOL) { H = 1; W = 1; }
    op.out = n->tensor(ti.B, H, W, ti.C);
    op.bytes = (double)ti.bytes * (kind == OP_ADD ? 2 : 1) + (double)n->T(op.out).bytes;
    n->ops.push_back(op);
    return op.out;
}

static int add_norm(dr_net* n, OpKind kind, const std::string& name, int in, int v0, int v1) {
    const int out = add_simple(n, kind, name, in);
    n->ops.back().v0.raw = v0; n->ops.back().v1.raw = v1; n->ops.back().eps = n->eps;
    return out;
}

static PRef rawref(int idx) { PRef r; r.raw = idx; return r; }
static PRef wsref(size_t off) { PRef r; r.ws_off = off; return r; }

// A k x k / stride s convolution over a few-channel image (s >= 2, s*s*C <= 64) as a space-to-depth copy of the
// image (a non-tensor layer of its own: one more pass over the input) followed by a ceil(k/s)^2 / stride 1
// convolution over 64 channels with re-laid filters: the form the TMA tensor-core kernel takes.
static int add_conv_s2d(dr_net* n, const std::string& name, int in, int k, int s, int p, int cout, unsigned flags, int wi, PRef b) {
    const Tensor ti = n->T(in);
    const int kp = (k + s - 1) / s, Cp = 64;
    const int Ho = out_size(ti.H, k, s, p), Wo = out_size(ti.W, k, s, p);
    Op op;
    op.kind = OP_S2D; op.name = name + ".s2d"; op.in0 = in;
    op.s2d_k = k; op.s2d_s = s; op.s2d_pad = p;
    op.out = n->tensor(ti.B, Ho + kp - 1, Wo + kp - 1, Cp);
    op.bytes = (double)ti.bytes + (double)n->T(op.out).bytes;
    n->ops.push_back(op);
    const size_t wo = n->ws_alloc((size_t)cout * kp * kp * Cp * 2);
    n->s2d_jobs.push_back({wi, cout, k, ti.C, s, Cp, wo});
    const int out = add_conv(n, name, op.out, kp, 1, 0, cout, flags, wsref(wo), b);
    Op& c = n->ops.back();                      // algorithmic work and bytes of the original convolution
    c.flops = 2.0 * (double)ti.B * Ho * Wo * cout * k * k * ti.C;
    c.bytes += (double)cout * k * k * ti.C * 2 - (double)cout * kp * kp * Cp * 2;
    return out;
}

static void add_concat(dr_net* n, const std::string& name, int in, int out, int coff) {
    Op op;
    op.kind = OP_CONCAT; op.name = name; op.in0 = in; op.out = out; op.coff = coff;
    op.bytes = 2.0 * (double)n->T(in).bytes;
    n->ops.push_back(op);
}


static const unsigned BR = DR_BIAS | DR_RELU;

// Inception-v1 channel table: (Cin; c1, c3r, c3, c5r, c5, pp).  c5r belongs to the original
// 4-branch module and is unused by the branch-slimmed form.
struct Inc { const char* name; int cin, c1, c3r, c3, c5r, c5, pp; };
static const Inc kInception[9] = {
    {"3a", 192, 64, 96, 128, 16, 32, 32},   {"3b", 256, 128, 128, 192, 32, 96, 64},
    {"4a", 480, 192, 96, 208, 16, 48, 64},  {"4b", 512, 160, 112, 224, 24, 64, 64},
    {"4c", 512, 128, 128, 256, 24, 64, 64}, {"4d", 512, 112, 144, 288, 32, 64, 64},
    {"4e", 528, 256, 160, 320, 32, 128, 128}, {"5a", 832, 256, 160, 320, 32, 128, 128},
    {"5b", 832, 384, 192, 384, 48, 128, 128}};

// arch DR_ARCH_GOOGLENET_STREAMLINE: the stem in the approximate form of Section 3.1 (Method): a pooling layer is
// dropped and its stride multiplied into the convolution below it (conv1 7x7/4, conv2 3x3/2), an LRN layer is pruned.
static void build_googlenet(dr_net* n) {
    const bool slim = n->mode == DR_MODE_SLIM;
    const bool streamline = n->arch == DR_ARCH_GOOGLENET_STREAMLINE;
    const int x = n->tensor(n->B, n->H, n->W, 3, 0, true);
    n->t_input = x;
    auto conv_p = [&](const std::string& name, int cout, int k, int cin, PRef* w, PRef* b) {
        *w = rawref(n->filt(name, cout, k, cin));
        *b = rawref(n->vec(name + ".b", cout));
    };
    PRef w, b;
    int t;
    // conv1: 7x7/2 -> ReLU -> pool -> LRN
    conv_p("conv1", 64, 7, 3, &w, &b);
    if (streamline) {
        if (slim) t = add_conv_s2d(n, "conv1", x, 7, 4, 3, 64, BR, w.raw, b);
        else { t = add_conv_s2d(n, "conv1.conv", x, 7, 4, 3, 64, DR_BIAS, w.raw, b); t = add_simple(n, OP_RELU, "conv1", t); }
    } else if (slim) {
        t = add_conv(n, "conv1", x, 7, 2, 3, 64, BR | DR_POOL | DR_LRN, w, b);
    } else {
        t = add_conv_s2d(n, "conv1.conv", x, 7, 2, 3, 64, DR_BIAS, w.raw, b);   // a layer of its own has no pooling to fuse: the tensor-core form of a 3-channel strided conv
        t = add_simple(n, OP_RELU, "conv1.relu", t);
        t = add_simple(n, OP_MAXPOOL, "conv1.pool", t);
        t = add_simple(n, OP_LRN, "conv1", t);
    }
    // conv2 reduce 1x1, conv2 3x3 -> ReLU -> LRN -> pool (the order of Section 3.1's example)
    conv_p("conv2r", 64, 1, 64, &w, &b);
    if (slim) t = add_conv(n, "conv2r", t, 1, 1, 0, 64, BR, w, b);
    else { t = add_conv(n, "conv2r.conv", t, 1, 1, 0, 64, DR_BIAS, w, b); t = add_simple(n, OP_RELU, "conv2r", t); }
    conv_p("conv2", 192, 3, 64, &w, &b);
    if (streamline) {
        if (slim) t = add_conv(n, "conv2", t, 3, 2, 1, 192, BR, w, b);
        else { t = add_conv(n, "conv2.conv", t, 3, 2, 1, 192, DR_BIAS, w, b); t = add_simple(n, OP_RELU, "conv2", t); }
    } else if (slim) {
        t = add_conv(n, "conv2", t, 3, 1, 1, 192, BR | DR_POOL | DR_LRN | DR_LRN_BEFORE_POOL, w, b);
    } else {
        t = add_conv(n, "conv2.conv", t, 3, 1, 1, 192, DR_BIAS, w, b);
        t = add_simple(n, OP_RELU, "conv2.relu", t);
        t = add_simple(n, OP_LRN, "conv2.lrn", t);
        t = add_simple(n, OP_MAXPOOL, "conv2", t);
    }
    for (const Inc& m : kInception) {
        const std::string mn = m.name;
        const Tensor ti = n->T(t);
        const int cm = m.c1 + m.c5 + m.pp;
        PRef w3r, b3r, w3, b3, w1, b1, w5, b5, wp, bp;
        conv_p(mn + ".3x3r", m.c3r, 1, m.cin, &w3r, &b3r);
        conv_p(mn + ".3x3", m.c3, 3, m.c3r, &w3, &b3);
        conv_p(mn + ".b1", m.c1, 1, m.cin, &w1, &b1);
        conv_p(mn + ".b5", m.c5, 5, m.cin, &w5, &b5);
        conv_p(mn + ".bp", m.pp, 3, m.cin, &wp, &bp);
        const int out = n->tensor(ti.B, ti.H, ti.W, m.c3 + cm);
        if (slim) {
            // merged 5x5 filter bank [c1 | c5 | pp] and bias, derived in dr_net_prepare
            const size_t wm = n->ws_alloc((size_t)cm * 25 * m.cin * 2), bm = n->ws_alloc((size_t)cm * 4);
            n->embeds.push_back({w1.raw, m.c1, m.cin, 1, 5, 0, wm});
            n->embeds.push_back({w5.raw, m.c5, m.cin, 5, 5, m.c1, wm});
            n->embeds.push_back({wp.raw, m.pp, m.cin, 3, 5, m.c1 + m.c5, wm});
            n->copies.push_back({b1.raw, bm, (size_t)m.c1 * 4});
            n->copies.push_back({b5.raw, bm + (size_t)m.c1 * 4, (size_t)m.c5 * 4});
            n->copies.push_back({bp.raw, bm + (size_t)(m.c1 + m.c5) * 4, (size_t)m.pp * 4});
            const int r = add_conv(n, mn + ".3x3r", t, 1, 1, 0, m.c3r, BR, w3r, b3r);
            const size_t i_reducer = n->ops.size() - 1;
            add_conv(n, mn + ".3x3", r, 3, 1, 1, m.c3, BR, w3, b3, out, 0);
            add_conv(n, mn + ".m5", t, 5, 1, 2, cm, BR, wsref(wm), wsref(bm), out, m.c3);
            // the reducer and the merged branch read the same tensor and write different ones: at small batch they
            // may go out as one launch
            n->ops[i_reducer].pair = (int)n->ops.size() - 1;
            n->ops[i_reducer].chain = (int)i_reducer + 1;
        } else {
            int r = add_conv(n, mn + ".3x3r.conv", t, 1, 1, 0, m.c3r, DR_BIAS, w3r, b3r);
            r = add_simple(n, OP_RELU, mn + ".3x3r", r);
            int a = add_conv(n, mn + ".3x3.conv", r, 3, 1, 1, m.c3, DR_BIAS, w3, b3);
            a = add_simple(n, OP_RELU, mn + ".3x3", a);
            int c1 = add_conv(n, mn + ".b1.conv", t, 1, 1, 0, m.c1, DR_BIAS, w1, b1);
            c1 = add_simple(n, OP_RELU, mn + ".b1", c1);
            int c5 = add_conv(n, mn + ".b5.conv", t, 5, 1, 2, m.c5, DR_BIAS, w5, b5);
            c5 = add_simple(n, OP_RELU, mn + ".b5", c5);
            int cp = add_conv(n, mn + ".bp.conv", t, 3, 1, 1, m.pp, DR_BIAS, wp, bp);
            cp = add_simple(n, OP_RELU, mn + ".bp", cp);
            add_concat(n, mn + ".cat0", a, out, 0);
            add_concat(n, mn + ".cat1", c1, out, m.c3);
            add_concat(n, mn + ".cat2", c5, out, m.c3 + m.c1);
            add_concat(n, mn + ".cat3", cp, out, m.c3 + m.c1 + m.c5);
        }
        t = out;
        if (mn == "3b") t = add_simple(n, OP_MAXPOOL, "pool3", t);
        if (mn == "4e") t = add_simple(n, OP_MAXPOOL, "pool4", t);
    }
    t = add_simple(n, OP_AVGPOOL, "avgpool", t);
    conv_p("fc", 1000, 1, 1024, &w, &b);
    n->t_logits = add_conv(n, "fc", t, 1, 1, 0, 1000, DR_BIAS | DR_OUT_F32, w, b);
}

// GoogLeNet with the paper's own branch slimming (Section 3.2): per module the 3x3 reducer is halved
// ("branch reducing"), the 1x1 branch is absorbed into the 3x3 convolution, whose output widens from c3 to
// c3 + c1 ("tensor-branch slimming"), and the pooling branch is absorbed into the 5x5 convolution, which keeps
// its reducer and widens from c5 to c5 + pp.  Two branches instead of four, same output width.  The paper
// re-trains these layers; here they carry random weights and the unslimmed mode runs the same two-branch
// topology with every ReLU / concat as its own launch.
static void build_googlenet_paper(dr_net* n) {
    const bool slim = n->mode == DR_MODE_SLIM;
    const int x = n->tensor(n->B, n->H, n->W, 3, 0, true);
    n->t_input = x;
    auto conv_p = [&](const std::string& name, int cout, int k, int cin, PRef* w, PRef* b) {
        *w = rawref(n->filt(name, cout, k, cin));
        *b = rawref(n->vec(name + ".b", cout));
    };
    // `cin` is the layer's own input width; the tensor `in` may carry more channels (zeros, see `reducer`), in which
    // case the filters get zero taps for them.  `cpad` > cout adds output channels with zero filters and zero bias,
    // which stay zero through the ReLU.  Work and bytes are counted for the layer as the paper defines it.
    auto cr = [&](const std::string& name, int in, int cin, int k, int pad, int cout, int cpad, int out = -2, int coff = 0) {
        PRef w, b;
        conv_p(name, cout, k, cin, &w, &b);
        const int cin_t = n->T(in).C;
        if (cin_t != cin || cpad != cout) {
            const size_t wo = n->ws_alloc((size_t)cpad * k * k * cin_t * 2), bo = n->ws_alloc((size_t)cpad * 4);
            n->pad_jobs.push_back({w.raw, wo, (size_t)cpad * k * k * cin_t * 2, (size_t)cout * k * k, (size_t)cin * 2, (size_t)cin_t * 2});
            n->pad_jobs.push_back({b.raw, bo, (size_t)cpad * 4, 1, (size_t)cout * 4, (size_t)cpad * 4});
            w = wsref(wo); b = wsref(bo);
        }
        const size_t first = n->ops.size();
        int r;
        if (slim) {
            r = add_conv(n, name, in, k, 1, pad, cpad, BR, w, b, out, coff);
        } else {
            const int t = add_conv(n, name + ".conv", in, k, 1, pad, cpad, DR_BIAS, w, b);
            r = add_simple(n, OP_RELU, name, t);
            if (out != -2) { add_concat(n, name + ".cat", r, out, coff); r = out; }
        }
        Op& c = n->ops[first];
        const Tensor& ti = n->T(in);
        const double M = (double)ti.B * ti.H * ti.W;
        c.flops = 2.0 * M * cout * k * k * cin;
        c.bytes = M * cin * 2 + (double)cout * k * k * cin * 2 + M * cout * 2 + cout * 4.0;
        return r;
    };
    // Reducers feed a spatial convolution whose tensor-core kernel takes input channels in blocks of 64: their
    // output tensor is rounded up to that, the extra channels zero.
    auto pad64 = [](int c) { return (c + 63) / 64 * 64; };
    PRef w, b;
    int t;
    conv_p("conv1", 64, 7, 3, &w, &b);
    if (slim) {
        t = add_conv(n, "conv1", x, 7, 2, 3, 64, BR | DR_POOL | DR_LRN, w, b);
    } else {
        t = add_conv_s2d(n, "conv1.conv", x, 7, 2, 3, 64, DR_BIAS, w.raw, b);   // a layer of its own has no pooling to fuse: the tensor-core form of a 3-channel strided conv
        t = add_simple(n, OP_RELU, "conv1.relu", t);
        t = add_simple(n, OP_MAXPOOL, "conv1.pool", t);
        t = add_simple(n, OP_LRN, "conv1", t);
    }
    t = cr("conv2r", t, 64, 1, 0, 64, 64);
    conv_p("conv2", 192, 3, 64, &w, &b);
    if (slim) {
        t = add_conv(n, "conv2", t, 3, 1, 1, 192, BR | DR_POOL | DR_LRN | DR_LRN_BEFORE_POOL, w, b);
    } else {
        t = add_conv(n, "conv2.conv", t, 3, 1, 1, 192, DR_BIAS, w, b);
        t = add_simple(n, OP_RELU, "conv2.relu", t);
        t = add_simple(n, OP_LRN, "conv2.lrn", t);
        t = add_simple(n, OP_MAXPOOL, "conv2", t);
    }
    for (const Inc& m : kInception) {
        const std::string mn = m.name;
        const Tensor ti = n->T(t);
        const int a3 = m.c3 + m.c1, a5 = m.c5 + m.pp;
        const int out = n->tensor(ti.B, ti.H, ti.W, a3 + a5);
        const int r3 = cr(mn + ".p3r", t, ti.C, 1, 0, m.c3r / 2, pad64(m.c3r / 2));
        cr(mn + ".p3", r3, m.c3r / 2, 3, 1, a3, a3, out, 0);
        const int r5 = cr(mn + ".p5r", t, ti.C, 1, 0, m.c5r, pad64(m.c5r));
        cr(mn + ".p5", r5, m.c5r, 5, 2, a5, a5, out, a3);
        t = out;
        if (mn == "3b") t = add_simple(n, OP_MAXPOOL, "pool3", t);
        if (mn == "4e") t = add_simple(n, OP_MAXPOOL, "pool4", t);
    }
    t = add_simple(n, OP_AVGPOOL, "avgpool", t);
    conv_p("fc", 1000, 1, 1024, &w, &b);
    n->t_logits = add_conv(n, "fc", t, 1, 1, 0, 1000, DR_BIAS | DR_OUT_F32, w, b);
}

static void build_resnet50(dr_net* n) {
    const bool slim = n->mode == DR_MODE_SLIM;
    const int x = n->tensor(n->B, n->H, n->W, 3, 0, true);
    n->t_input = x;
    // conv -> BatchNorm -> Scale [-> ReLU] [-> pool]; slim: one conv with folded parameters
    auto cbs = [&](const std::string& name, int in, int k, int s, int p, int cout, bool relu, bool pool, int residual) {
        const int cin = n->T(in).C;
        const int wi = n->filt(name, cout, k, cin);
        const int mean = n->vec(name + ".bn.mean", cout), var = n->vec(name + ".bn.var", cout);
        const int gamma = n->vec(name + ".bn.gamma", cout), beta = n->vec(name + ".bn.beta", cout);
        if (slim) {
            const size_t wo = n->ws_alloc((size_t)cout * k * k * cin * 2), bo = n->ws_alloc((size_t)cout * 4);
            n->folds.push_back({wi, mean, var, gamma, beta, wo, bo, cout, k * k * cin});
            unsigned f = DR_BIAS;
            if (residual != -2) f |= DR_RESIDUAL | (relu ? DR_RELU_AFTER_RESIDUAL : 0);
            else if (relu) f |= DR_RELU;
            if (pool) f |= DR_POOL;
            return add_conv(n, name, in, k, s, p, cout, f, wsref(wo), wsref(bo), -2, 0, residual);
        }
        int t = (s >= 2 && s * s * cin <= 64) ? add_conv_s2d(n, name + ".conv", in, k, s, p, cout, 0, wi, PRef())
                                              : add_conv(n, name + ".conv", in, k, s, p, cout, 0, rawref(wi), PRef());
        t = add_norm(n, OP_BN, name + ".bn", t, mean, var);
        const bool last = !relu && !pool && residual == -2;
        t = add_norm(n, OP_SCALE, last ? name : name + ".scale", t, gamma, beta);
        if (residual != -2) t = add_simple(n, OP_ADD, relu ? name + ".add" : name, t, residual);
        if (relu) t = add_simple(n, OP_RELU, pool ? name + ".relu" : name, t);
        if (pool) t = add_simple(n, OP_MAXPOOL, name, t);
        return t;
    };
    int t = cbs("conv1", x, 7, 2, 3, 64, true, true, -2);
    static const int widths[4] = {64, 128, 256, 512}, blocks[4] = {3, 4, 6, 3};
    for (int si = 0; si < 4; ++si)
        for (int bi = 0; bi < blocks[si]; ++bi) {
            const std::string blk = "res" + std::to_string(si + 2) + std::string(1, (char)('a' + bi));
            const int w = widths[si];
            const int s = (bi == 0 && si > 0) ? 2 : 1;   // stride on the first 1x1 and on the projection
            int res = t;
            if (bi == 0) res = cbs(blk + ".br1", t, 1, s, 0, 4 * w, false, false, -2);
            int u = cbs(blk + ".2a", t, 1, s, 0, w, true, false, -2);
            u = cbs(blk + ".2b", u, 3, 1, 1, w, true, false, -2);
            t = cbs(blk + ".2c", u, 1, 1, 0, 4 * w, true, false, res);
        }
    t = add_simple(n, OP_AVGPOOL, "avgpool", t);
    const int wi = n->filt("fc", 1000, 1, 2048), bi = n->vec("fc.b", 1000);
    n->t_logits = add_conv(n, "fc", t, 1, 1, 0, 1000, DR_BIAS | DR_OUT_F32, rawref(wi), rawref(bi));
}

// Split-K scratch of the workspace: [parameters][activation arena][scratch][counters, one block per convolution]
static size_t sk_region_bytes(const dr_net* n) {
    return n->sk_scratch_bytes ? (n->sk_scratch_bytes + 255) / 256 * 256 + (size_t)n->n_conv * DR_CONV_WS_COUNTER_BYTES : 0;
}
static void set_splitk_scratch(const dr_net* n, const Op& op, char* ws, ConvParams* p) {
    if (!n->sk_scratch_bytes || n->mode != DR_MODE_SLIM) return;
    char* base = ws + n->param_bytes + n->act_bytes;
    p->sk_scratch = reinterpret_cast<float*>(base);
    p->sk_scratch_bytes = n->sk_scratch_bytes;
    p->sk_counters = reinterpret_cast<int*>(base + (n->sk_scratch_bytes + 255) / 256 * 256 + (size_t)op.conv_index * DR_CONV_WS_COUNTER_BYTES);
}

// AlexNet (two-tower form, 227x227 input).  Slim layers (Section 4.3): conv1 = conv + ReLU + LRN, conv2 = grouped
// conv + ReLU + LRN; the unpadded 3x3/2 pools stay separate, as in the paper's table.  Grouped layers run as dense
// convolutions over block-diagonal filters (dr_embed_groups) in both modes; fc6 is a 6x6 convolution over the 6x6
// plane pool5 leaves.  Dropout is the identity at inference.
static void build_alexnet(dr_net* n) {
    const bool slim = n->mode == DR_MODE_SLIM;
    const int x = n->tensor(n->B, n->H, n->W, 3, 0, true);
    n->t_input = x;
    struct L { const char* name; int cout, k, s, p, groups; bool lrn, pool, relu; };
    static const L layers[8] = {{"conv1", 96, 11, 4, 0, 1, true, true, true},   {"conv2", 256, 5, 1, 2, 2, true, true, true},
                                {"conv3", 384, 3, 1, 1, 1, false, false, true}, {"conv4", 384, 3, 1, 1, 2, false, false, true},
                                {"conv5", 256, 3, 1, 1, 2, false, true, true},  {"fc6", 4096, 6, 1, 0, 1, false, false, true},
                                {"fc7", 4096, 1, 1, 0, 1, false, false, true},  {"fc8", 1000, 1, 1, 0, 1, false, false, false}};
    int t = x;
    for (int i = 0; i < 8; ++i) {
        const L& l = layers[i];
        const std::string name = l.name;
        const int cin = n->T(t).C;
        const int wi = n->param(name + ".w", l.cout, l.k, l.k, cin / l.groups, 0);
        const int bi = n->vec(name + ".b", l.cout);
        PRef w = rawref(wi);
        if (l.groups > 1) {
            const size_t wo = n->ws_alloc((size_t)l.cout * l.k * l.k * cin * 2);
            n->group_jobs.push_back({wi, l.cout, cin / l.groups, l.k, l.groups, wo});
            w = wsref(wo);
        }
        const bool last = i == 7;
        const char* pool_name = i == 0 ? "pool1" : i == 1 ? "pool2" : "pool5";
        const bool s2d = l.s >= 2 && l.s * l.s * cin <= 64;      // conv1: 11x11/4 over 3 channels
        if (slim) {
            unsigned f = DR_BIAS | (l.relu ? DR_RELU : 0) | (l.lrn ? DR_LRN : 0) | (last ? DR_OUT_F32 : 0);
            if (s2d) t = add_conv_s2d(n, name, t, l.k, l.s, l.p, l.cout, f, wi, rawref(bi));
            else t = add_conv(n, name, t, l.k, l.s, l.p, l.cout, f, w, rawref(bi));
            n->ops.back().flops /= l.groups;        // algorithmic work of the grouped layer, not of its dense stand-in
        } else {
            const bool plain = !l.relu && !l.lrn;
            const unsigned f = DR_BIAS | (last ? DR_OUT_F32 : 0);
            if (s2d) t = add_conv_s2d(n, plain ? name : name + ".conv", t, l.k, l.s, l.p, l.cout, f, wi, rawref(bi));
            else t = add_conv(n, plain ? name : name + ".conv", t, l.k, l.s, l.p, l.cout, f, w, rawref(bi));
            n->ops.back().flops /= l.groups;
            if (l.relu) t = add_simple(n, OP_RELU, l.lrn ? name + ".relu" : name, t);
            if (l.lrn) t = add_simple(n, OP_LRN, name, t);
        }
        if (l.pool) t = add_simple(n, OP_MAXPOOL, pool_name, t, -2, 0);
        if (last) n->t_logits = t;
    }
}

static const char* tensor_ptr(const dr_net* n, int id, const void* x, const char* arena, const float* logits) {
    if (id == n->t_input) return (const char*)x;
    if (id == n->t_logits) return (const char*)logits;
    return arena + n->T(id).off;
}

}  // namespace dr

extern "C" {

int dr_net_create(dr_net** net, int arch, int mode, int B, int H, int W) {
    if (!net || B <= 0 || H <= 0 || W <= 0) return DR_ERR_INVALID_ARG;
    if (arch < DR_ARCH_GOOGLENET || arch > DR_ARCH_ALEXNET) return DR_ERR_INVALID_ARG;
    if (arch == DR_ARCH_ALEXNET && (H != 227 || W != 227)) return DR_ERR_INVALID_ARG;   // fc6 is a 6x6 convolution over pool5's 6x6 plane
    if (mode != DR_MODE_SLIM && mode != DR_MODE_UNSLIMMED) return DR_ERR_INVALID_ARG;
    // five halvings (stem conv, four pools / strided stages) must leave at least one pixel
    if (H < 32 || W < 32) return DR_ERR_INVALID_ARG;
    dr_net* n = new dr_net();
    n->arch = arch; n->mode = mode; n->B = B; n->H = H; n->W = W;
    if (arch == DR_ARCH_GOOGLENET || arch == DR_ARCH_GOOGLENET_STREAMLINE) build_googlenet(n);
    else if (arch == DR_ARCH_GOOGLENET_PAPER) build_googlenet_paper(n);
    else if (arch == DR_ARCH_ALEXNET) build_alexnet(n);
    else build_resnet50(n);
    // scratch the split-K kernel wants for the layers with few output tiles (slim mode only: the unslimmed
    // baseline keeps one plain launch per layer)
    if (mode == DR_MODE_SLIM)
        for (const Op& op : n->ops) {
            if (op.kind != OP_CONV) continue;
            const Tensor& ti = n->T(op.in0);
            ConvParams p;
            const void* dummy = reinterpret_cast<const void*>(uintptr_t(256));
            if (conv_make_params(&op.cd, ti.B, ti.H, ti.W, dummy, dummy, (const float*)dummy, dummy, (void*)dummy, nullptr, &p) != DR_OK) continue;
            size_t need = conv_splitk_scratch_bytes(p);
            if (op.pair >= 0) {
                const Op& oa = n->ops[op.pair];
                const Op& oc = n->ops[op.chain];
                ConvParams pa, pc;
                if (conv_make_params(&oa.cd, ti.B, ti.H, ti.W, dummy, dummy, (const float*)dummy, dummy, (void*)dummy, nullptr, &pa) == DR_OK &&
                    conv_make_params(&oc.cd, ti.B, ti.H, ti.W, dummy, dummy, (const float*)dummy, dummy, (void*)dummy, nullptr, &pc) == DR_OK) {
                    const size_t two = conv_splitk_group_scratch_bytes(pa, p, nullptr), three = conv_splitk_group_scratch_bytes(pa, p, &pc);
                    if (two > need) need = two;
                    if (three > need) need = three;
                }
            }
            if (need > n->sk_scratch_bytes) n->sk_scratch_bytes = need;
        }
    *net = n;
    return DR_OK;
}

int dr_net_destroy(dr_net* n) {
    if (!n) return DR_ERR_INVALID_ARG;
    for (cudaEvent_t e : n->ev) cudaEventDestroy(e);
    delete n;
    return DR_OK;
}

int dr_net_num_params(const dr_net* n) { return n ? (int)n->specs.size() : DR_ERR_INVALID_ARG; }

int dr_net_param_spec(const dr_net* n, int idx, dr_param_spec* spec) {
    if (!n || !spec || idx < 0 || idx >= (int)n->specs.size()) return DR_ERR_INVALID_ARG;
    *spec = n->specs[idx];
    return DR_OK;
}

int dr_net_set_param(dr_net* n, int idx, const void* dev) {
    if (!n || !dev || idx < 0 || idx >= (int)n->specs.size()) return DR_ERR_INVALID_ARG;
    if (!aligned16(dev)) return DR_ERR_ALIGNMENT;
    n->raw[idx] = dev;
    n->prepared_ws = nullptr;
    return DR_OK;
}

int dr_net_workspace_bytes(const dr_net* n, size_t* bytes) {
    if (!n || !bytes) return DR_ERR_INVALID_ARG;
    *bytes = n->param_bytes + n->act_bytes + sk_region_bytes(n) + 256;
    return DR_OK;
}

int dr_net_activation_bytes(const dr_net* n, size_t* bytes) {
    if (!n || !bytes) return DR_ERR_INVALID_ARG;
    *bytes = n->act_bytes;
    return DR_OK;
}

int dr_net_prepare(dr_net* n, void* workspace, void* stream) {
    if (!n) return DR_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255)) return DR_ERR_WORKSPACE;
    for (const void* p : n->raw)
        if (!p) return DR_ERR_INVALID_ARG;
    char* ws = (char*)workspace;
    cudaStream_t s = (cudaStream_t)stream;
    for (const FoldJob& f : n->folds) {
        const int st = dr_fold_bn(f.Cout, f.K, n->raw[f.w], nullptr, (const float*)n->raw[f.mean], (const float*)n->raw[f.var],
                                  1.f, n->eps, (const float*)n->raw[f.gamma], (const float*)n->raw[f.beta], ws + f.w_off,
                                  (float*)(ws + f.b_off), stream);
        if (st != DR_OK) return st;
    }
    for (const EmbedJob& e : n->embeds) {
        const int st = dr_embed_filter(e.Cout, e.Cin, e.ks, e.kb, n->raw[e.w_small], e.joff, ws + e.w_off, stream);
        if (st != DR_OK) return st;
    }
    for (const S2dJob& j : n->s2d_jobs) {
        const int st = dr_s2d_filter(j.Cout, j.k, j.C, j.s, j.Cp, n->raw[j.w], ws + j.w_off, stream);
        if (st != DR_OK) return st;
    }
    for (const GroupJob& g : n->group_jobs) {
        const int st = dr_embed_groups(g.Cout, g.Cin_g, g.k, g.groups, n->raw[g.w_grouped], ws + g.w_off, stream);
        if (st != DR_OK) return st;
    }
    for (const PadJob& j : n->pad_jobs) {
        if (cudaMemsetAsync(ws + j.dst_off, 0, j.total, s) != cudaSuccess) return DR_ERR_CUDA;
        if (cudaMemcpy2DAsync(ws + j.dst_off, j.pitch, n->raw[j.src], j.row_bytes, j.row_bytes, j.rows, cudaMemcpyDeviceToDevice, s) !=
            cudaSuccess)
            return DR_ERR_CUDA;
    }
    for (const CopyJob& c : n->copies)
        if (cudaMemcpyAsync(ws + c.dst_off, n->raw[c.src], c.bytes, cudaMemcpyDeviceToDevice, s) != cudaSuccess) return DR_ERR_CUDA;
    if (n->sk_scratch_bytes && n->mode == DR_MODE_SLIM) {   // tile counters start at zero; the kernels leave them at zero
        char* counters = ws + n->param_bytes + n->act_bytes + (n->sk_scratch_bytes + 255) / 256 * 256;
        if (cudaMemsetAsync(counters, 0, (size_t)n->n_conv * DR_CONV_WS_COUNTER_BYTES, s) != cudaSuccess) return DR_ERR_CUDA;
    }
    // decide the kernel of every convolution once
    const char* arena = ws + n->param_bytes;
    for (Op& op : n->ops) {
        if (op.kind != OP_CONV) continue;
        const Tensor& ti = n->T(op.in0);
        ConvParams p;
        const char* dummy = arena;   // addresses only need to be aligned for validation here
        const int st = conv_make_params(&op.cd, ti.B, ti.H, ti.W, dummy, dummy, (const float*)dummy, dummy, (void*)dummy, nullptr, &p);
        if (st != DR_OK) return st;
        set_splitk_scratch(n, op, ws, &p);
        op.path = conv_pick_path(p, forced_conv_path());
        if (op.path < 0) return DR_ERR_UNSUPPORTED;
    }
    for (Op& op : n->ops) {
        op.group = 0;
        if (op.kind != OP_CONV || op.pair < 0 || forced_conv_path() != DR_PATH_AUTO) continue;
        const Op& oa = n->ops[op.pair];
        const Op& oc = n->ops[op.chain];
        const Tensor& ti = n->T(op.in0);
        ConvParams pa, pb, pc;
        const char* dummy = arena;
        if (conv_make_params(&oa.cd, ti.B, ti.H, ti.W, dummy, dummy, (const float*)dummy, dummy, (void*)dummy, nullptr, &pa) != DR_OK) continue;
        if (conv_make_params(&op.cd, ti.B, ti.H, ti.W, dummy, dummy, (const float*)dummy, dummy, (void*)dummy, nullptr, &pb) != DR_OK) continue;
        if (conv_make_params(&oc.cd, ti.B, ti.H, ti.W, dummy, dummy, (const float*)dummy, dummy, (void*)dummy, nullptr, &pc) != DR_OK) continue;
        set_splitk_scratch(n, oa, ws, &pa);
        if (oa.path != DR_PATH_UMMA_SPLITK) continue;
        if (conv_splitk_group_supports(pa, pb, &pc)) op.group = 3;
        else if (conv_splitk_group_supports(pa, pb, nullptr)) op.group = 2;
    }
    n->prepared_ws = workspace;
    return DR_OK;
}

int dr_net_forward(dr_net* n, const void* x, void* workspace, float* logits, void* stream) {
    if (!n || !x || !logits) return DR_ERR_INVALID_ARG;
    if (!workspace || workspace != n->prepared_ws) return DR_ERR_WORKSPACE;
    if (!aligned16(x) || !aligned16(logits)) return DR_ERR_ALIGNMENT;
    const char* ws = (const char*)workspace;
    char* arena = (char*)workspace + n->param_bytes;
    cudaStream_t s = (cudaStream_t)stream;
    if (n->timing && n->ev.size() != 2 * n->ops.size()) {
        for (cudaEvent_t e : n->ev) cudaEventDestroy(e);
        n->ev.assign(2 * n->ops.size(), nullptr);
        for (auto& e : n->ev)
            if (cudaEventCreate(&e) != cudaSuccess) return DR_ERR_CUDA;
    }
    n->done.assign(n->ops.size(), 0);
    for (size_t i = 0; i < n->ops.size(); ++i) {
        if (n->done[i]) continue;              // went out together with an earlier layer
        const Op& op = n->ops[i];
        const Tensor& ti = n->T(op.in0);
        const Tensor& to = n->T(op.out);
        const char* in0 = tensor_ptr(n, op.in0, x, arena, logits);
        const char* in1 = op.in1 >= -1 ? tensor_ptr(n, op.in1, x, arena, logits) : nullptr;
        char* out = (char*)tensor_ptr(n, op.out, x, arena, logits);
        if (n->timing && cudaEventRecord(n->ev[2 * i], s) != cudaSuccess) return DR_ERR_CUDA;
        int st = DR_OK;
        switch (op.kind) {
            case OP_CONV: {
                ConvParams p;
                st = conv_make_params(&op.cd, ti.B, ti.H, ti.W, in0, op.w.resolve(n->raw, ws), (const float*)op.b.resolve(n->raw, ws),
                                      (op.cd.flags & DR_RESIDUAL) ? in1 : nullptr, out, nullptr, &p);
                if (st == DR_OK && op.group && !n->timing) {
                    // this layer, the later one that reads the same input and (group 3) the one that reads this layer's
                    // output, as one launch (per-layer timing keeps them apart)
                    const Op& oa = n->ops[op.pair];
                    const Op& oc = n->ops[op.chain];
                    ConvParams pa, pc;
                    st = conv_make_params(&oa.cd, ti.B, ti.H, ti.W, in0, oa.w.resolve(n->raw, ws), (const float*)oa.b.resolve(n->raw, ws),
                                          nullptr, (char*)tensor_ptr(n, oa.out, x, arena, logits), nullptr, &pa);
                    if (st == DR_OK && op.group == 3) {
                        const Tensor& tc = n->T(oc.in0);
                        st = conv_make_params(&oc.cd, tc.B, tc.H, tc.W, out, oc.w.resolve(n->raw, ws), (const float*)oc.b.resolve(n->raw, ws),
                                              nullptr, (char*)tensor_ptr(n, oc.out, x, arena, logits), nullptr, &pc);
                    }
                    if (st == DR_OK) {
                        set_splitk_scratch(n, oa, (char*)workspace, &pa);
                        st = conv_splitk_group_launch(pa, p, op.group == 3 ? &pc : nullptr, s);
                        n->done[op.pair] = 1;
                        if (op.group == 3) n->done[op.chain] = 1;
                    }
                    break;
                }
                if (st == DR_OK && op.pair >= 0 && !op.group && !n->timing && op.path == DR_PATH_UMMA_TMA &&
                    n->ops[op.pair].path == DR_PATH_UMMA_TMA && tunable("DR_NET_OVERLAP", 2) != 0) {
                    // Large batch.  DR_NET_OVERLAP = 2 (default): this layer, then the merged 5x5 (which reads the same input),
                    // then the 3x3 that reads this layer's output, launched so that its CTAs fill the SMs the merged 5x5's
                    // last round of tiles leaves idle.  DR_NET_OVERLAP = 1: the merged 5x5 first and this short layer
                    // behind it in that way (measured: 3.99 ms per step without, 3.91 with 1, 3.89 with 2).  The overlapped layer reads nothing the merged 5x5
                    // writes and does not finish before it has.
                    const Op& oa = n->ops[op.pair];
                    const Op& oc = n->ops[op.chain];
                    const int mode = tunable("DR_NET_OVERLAP", 2);
                    ConvParams pa, pc;
                    st = conv_make_params(&oa.cd, ti.B, ti.H, ti.W, in0, oa.w.resolve(n->raw, ws), (const float*)oa.b.resolve(n->raw, ws),
                                          nullptr, (char*)tensor_ptr(n, oa.out, x, arena, logits), nullptr, &pa);
                    if (st == DR_OK && mode == 2 && oc.path == DR_PATH_UMMA_TMA) {
                        const Tensor& tc = n->T(oc.in0);
                        st = conv_make_params(&oc.cd, tc.B, tc.H, tc.W, out, oc.w.resolve(n->raw, ws), (const float*)oc.b.resolve(n->raw, ws),
                                              nullptr, (char*)tensor_ptr(n, oc.out, x, arena, logits), nullptr, &pc);
                        // the reducer may start while the kernel before it drains (it waits before its first load); the merged 5x5
                        // behind it stays an ordinary launch, so that the 3x3, which starts early and reads the reducer's output
                        // without waiting, cannot start before the reducer has completed
                        p.pdl_wait = (i > 0 && tunable("DR_NET_PDL", 1) != 0) ? 1 : 0;
                        if (st == DR_OK) st = conv_launch_path(p, op.path, s);
                        if (st == DR_OK) st = conv_launch_path(pa, oa.path, s);
                        if (st == DR_OK) {
                            pc.overlap_prev = 1;
                            st = conv_launch_path(pc, oc.path, s);
                            n->done[op.pair] = 1;
                            n->done[op.chain] = 1;
                        }
                        break;
                    }
                    if (st == DR_OK) st = conv_launch_path(pa, oa.path, s);
                    if (st == DR_OK) {
                        p.overlap_prev = 1;
                        st = conv_launch_path(p, op.path, s);
                        n->done[op.pair] = 1;
                    }
                    break;
                }
                if (st == DR_OK) {
                    set_splitk_scratch(n, op, (char*)workspace, &p);
                    // a layer of its own on the TMA kernel: its CTAs may set up while the kernel before it drains
                    if ((op.path == DR_PATH_UMMA_TMA || op.path == DR_PATH_UMMA_PATCH) && i > 0 && !n->timing && tunable("DR_NET_PDL", 1) != 0) p.pdl_wait = 1;
                    st = conv_launch_path(p, op.path, s);
                }
                break;
            }
            case OP_RELU: st = dr_relu((size_t)ti.B * ti.H * ti.W * ti.C, in0, out, stream); break;
            case OP_MAXPOOL:
                g_pool_pdl = i > 0 && !n->timing && tunable("DR_NET_PDL", 1) != 0;
                st = dr_maxpool(ti.B, ti.H, ti.W, ti.C, 3, 2, op.pool_pad, in0, out, nullptr, stream);
                g_pool_pdl = false;
                break;
            case OP_LRN: st = dr_lrn(ti.B, ti.H, ti.W, ti.C, 5, 1e-4f, 0.75f, 1.f, in0, out, stream); break;
            case OP_BN:
                st = dr_bn(ti.B, ti.H, ti.W, ti.C, in0, (const float*)op.v0.resolve(n->raw, ws), (const float*)op.v1.resolve(n->raw, ws),
                           1.f, op.eps, nullptr, nullptr, out, stream);
                break;
            case OP_SCALE:
                st = dr_scale(ti.B, ti.H, ti.W, ti.C, in0, (const float*)op.v0.resolve(n->raw, ws), (const float*)op.v1.resolve(n->raw, ws), out, stream);
                break;
            case OP_ADD: st = dr_add((size_t)ti.B * ti.H * ti.W * ti.C, in0, in1, out, stream); break;
            case OP_CONCAT: st = dr_concat((size_t)ti.B * ti.H * ti.W, ti.C, in0, to.C, op.coff, out, stream); break;
            case OP_AVGPOOL:
                g_pool_pdl = i > 0 && !n->timing && tunable("DR_NET_PDL", 1) != 0;
                st = dr_avgpool_global(ti.B, ti.H, ti.W, ti.C, in0, out, stream);
                g_pool_pdl = false;
                break;
            case OP_S2D: st = dr_space_to_depth(ti.B, ti.H, ti.W, ti.C, op.s2d_k, op.s2d_s, op.s2d_pad, to.C, in0, out, stream); break;
        }
        if (st != DR_OK) return st;
        if (n->timing && cudaEventRecord(n->ev[2 * i + 1], s) != cudaSuccess) return DR_ERR_CUDA;
    }
    return DR_OK;
}

int dr_net_num_layers(const dr_net* n) { return n ? (int)n->ops.size() : DR_ERR_INVALID_ARG; }

int dr_net_layer_info(const dr_net* n, int layer, dr_layer_info* info) {
    if (!n || !info || layer < 0 || layer >= (int)n->ops.size()) return DR_ERR_INVALID_ARG;
    const Op& op = n->ops[layer];
    const Tensor& to = n->T(op.out);
    dr_layer_info li{};
    std::strncpy(li.name, op.name.c_str(), sizeof(li.name) - 1);
    li.kind = op.kind == OP_CONV ? 0 : 1;
    li.dims[0] = to.B; li.dims[1] = to.H; li.dims[2] = to.W;
    li.dims[3] = op.kind == OP_CONV ? op.cd.Cout : (op.kind == OP_CONCAT ? n->T(op.in0).C : to.C);
    li.ldc = to.C; li.coff = op.coff; li.is_f32 = to.is_f32;
    li.ptr = nullptr;
    if (n->prepared_ws && to.off != (size_t)-1)
        li.ptr = (const char*)n->prepared_ws + n->param_bytes + to.off + (size_t)op.coff * (to.is_f32 ? 4 : 2);
    li.flops = op.flops; li.bytes = op.bytes; li.conv_path = op.kind == OP_CONV ? op.path : -1;
    *info = li;
    return DR_OK;
}

int dr_net_set_timing(dr_net* n, int enabled) {
    if (!n) return DR_ERR_INVALID_ARG;
    n->timing = enabled != 0;
    return DR_OK;
}

int dr_net_layer_time_us(dr_net* n, int layer, float* us) {
    if (!n || !us || layer < 0 || layer >= (int)n->ops.size()) return DR_ERR_INVALID_ARG;
    if (n->ev.size() != 2 * n->ops.size()) return DR_ERR_INVALID_ARG;
    if (cudaEventSynchronize(n->ev[2 * layer + 1]) != cudaSuccess) return DR_ERR_CUDA;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, n->ev[2 * layer], n->ev[2 * layer + 1]) != cudaSuccess) return DR_ERR_CUDA;
    *us = ms * 1000.f;
    return DR_OK;
}

}  // extern "C"
