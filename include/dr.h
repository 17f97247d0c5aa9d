/*
 * libdeeprebirth — execution of DeepRebirth "slim layers" on NVIDIA B200 (sm_100a).
 *
 * A slim layer is a convolution that has absorbed the non-tensor layers around it
 * (DeepRebirth, Section 3): BatchNorm and Scale are folded into its weights and bias by the
 * closed form of Lemma 2 (Section 3.1, "streamline slimming"); ReLU, max-pooling and
 * cross-channel LRN run in its epilogue instead of as layers of their own; and the parallel
 * branches of an inception module run as one wide convolution that writes its slice of the
 * concatenated output in place (Section 3.2, "branch slimming").  Unlike the paper, which
 * approximates the absorbed pooling/LRN layers and re-trains, the epilogue here computes them
 * exactly, so a slim layer returns what the original layer sequence returns.
 *
 * Conventions
 *  - Plain C ABI.  Every call returns an int status: DR_OK (0) or a negative DR_ERR_* code;
 *    dr_strerror() names it.  Arguments are validated before anything is launched; on an error
 *    nothing has been launched unless the code is DR_ERR_CUDA or DR_ERR_DEVICE_TIMEOUT.
 *  - All tensor pointers are DEVICE pointers owned by the caller, 16-byte aligned, and must
 *    stay valid until the work queued on `stream` has finished.  The library allocates no
 *    device memory: scratch space is sized by a *_workspace_bytes call and passed in.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *    enqueue work; they do not synchronise unless stated.
 *  - Activations are NHWC bfloat16: element (n,h,w,c) of a tensor with channel stride ldc and
 *    channel offset coff lives at ((n*H + h)*W + w)*ldc + coff + c.  Dense tensors have
 *    ldc = C, coff = 0.  Filters are [Cout][k][k][Cin] bfloat16; bias and BatchNorm/Scale
 *    vectors are float32 [Cout].  Accumulation and all epilogue arithmetic are float32;
 *    results are rounded to bfloat16 (nearest even) once, when stored.
 *  - Device-side waits are bounded.  If one runs out, the kernel records
 *    DR_ERR_DEVICE_TIMEOUT, releases what it holds and returns; dr_device_status() reads the
 *    record after a synchronisation.
 */
#ifndef DR_H_
#define DR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------------------ */
#define DR_OK                   0
#define DR_ERR_INVALID_ARG     (-1)  /* null pointer, non-positive size, inconsistent descriptor */
#define DR_ERR_UNSUPPORTED     (-2)  /* a valid request this build has no kernel for            */
#define DR_ERR_ALIGNMENT       (-3)  /* pointer / ldc / coff not aligned as documented          */
#define DR_ERR_WORKSPACE       (-4)  /* workspace missing, too small, or net not prepared       */
#define DR_ERR_CUDA            (-5)  /* a CUDA runtime/driver call failed                       */
#define DR_ERR_DEVICE_TIMEOUT  (-6)  /* a bounded device-side wait ran out                      */

const char* dr_strerror(int status);

/* ---- slim-layer descriptor --------------------------------------------------------- */
/* Epilogue flags.  The epilogue applies, in this order: +bias, ReLU, then pooling and LRN in
 * the order DR_LRN_BEFORE_POOL selects, then +residual, then the second ReLU.              */
#define DR_BIAS                 0x01u
#define DR_RELU                 0x02u
#define DR_POOL                 0x04u  /* max-pool pool_k x pool_k / pool_stride, pad pool_pad   */
#define DR_LRN                  0x08u  /* LRN across channels                                    */
#define DR_RESIDUAL             0x10u  /* add a dense [B,Ho,Wo,Cout] bfloat16 tensor            */
#define DR_LRN_BEFORE_POOL      0x20u  /* LRN then pool (GoogLeNet conv2); default pool then LRN */
#define DR_RELU_AFTER_RESIDUAL  0x40u
#define DR_OUT_F32              0x80u  /* store float32 instead of bfloat16 (final logits)       */

typedef struct dr_conv_desc {
    int k, stride, pad;        /* square kernel; output extent floor((H + 2*pad - k)/stride) + 1 */
    int Cin, Cout;
    unsigned flags;            /* DR_* epilogue flags                                            */
    int pool_k, pool_stride, pool_pad;              /* used with DR_POOL; only 3,2,1 is built    */
    int lrn_size;                                   /* used with DR_LRN; odd, <= 15              */
    float lrn_alpha, lrn_beta, lrn_k;
    int y_ldc, y_coff;         /* channel stride / offset of y; 0,0 means dense (ldc = Cout)     */
} dr_conv_desc;

/* ---- parameter generation (offline slimming) ---------------------------------------- */

/* Lemma 2 / Eq. (W_B_S), Section 3.1: closed form of convolution -> BatchNorm -> Scale.
 *   eta_j = gamma_j / sqrt(var_j/m + eps);  w_out[j,:] = eta_j * w_in[j,:];
 *   b_out[j] = eta_j * b_in[j] + beta_j - eta_j * mean_j / m.
 * mean/var are the stored BatchNorm blobs and m their scale factor (true statistics are
 * mean/m and var/m); eps = 0 reproduces the paper's formula.  K = k*k*Cin values per filter.
 * w_in, w_out: bfloat16 [Cout][K] (may alias).  b_in: float32 [Cout] or NULL (zero bias).
 * Computed in float32, w_out rounded to bfloat16 once.  Errors: INVALID_ARG on nulls/sizes. */
int dr_fold_bn(int Cout, int K, const void* w_in, const float* b_in, const float* mean,
               const float* var, float m, float eps, const float* gamma, const float* beta,
               void* w_out, float* b_out, void* stream);

/* The exact form of "adjust to the same size" in Section 3.2: write a [Cout][ks][ks][Cin]
 * filter bank, zero-embedded at the centre of kb x kb taps, into filters [joff, joff+Cout) of
 * w_big ([*][kb][kb][Cin], bfloat16); with pad kb/2 the stride-1 convolution is unchanged.
 * Concatenating filter banks along Cout is Eq. (W_b).  kb >= ks, both odd.                  */
int dr_embed_filter(int Cout, int Cin, int ks, int kb, const void* w_small, int joff,
                    void* w_big, void* stream);

/* A grouped convolution (AlexNet's two-tower layers, Section 4.3) as the dense convolution it is a special case
 * of: w_grouped [Cout][k][k][Cin_g] (filter j belongs to group j / (Cout/groups) and sees input channels
 * [g*Cin_g, (g+1)*Cin_g)) is written into w_dense [Cout][k][k][Cin_g*groups] with zeros across groups.  The
 * slim layer the paper generates for such a layer is an ordinary convolution layer; the convolution kernels
 * never look at the zeros.  Errors: INVALID_ARG (Cout not a multiple of groups, nulls, sizes).               */
int dr_embed_groups(int Cout, int Cin_g, int k, int groups, const void* w_grouped, void* w_dense,
                    void* stream);

/* A strided convolution over few input channels (AlexNet's 11x11/4 and the stride-product 7x7/4 stem of Section 3.1
 * on 3-channel images) as a stride-1 convolution over a space-to-depth copy of the input: with kp = ceil(k/s),
 *   y[n][R][S][(ah*s + aw)*C + c] = x[n][R*s + ah - pad][S*s + aw - pad][c]        (zero outside the image),
 *   w_out[j][R][S][(ah*s + aw)*C + c] = w[j][R*s + ah][S*s + aw][c]                 (zero for taps >= k),
 * the kp x kp / stride 1 / pad 0 convolution of y with w_out equals the k x k / stride s / pad `pad` convolution
 * of x with w, exactly.  y has Ho + kp - 1 rows and Wo + kp - 1 columns (Ho, Wo the convolution's output extent)
 * and Cp >= s*s*C channels (a multiple of 8; the extra ones are zero), so the tensor-core kernels can load it.
 * dr_space_to_depth runs per forward pass (one read of x, one write of y); dr_s2d_filter once per filter bank.
 * Errors: INVALID_ARG, ALIGNMENT.                                                                            */
int dr_space_to_depth(int B, int H, int W, int C, int k, int s, int pad, int Cp, const void* x, void* y,
                      void* stream);
int dr_s2d_filter(int Cout, int k, int C, int s, int Cp, const void* w, void* w_out, void* stream);
/* The same re-layout read backwards, for the layer-wise regression (Eq. (w_b)) of such a layer: the filter gradient
 * of the stride-1 stand-in, dw_s2d float32 [Cout][kp][kp][Cp] (from dr_conv_wgrad on the space-to-depth image), gives
 * the gradient of the original filter, dw float32 [Cout][k][k][C]: dw[j][r][q][c] = dw_s2d[j][r/s][q/s][((r%s)*s + q%s)*C + c].
 * The update is applied to the original filter, which dr_s2d_filter then lays out again.                       */
int dr_s2d_filter_grad(int Cout, int k, int C, int s, int Cp, const float* dw_s2d, float* dw, void* stream);

/* ---- slim layers -------------------------------------------------------------------- */

/* One slim convolution layer (Eq. (tY_j = tW), Section 3.1, with the epilogue of the
 * descriptor): y = epilogue(conv(x; w) ).
 *  x: [B,H,W,Cin] dense bfloat16.   w: [Cout][k][k][Cin] bfloat16.   b: float32 [Cout] (DR_BIAS).
 *  residual: dense [B,Ho,Wo,Cout] bfloat16 (DR_RESIDUAL) else NULL.
 *  y: [B,Hy,Wy,*] with channel stride y_ldc, offset y_coff; (Hy,Wy) is the conv output extent,
 *     or the pooled extent with DR_POOL.  bfloat16, or float32 with DR_OUT_F32.
 *  argmax: NULL, or int32 [B,Hy,Wy,Cout] (DR_POOL only): flat position h*Wo+w in the conv
 *     output plane of the first maximum in row-major window order.
 * Restrictions: DR_POOL/DR_LRN need Cout <= 256 and exclude DR_RESIDUAL and DR_OUT_F32;
 * y_ldc, y_coff multiples of 8.  Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA.          */
int dr_conv_slim(const dr_conv_desc* desc, int B, int H, int W, const void* x, const void* w,
                 const float* b, const void* residual, void* y, int32_t* argmax, void* stream);

/* dr_conv_slim with scratch memory at hand.  A layer with few output pixels and a long
 * reduction (single-image inference, the regime of the paper's timings in Section 4.1: the 14x14
 * and 7x7 stages have 196 and 49 pixels against K = k*k*Cin up to 20800) is then computed split
 * along K: every SM multiplies a slice of K for one output tile, the float32 partial tiles meet
 * in the workspace and are summed in slice order, so the result does not depend on timing.
 * Same arithmetic (float32 accumulation, one rounding at the store), arguments and errors as
 * dr_conv_slim.  dr_conv_workspace_bytes() gives the size the layer can use (0: it would run as
 * in dr_conv_slim).  workspace: NULL, or device memory aligned to 256 bytes whose first
 * DR_CONV_WS_COUNTER_BYTES are zero before the first call; every call leaves them zero again, so
 * calls on one stream can share a workspace.  Calls that may overlap on the GPU need their own.
 * A workspace smaller than the layer wants is not an error: the layer runs as in dr_conv_slim. */
#define DR_CONV_WS_COUNTER_BYTES 1024
int dr_conv_workspace_bytes(const dr_conv_desc* desc, int B, int H, int W, size_t* bytes);
int dr_conv_slim_ws(const dr_conv_desc* desc, int B, int H, int W, const void* x, const void* w,
                    const float* b, const void* residual, void* y, int32_t* argmax, void* workspace,
                    size_t workspace_bytes, void* stream);

/* Branch-slimmed inception module (Section 3.2; the merged-branch identity Eqs. (LR), (W_b)):
 *   y[..., 0:c3)      = ReLU(conv3x3(ReLU(conv1x1(x; w[0]) + b[0]); w[1]) + b[1])
 *   y[..., c3:c3+cm)  = ReLU(conv5x5(x; w[2]) + b[2])          (pad 2, the merged branches)
 * written in place into y [B,H,W,c3+cm].  workspace holds the 1x1 output:
 * dr_inception_workspace_bytes() bytes.  pool_after != 0: the module is followed by the 3x3 / 2, pad 1 max-pooling layer
 * that follows inception 3b and 4e (Section 3.1: the pooling layer goes with the layer below it): y is then
 * [B,Hp,Wp,c3+cm] with Hp = (H - 1) / 2 + 1, the un-pooled output is kept in the workspace (which
 * dr_inception_workspace_bytes sizes accordingly) and pooled from there by dr_maxpool's kernel.                  */
typedef struct dr_inception_desc {
    int Cin, c3r, c3, cm;
    int pool_after;
} dr_inception_desc;
int dr_inception_workspace_bytes(const dr_inception_desc* desc, int B, int H, int W, size_t* bytes);
int dr_inception_slim(const dr_inception_desc* desc, int B, int H, int W, const void* x,
                      const void* const w[3], const float* const b[3], void* y, void* workspace,
                      void* stream);

/* dr_inception_slim for callers that cannot hand over scratch memory.  (The paper has no
 * counterpart: this is a deployment convenience of the library.)
 *
 * Who needs it: code that runs where device allocation is off limits — a plug-in executing
 * inside a host application's latency-critical loop, where cudaMalloc would synchronise the
 * device and stall every stream; a process whose memory budget was fixed at start-up and whose
 * allocator is closed afterwards; a component that may only touch the buffers it is handed for
 * input and output.  Such callers still pass x, the parameters and y, but no workspace: the
 * 1x1 reducer's output goes to a fixed array of DR_INCEPTION_STATIC_SCRATCH_BYTES inside the
 * library, which every GPU that loads the library keeps reserved until the process exits.
 *
 * Same arithmetic, arguments and errors as dr_inception_slim, plus:
 *  - B*H*W*c3r*2 bytes (rounded up to 256) must fit the array; a larger request returns
 *    DR_ERR_WORKSPACE and launches nothing.  Use dr_inception_slim with your own workspace then.
 *  - The call allocates nothing: no cudaMalloc/cudaFree, no allocating library routine.
 *  - The first call on each device looks up the array's device address (a host-side query, no
 *    allocation).  Make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps whatever the last call left in it.
 *    Nothing needs clearing between calls (the reducer overwrites everything the 3x3 convolution
 *    reads), but two calls whose kernels may overlap on the GPU — different streams without an
 *    ordering between them — race on it.  Issue them on one stream or order them with events. */
#define DR_INCEPTION_STATIC_SCRATCH_BYTES (4u << 20)
int dr_inception_slim_static(const dr_inception_desc* desc, int B, int H, int W, const void* x,
                             const void* const w[3], const float* const b[3], void* y, void* stream);

/* ---- stand-alone non-tensor layers (the "unslimmed" baseline, Section 2 / Table 2) -------
 * Each reads its input from and writes its output to device memory: one round trip per
 * layer, which is the cost the slim layers remove.  All tensors dense NHWC bfloat16.       */
int dr_relu(size_t n, const void* x, void* y, void* stream);
/* floor-mode output extent; padding never wins; argmax as in dr_conv_slim, or NULL */
int dr_maxpool(int B, int H, int W, int C, int k, int s, int p, const void* x, void* y,
               int32_t* argmax, void* stream);
/* y_c = x_c * (k + alpha/size * sum_{|c'-c| <= size/2, 0 <= c' < C} x_c'^2)^(-beta) */
int dr_lrn(int B, int H, int W, int C, int size, float alpha, float beta, float k, const void* x,
           void* y, void* stream);
/* BatchNorm layer, y = (x - mean/m)/sqrt(var/m + eps); followed by the Scale layer
 * y = gamma*y + beta when gamma is not NULL (Eq. (Y_batch_scala_conv), Section 3.1)        */
int dr_bn(int B, int H, int W, int C, const void* x, const float* mean, const float* var, float m,
          float eps, const float* gamma, const float* beta, void* y, void* stream);
/* Scale layer alone: y = gamma_c * x + beta_c */
int dr_scale(int B, int H, int W, int C, const void* x, const float* gamma, const float* beta, void* y,
             void* stream);
int dr_add(size_t n, const void* a, const void* b, void* y, void* stream);
/* copy dense [npix][C] into channels [coff, coff+C) of a tensor with channel stride ldc */
int dr_concat(size_t npix, int C, const void* x, int ldc, int coff, void* y, void* stream);
/* mean over the H x W plane: [B,H,W,C] -> [B,1,1,C] */
int dr_avgpool_global(int B, int H, int W, int C, const void* x, void* y, void* stream);

/* ---- whole networks ----------------------------------------------------------------- */
#define DR_ARCH_GOOGLENET  0   /* Inception-v1 topology, branch-slimmed modules (Section 4.1)    */
#define DR_ARCH_RESNET50   1   /* bottleneck v1; every conv followed by BatchNorm+Scale (4.3)    */
#define DR_ARCH_GOOGLENET_PAPER 2 /* GoogLeNet slimmed the paper's way (Section 3.2): per module two branches,
                                     1x1 -> 3x3 (reducer halved, output c3+c1) and 1x1 -> 5x5 (output c5+pp)   */
#define DR_ARCH_GOOGLENET_STREAMLINE 3 /* DR_ARCH_GOOGLENET with the stem in the paper's approximate streamline form
                                          (Section 3.1): the pools after conv1 and conv2 are dropped and their stride
                                          multiplied into the convolution (7x7/4, 3x3/2), both LRN layers pruned.  Not
                                          function-preserving: the paper re-trains; here it is a timing workload with
                                          parity against its own definition.                                          */
#define DR_ARCH_ALEXNET 4 /* AlexNet (two-tower groups, 227x227 input; Section 4.3): slim layers conv1 = conv + ReLU + LRN and
                             conv2 = grouped conv + ReLU + LRN; the unpadded 3x3/2 pools stay layers of their own, as in
                             the paper's Table "AlexNet Result" (conv1+norm1 -> conv1, conv2+norm2 -> conv2)            */
#define DR_MODE_SLIM       0   /* slim layers: folded BN, fused epilogues, merged branches       */
#define DR_MODE_UNSLIMMED  1   /* every layer of the original sequence as its own launch         */

typedef struct dr_net dr_net;

typedef struct dr_param_spec {
    char name[48];     /* e.g. "3a.b5.w", "res2a.2a.bn.gamma"                                    */
    int dims[4];       /* filters: Cout,k,k,Cin; vectors: C,1,1,1                                */
    int is_f32;        /* 0: bfloat16, 1: float32                                                */
    size_t count;      /* number of elements                                                     */
} dr_param_spec;

typedef struct dr_layer_info {
    char name[48];
    int kind;          /* 0 tensor layer (conv / FC), 1 non-tensor layer (Section 2's definition)*/
    int dims[4];       /* B,H,W,C of the slice this layer writes                                 */
    int ldc, coff;     /* channel stride / offset of that slice                                  */
    int is_f32;
    const void* ptr;   /* device address of element (0,0,0,0) of the slice; valid after prepare  */
    double flops;      /* 2*M*N*K for tensor layers, 0 otherwise                                 */
    double bytes;      /* algorithmic bytes read + written                                       */
    int conv_path;     /* which convolution kernel runs it (DR_PATH_*), -1 for non-tensor        */
} dr_layer_info;

/* Both modes take the SAME parameter list: the original, un-slimmed parameters (separate
 * branch filters, BatchNorm/Scale vectors).  In slim mode dr_net_prepare() derives the slim
 * parameters from them (dr_fold_bn, dr_embed_filter + concatenation) into the workspace.
 * dr_net_create is host-only.  B,H,W: batch and input plane (3 channels).                  */
int dr_net_create(dr_net** net, int arch, int mode, int B, int H, int W);
int dr_net_destroy(dr_net* net);
int dr_net_num_params(const dr_net* net);
int dr_net_param_spec(const dr_net* net, int idx, dr_param_spec* spec);
int dr_net_set_param(dr_net* net, int idx, const void* dev);   /* borrowed, not copied */
int dr_net_workspace_bytes(const dr_net* net, size_t* bytes);
/* Once per (net, workspace), after every parameter is set: derives slim parameters, lays the
 * activation buffers out in the workspace.  Enqueues on stream.  The workspace must be
 * 256-byte aligned and must not be used for anything else while the net is in use.        */
int dr_net_prepare(dr_net* net, void* workspace, void* stream);
/* x: [B,H,W,3] bfloat16; logits: float32 [B][1000].  One launch per layer on `stream`. */
int dr_net_forward(dr_net* net, const void* x, void* workspace, float* logits, void* stream);
int dr_net_num_layers(const dr_net* net);
int dr_net_layer_info(const dr_net* net, int layer, dr_layer_info* info);
/* Per-layer CUDA-event timing (the layer-wise protocol of Section 4.1): when enabled, each
 * forward records events around every launch; dr_net_layer_time_us synchronises on them.  */
int dr_net_set_timing(dr_net* net, int enabled);
int dr_net_layer_time_us(dr_net* net, int layer, float* us);
/* Bytes of the workspace that hold activations (run-time memory, Table 6's quantity). */
int dr_net_activation_bytes(const dr_net* net, size_t* bytes);

/* ---- diagnostics -------------------------------------------------------------------- */
#define DR_PATH_AUTO         0
#define DR_PATH_SIMT         1  /* CUDA-core implicit GEMM: any shape, slow                      */
#define DR_PATH_UMMA_GATHER  2  /* tcgen05 MMA, operands gathered by producer warps              */
#define DR_PATH_UMMA_TMA     3  /* tcgen05 MMA, operands loaded by TMA (im2col / tiled)          */
#define DR_PATH_UMMA_PATCH   4  /* pooling layers: 2-D output patches, TMA box loads, fused pool/LRN */
#define DR_PATH_UMMA_STEM    5  /* the 7x7/2 3-channel stem with fused pool/LRN                  */
#define DR_PATH_RETIRED_6    6  /* number of a removed kernel; forcing it gives DR_ERR_UNSUPPORTED  */
#define DR_PATH_UMMA_STEM_D  7  /* the stem with the MMA reading the input rows in place (no im2col) */
#define DR_PATH_UMMA_SPLITK  8  /* few output tiles: K split across the SMs, partial tiles summed in scratch (needs a workspace) */
#define DR_PATH_UMMA_QLIN    9  /* stride-1 3x3 / 5x5: the tile's input patch loaded once, every tap read out of it by the MMA */
/* Force a convolution kernel (tests, A/B timing); DR_PATH_AUTO picks the fastest that
 * supports the layer.  A forced path that cannot run the layer gives DR_ERR_UNSUPPORTED.   */
int dr_set_conv_path(int path);
int dr_last_conv_path(void);            /* path taken by the latest dr_conv_slim call */
/* Synchronises the device, then reads and clears the record the kernels leave when a bounded
 * wait runs out: returns DR_OK or DR_ERR_DEVICE_TIMEOUT; info[0..3] (may be NULL) receive the
 * code, a kernel-specific site id, the block index and the tile index.                    */
int dr_device_status(int info[4]);
/* Self-test of the bounded-wait path: launches one small kernel that waits, for at most limit_cycles SM cycles
 * (1 .. 2e9), on a barrier nothing arrives on, and then leaves the same record a convolution kernel would.
 * dr_device_status() afterwards returns DR_ERR_DEVICE_TIMEOUT with info[1] = 99; the context stays usable. */
int dr_selftest_wait_timeout(long long limit_cycles, void* stream);
/* ---- layer-wise regression of a slim layer (Section 3.1, Eq. (w_b) and Lemma 1) -------------------------
 * The slim layer f~(W, b; X) = ReLU(conv(X; W) + b) is re-learned from pairs (X, Y_CNN) of the input and the
 * output feature map of the layer group it replaces, by SGD on L = 1/(2B) * sum_i ||Y_CNN^i - f~(W, b; X^i)||_F^2
 * over mini-batches of B images.  The paper fixes neither the constant in front of the sum nor the form of the
 * update; the constant is the Euclidean loss's 1/(2B), the update is
 *     v <- momentum * v + lr * (g + decay * w);   w <- w - v.
 * One step = dr_conv_slim (forward, Y) -> dr_regress_grad -> dr_conv_wgrad -> dr_sgd_update (filters, bias);
 * dr_regress_step runs exactly that sequence.  All device buffers are the caller's; nothing is allocated.      */

/* dZ = dL/dZ for Y = ReLU(Z): (Y - Y_CNN) / B where Y > 0 (everywhere when relu == 0), rounded to bfloat16;
 * db[c] = sum over pixels of that (rounded) dZ; *loss = 1/(2B) * sum (Y - Y_CNN)^2 (loss may be NULL).
 *  y, yt, dz: dense [B,H,W,C] bfloat16 (dz may not alias y or yt); db: float32 [C].  C a multiple of 8 and <= 2048
 *  takes the vector kernel, other C a plain element-wise one.
 *  workspace: dr_regress_workspace_bytes(C) bytes, 256-byte aligned.  Sums are taken in a fixed order.
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE.                                                                   */
int dr_regress_workspace_bytes(int C, size_t* bytes);
int dr_regress_grad(int B, int H, int W, int C, const void* y, const void* yt, int relu, void* dz, float* db,
                    float* loss, void* workspace, size_t workspace_bytes, void* stream);

/* The same for a SHARD of a mini-batch (a data-parallel step: the mini-batch of `batch` images is split over ranks, this
 * call sees B <= batch of them).  Eq. (w_b) sums over samples, so with the mini-batch's constant in every shard,
 *   dZ = (Y - Y_CNN) / batch,   loss = 1/(2 batch) * sum over the shard,
 * the shards' db, loss (and the filter gradients taken from their dZ) ADD UP to the whole step's: a sum-all-reduce of
 * dW, db and loss over the ranks, then dr_sgd_update on every rank.  dr_regress_grad is this call with batch = B.     */
int dr_regress_grad_shard(int B, int batch, int H, int W, int C, const void* y, const void* yt, int relu, void* dz,
                          float* db, float* loss, void* workspace, size_t workspace_bytes, void* stream);

/* Filter gradient of the convolution of `desc` (k, stride, pad, Cin, Cout; flags and y_ldc are not looked at):
 *   dw[j][r][s][c] = sum over (n, ho, wo) of dz[n][ho][wo][j] * x[n][ho*stride - pad + r][wo*stride - pad + s][c]
 * with x zero outside the image.  x: [B,H,W,Cin] dense bfloat16; dz: [B,Ho,Wo,Cout] dense bfloat16;
 * dw: float32 [Cout][k][k][Cin], overwritten.  Products are exact, sums float32 on the tensor cores; the pixel
 * range is cut into pieces whose partial sums (in `workspace`) are added in a fixed order.
 * Layers with Cin < 64, or with Cin or Cout not a multiple of 8, run on a plain CUDA-core kernel instead (one thread
 * per filter element, pixels summed in order; there for completeness, needs no workspace).
 * workspace: dr_conv_wgrad_workspace_bytes bytes (may be 0), 256-byte aligned.  Errors: INVALID_ARG, ALIGNMENT, WORKSPACE. */
int dr_conv_wgrad_workspace_bytes(const dr_conv_desc* desc, int B, int H, int W, size_t* bytes);
int dr_conv_wgrad(const dr_conv_desc* desc, int B, int H, int W, const void* x, const void* dz, float* dw,
                  void* workspace, size_t workspace_bytes, void* stream);

/* v <- momentum * v + lr * (g + decay * w);  w <- w - v  over n float32 elements, in place; w_bf16 (NULL or n
 * bfloat16) receives the updated w rounded to nearest even, the copy the next forward pass reads.             */
int dr_sgd_update(size_t n, float* w, float* v, const float* g, float lr, float momentum, float decay,
                  void* w_bf16, void* stream);

/* One whole step on a mini-batch.  desc: the slim layer (DR_BIAS required; DR_RELU optional; no pooling, LRN,
 * residual, float32 output or channel slice).  x: [B,H,W,Cin]; yt: Y_CNN, [B,Ho,Wo,Cout]; w, b: float32 master
 * parameters, vw, vb: their momentum buffers, w_bf16: the bfloat16 filters the forward pass reads (all updated);
 * y, dz: [B,Ho,Wo,Cout] bfloat16 scratch (y holds the forward output of the parameters before the update);
 * dw: float32 [Cout][k][k][Cin] and db: float32 [Cout] receive the gradients; *loss the loss before the update.
 * The bias takes no weight decay.  workspace: dr_regress_step_workspace_bytes bytes, 256-byte aligned, zero-filled
 * before the first call (the forward pass of a layer with few output tiles keeps its tile counters there and
 * leaves them at zero; the gradient scratch in front of them is overwritten every call).
 * Layers with Cin < 64 or channel counts that are not multiples of 8 are taken too (on the plain kernels of
 * dr_conv_wgrad / dr_regress_grad).  Errors: INVALID_ARG, UNSUPPORTED (flags other than bias / ReLU, a channel slice),
 * ALIGNMENT, WORKSPACE, and whatever the forward pass returns.                                                */
int dr_regress_step_workspace_bytes(const dr_conv_desc* desc, int B, int H, int W, size_t* bytes);
int dr_regress_step(const dr_conv_desc* desc, int B, int H, int W, const void* x, const void* yt, float* w, float* b,
                    float* vw, float* vb, void* w_bf16, float lr, float momentum, float decay, void* y, void* dz,
                    float* dw, float* db, float* loss, void* workspace, size_t workspace_bytes, void* stream);

/* One rank's part of a data-parallel step: forward on its shard (B of the mini-batch's `batch` images), dr_regress_grad_shard,
 * dr_conv_wgrad; no update.  dw, db, *loss are the shard's contributions (see dr_regress_grad_shard): sum them over the
 * ranks (e.g. one all-reduce of Cout*k*k*Cin + Cout + 1 floats), then call dr_sgd_update for the filters and the bias as
 * dr_regress_step does.  Arguments, workspace (dr_regress_step_workspace_bytes) and errors as dr_regress_step.        */
int dr_regress_shard_grads(const dr_conv_desc* desc, int B, int batch, int H, int W, const void* x, const void* yt,
                           const void* w_bf16, const float* b, void* y, void* dz, float* dw, float* db, float* loss,
                           void* workspace, size_t workspace_bytes, void* stream);

/* Kernels of this library launched by this process so far. */
long long dr_launch_count(void);
/* Tensor maps (TMA descriptors) the library has had the driver encode so far.  Maps are remembered by the arguments
 * they were encoded from, so a layer called again on the same buffers encodes nothing.                          */
long long dr_tensor_map_encodes(void);
/* How dr_conv_slim would run a layer (no launch): plan[0] the kernel (DR_PATH_*), plan[1] output channels per
 * accumulator block, plan[2] such blocks along Cout, plan[3] 1 if CTA pairs (cta_group::2) are used, plan[4] 1 if a
 * tile carries two blocks that share the activation tile, plan[5..7] reserved (0).  workspace_bytes: the scratch the
 * call would be given (as in dr_conv_slim_ws; 0 for dr_conv_slim).  Errors as dr_conv_slim's validation.        */
int dr_conv_plan(const dr_conv_desc* desc, int B, int H, int W, size_t workspace_bytes, int plan[8]);

#ifdef __cplusplus
}
#endif
#endif /* DR_H_ */
