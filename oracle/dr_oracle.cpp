// CPU checker for the DeepRebirth slim-layer execution path.
//
// TEST INFRASTRUCTURE ONLY.  Plain, slow, direct-loop definitions in double
// precision of every layer the method executes, in the UNFUSED and UNMERGED
// form the paper starts from (Eq. f_map, Section 3.1): convolution, then
// BatchNorm, then Scale, then ReLU, then pooling / LRN as separate passes;
// an inception module as separate branch convolutions whose outputs are
// concatenated (Eq. LR, Section 3.2).  Nothing here is blocked, fused or
// reordered, and nothing is shared with the CUDA library: no headers, tables,
// helpers or constants.  The only threading is an OpenMP "parallel for" over
// independent output pixels.
//
// Tensors are NHWC, dense, double.  Filters are [Cout][kh][kw][Cin].
//
// Pinned by tests/test_oracle_pins.py (closed forms, brute force, the paper's
// identities, PyTorch CPU float64 on tiny shapes).
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>

#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

int orc_num_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

// Output extent of a convolution or floor-mode pooling window.
int orc_out_size(int in, int k, int stride, int pad) { return (in + 2 * pad - k) / stride + 1; }

// Convolution, Eq. (tY_j = tW * X + B) of the Lemma-2 proof (Section 3.1):
//   y[n,ho,wo,j] = b[j] + sum_{r,s,c} x[n, ho*stride-pad+r, wo*stride-pad+s, c] * w[j,r,s,c]
// with zeros outside the input plane.  bias may be null.
void orc_conv2d(int B, int H, int W, int Cin, const double* x, int k, int stride, int pad, int Cout,
                const double* w, const double* bias, double* y) {
    const int Ho = orc_out_size(H, k, stride, pad), Wo = orc_out_size(W, k, stride, pad);
    const long npix = (long)B * Ho * Wo;
#pragma omp parallel for schedule(static)
    for (long p = 0; p < npix; ++p) {
        const int n = (int)(p / ((long)Ho * Wo));
        const int ho = (int)((p / Wo) % Ho), wo = (int)(p % Wo);
        for (int j = 0; j < Cout; ++j) {
            double acc = bias ? bias[j] : 0.0;
            for (int r = 0; r < k; ++r) {
                const int hi = ho * stride - pad + r;
                if (hi < 0 || hi >= H) continue;
                for (int s = 0; s < k; ++s) {
                    const int wi = wo * stride - pad + s;
                    if (wi < 0 || wi >= W) continue;
                    const double* xp = x + (((long)n * H + hi) * W + wi) * Cin;
                    const double* wp = w + (((long)j * k + r) * k + s) * Cin;
                    double t = 0.0;
#pragma omp simd reduction(+ : t)
                    for (int c = 0; c < Cin; ++c) t += xp[c] * wp[c];
                    acc += t;
                }
            }
            y[p * Cout + j] = acc;
        }
    }
}

// BatchNorm layer as the paper's framework stores it (Section 3.1, the BN step of
// Eq. Y_batch_scala_conv): accumulated mean mu and variance sigma^2 with a scale
// factor m, so the true statistics are mu/m and sigma^2/m.  eps = 0 is the paper's
// formula; eps > 0 is the usual numerical guard.
void orc_batchnorm(long npix, int C, const double* x, const double* mu, const double* sigma2, double m,
                   double eps, double* y) {
#pragma omp parallel for schedule(static)
    for (long p = 0; p < npix; ++p)
        for (int j = 0; j < C; ++j)
            y[p * C + j] = (x[p * C + j] - mu[j] / m) / std::sqrt(sigma2[j] / m + eps);
}

// Scale layer (the Scaling step of Eq. Y_batch_scala_conv): y = gamma_j * x + beta_j.
void orc_scale(long npix, int C, const double* x, const double* gamma, const double* beta, double* y) {
#pragma omp parallel for schedule(static)
    for (long p = 0; p < npix; ++p)
        for (int j = 0; j < C; ++j) y[p * C + j] = gamma[j] * x[p * C + j] + beta[j];
}

void orc_relu(long n, const double* x, double* y) {
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n; ++i) y[i] = x[i] > 0.0 ? x[i] : 0.0;
}

// Max pooling over the k x k window (the "nearby p regions" of Section 3.1), stride s,
// pad p, floor-mode output size.  Padding never wins.  argmax (may be null) receives the
// flat position h*W+w, inside the un-padded input plane, of the first maximum met in
// row-major window order (a later equal value does not replace an earlier one).
void orc_maxpool(int B, int H, int W, int C, int k, int s, int p, const double* x, double* y,
                 int32_t* argmax) {
    const int Ho = orc_out_size(H, k, s, p), Wo = orc_out_size(W, k, s, p);
    const long npix = (long)B * Ho * Wo;
#pragma omp parallel for schedule(static)
    for (long q = 0; q < npix; ++q) {
        const int n = (int)(q / ((long)Ho * Wo));
        const int ho = (int)((q / Wo) % Ho), wo = (int)(q % Wo);
        for (int c = 0; c < C; ++c) {
            double best = -std::numeric_limits<double>::infinity();
            int32_t where = -1;
            for (int r = 0; r < k; ++r) {
                const int hi = ho * s - p + r;
                if (hi < 0 || hi >= H) continue;
                for (int t = 0; t < k; ++t) {
                    const int wi = wo * s - p + t;
                    if (wi < 0 || wi >= W) continue;
                    const double v = x[(((long)n * H + hi) * W + wi) * C + c];
                    if (where < 0 || v > best) { best = v; where = hi * W + wi; }
                }
            }
            y[q * C + c] = best;
            if (argmax) argmax[q * C + c] = where;
        }
    }
}

// Local response normalisation across channels, the paper's framework's form:
//   scale_c = kappa + (alpha / size) * sum_{c' in [c - size/2, c + size/2], 0 <= c' < C} x_{c'}^2
//   y_c     = x_c * scale_c^(-beta)
void orc_lrn(long npix, int C, int size, double alpha, double beta, double kappa, const double* x,
             double* y) {
    const int half = size / 2;
#pragma omp parallel for schedule(static)
    for (long p = 0; p < npix; ++p)
        for (int c = 0; c < C; ++c) {
            double ss = 0.0;
            for (int d = -half; d <= half; ++d) {
                const int cc = c + d;
                if (cc < 0 || cc >= C) continue;
                ss += x[p * C + cc] * x[p * C + cc];
            }
            y[p * C + c] = x[p * C + c] * std::pow(kappa + alpha / size * ss, -beta);
        }
}

void orc_add(long n, const double* a, const double* b, double* y) {
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n; ++i) y[i] = a[i] + b[i];
}

// Write a C-channel tensor into channels [coff, coff+C) of a tensor with ldc channels
// (the concatenation of Eq. LR, Section 3.2, one branch at a time).
void orc_concat_into(long npix, int C, const double* x, int ldc, int coff, double* y) {
    for (long p = 0; p < npix; ++p)
        for (int c = 0; c < C; ++c) y[p * ldc + coff + c] = x[p * C + c];
}

// Mean over the whole H x W plane per (image, channel).
void orc_avgpool_global(int B, int H, int W, int C, const double* x, double* y) {
    for (int n = 0; n < B; ++n)
        for (int c = 0; c < C; ++c) {
            double s = 0.0;
            for (long q = 0; q < (long)H * W; ++q) s += x[((long)n * H * W + q) * C + c];
            y[(long)n * C + c] = s / ((double)H * W);
        }
}

// Lemma 2 (Eq. W_B_S, Section 3.1), closed form of conv -> BatchNorm -> Scale:
//   eta_j = gamma_j / sqrt(sigma2_j / m [+ eps]);  W~_j = eta_j W_j;
//   B~_j  = eta_j B_j + beta_j - eta_j mu_j / m.
// K = kh*kw*Cin values per output channel.  b_in may be null (zero bias).
void orc_fold_bn(int Cout, long K, const double* w_in, const double* b_in, const double* mu,
                 const double* sigma2, double m, double eps, const double* gamma, const double* beta,
                 double* w_out, double* b_out) {
    for (int j = 0; j < Cout; ++j) {
        const double eta = gamma[j] / std::sqrt(sigma2[j] / m + eps);
        for (long i = 0; i < K; ++i) w_out[j * K + i] = eta * w_in[j * K + i];
        b_out[j] = eta * (b_in ? b_in[j] : 0.0) + beta[j] - eta * mu[j] / m;
    }
}

// "Adjust to the same size" of Section 3.2 made exact: place a ks x ks filter bank
// at the centre of a kb x kb one (zeros elsewhere); with pad kb/2 instead of ks/2 the
// stride-1 convolution is unchanged.  Writes filters [joff, joff+Cout) of w_big.
void orc_embed_filter(int Cout, int Cin, int ks, int kb, const double* w_small, int joff,
                      double* w_big) {
    const int o = (kb - ks) / 2;
    for (int j = 0; j < Cout; ++j) {
        double* dst = w_big + (long)(joff + j) * kb * kb * Cin;
        std::memset(dst, 0, sizeof(double) * kb * kb * Cin);
        for (int r = 0; r < ks; ++r)
            for (int s = 0; s < ks; ++s)
                for (int c = 0; c < Cin; ++c)
                    dst[((long)(r + o) * kb + (s + o)) * Cin + c] = w_small[(((long)j * ks + r) * ks + s) * Cin + c];
    }
}

// Round each value to the nearest bfloat16 (8 significant bits, ties to even).  Used
// only where the slim path stores a tensor in bfloat16 between layers.
void orc_round_bf16(long n, const double* x, double* y) {
    for (long i = 0; i < n; ++i) {
        const double v = x[i];
        if (v == 0.0 || !std::isfinite(v)) { y[i] = v; continue; }
        int e;
        const double mant = std::frexp(v, &e);              // |mant| in [0.5, 1)
        if (e < -125) {                                       // below the normal range: fixed quantum 2^-133
            y[i] = std::ldexp(std::nearbyint(std::ldexp(v, 133)), -133);
        } else {
            y[i] = std::ldexp(std::nearbyint(std::ldexp(mant, 8)), e - 8);
        }
    }
}

}  // extern "C"
