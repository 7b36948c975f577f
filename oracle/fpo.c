/*
 * CPU oracle primitives (fp64, NCHW activations, KCRS filters).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against; nothing in the product path links, loads or
 * calls it, and it shares no code with the CUDA sources.
 *
 * Every routine is the literal definition of its operator written as nested
 * loops; the only parallelism is an OpenMP split over images.  The paper
 * (Sec. IV) specifies the method in terms of these standard operators:
 * convolution with a k x c x r x s filter bank (Sec. IV-B.1), batch
 * normalisation in its inference form (Eq. 3-5 restate it as an affine map;
 * the form below is the textbook one so that Eq. 3-5 are themselves tested),
 * ReLU, element-wise addition, pooling and a fully connected layer.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC fpo.c -o libfpo.so
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

/* y[n,k,p,q] = sum_{c,r,s} x[n,c,p*st+r-pad,q*st+s-pad] * w[k,c,r,s], zero padding. */
void fpo_conv2d(const double* x, const double* w, double* y, int N, int C, int H, int W, int K, int R,
                int S, int stride, int pad) {
    const int P = (H + 2 * pad - R) / stride + 1;
    const int Q = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int k = 0; k < K; ++k) {
            double* yk = y + ((size_t)n * K + k) * P * Q;
            for (int i = 0; i < P * Q; ++i) yk[i] = 0.0;
            for (int c = 0; c < C; ++c) {
                const double* xc = x + ((size_t)n * C + c) * H * W;
                for (int r = 0; r < R; ++r) {
                    for (int s = 0; s < S; ++s) {
                        const double wv = w[(((size_t)k * C + c) * R + r) * S + s];
                        for (int p = 0; p < P; ++p) {
                            const int ih = p * stride + r - pad;
                            if (ih < 0 || ih >= H) continue;
                            for (int q = 0; q < Q; ++q) {
                                const int iw = q * stride + s - pad;
                                if (iw < 0 || iw >= W) continue;
                                yk[p * Q + q] += wv * xc[ih * W + iw];
                            }
                        }
                    }
                }
            }
        }
    }
}

/* Inference batch norm, textbook form: gamma*(x-mean)/sqrt(var+eps)+beta per channel. */
void fpo_bn(const double* x, double* y, int N, int C, int HW, const double* gamma, const double* beta,
            const double* mean, const double* var, double eps) {
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c) {
            const double den = sqrt(var[c] + eps);
            const double* xi = x + ((size_t)n * C + c) * HW;
            double* yi = y + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) yi[i] = gamma[c] * (xi[i] - mean[c]) / den + beta[c];
        }
}

/* Per-channel bias add (used by the fused graph: folded BN shift). */
void fpo_bias(double* y, int N, int C, int HW, const double* b) {
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c) {
            double* yi = y + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) yi[i] += b[c];
        }
}

void fpo_relu(const double* x, double* y, size_t count) {
    for (size_t i = 0; i < count; ++i) y[i] = x[i] > 0.0 ? x[i] : 0.0;
}

void fpo_add(const double* a, const double* b, double* y, size_t count) {
    for (size_t i = 0; i < count; ++i) y[i] = a[i] + b[i];
}

/* Parameter-free downsampling shortcut: y[n,k,i,j] = x[n,k-pad_lo,i*st,j*st] for
 * pad_lo <= k < pad_lo+C, zero for the other channels.  Output is ceil(H/st) x ceil(W/st). */
void fpo_shortcut_a(const double* x, double* y, int N, int C, int H, int W, int K, int stride, int pad_lo) {
    const int P = (H + stride - 1) / stride, Q = (W + stride - 1) / stride;
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k)
            for (int p = 0; p < P; ++p)
                for (int q = 0; q < Q; ++q) {
                    const int c = k - pad_lo;
                    double v = 0.0;
                    if (c >= 0 && c < C) v = x[(((size_t)n * C + c) * H + p * stride) * W + q * stride];
                    y[(((size_t)n * K + k) * P + p) * Q + q] = v;
                }
}

/* Max pooling; padded positions never take part in the max. */
void fpo_maxpool(const double* x, double* y, int N, int C, int H, int W, int R, int stride, int pad) {
    const int P = (H + 2 * pad - R) / stride + 1;
    const int Q = (W + 2 * pad - R) / stride + 1;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int p = 0; p < P; ++p)
                for (int q = 0; q < Q; ++q) {
                    double m = -INFINITY;
                    for (int r = 0; r < R; ++r)
                        for (int s = 0; s < R; ++s) {
                            const int ih = p * stride + r - pad, iw = q * stride + s - pad;
                            if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue;
                            const double v = x[(((size_t)n * C + c) * H + ih) * W + iw];
                            if (v > m) m = v;
                        }
                    y[(((size_t)n * C + c) * P + p) * Q + q] = m;
                }
}

/* Global average pooling: mean over all H*W positions. */
void fpo_gavgpool(const double* x, double* y, int N, int C, int HW) {
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c) {
            double s = 0.0;
            const double* xi = x + ((size_t)n * C + c) * HW;
            for (int i = 0; i < HW; ++i) s += xi[i];
            y[(size_t)n * C + c] = s / (double)HW;
        }
}

/* Fully connected: y[n,k] = sum_c x[n,c]*w[k,c] + b[k]. */
void fpo_fc(const double* x, const double* w, const double* b, double* y, int N, int C, int K) {
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            double s = 0.0;
            for (int c = 0; c < C; ++c) s += x[(size_t)n * C + c] * w[(size_t)k * C + c];
            y[(size_t)n * K + k] = s + (b ? b[k] : 0.0);
        }
}

/*
 * BN folding in single precision (Eq. 3-5 and the merge of BN into the preceding
 * convolution, Sec. V-C "*" models).  Filter scores are taken on these fp32 folded
 * weights, so the operation order is fixed: every step is one round-to-nearest fp32
 * operation, no fused multiply-add (compile with -ffp-contract=off):
 *   t = var + eps;  r = sqrt(t);  omega = gamma / r;  w' = omega * w;
 *   m = omega * mean;  lambda = beta - m.
 */
void fpo_fold_bn_f32(const float* w, int K, int per_filter, const float* gamma, const float* beta,
                     const float* mean, const float* var, float eps, float* w_out, float* b_out,
                     float* omega_out) {
    for (int k = 0; k < K; ++k) {
        volatile float t = var[k] + eps;
        volatile float r = sqrtf(t);
        volatile float omega = gamma[k] / r;
        for (int i = 0; i < per_filter; ++i) {
            volatile float p = omega * w[(size_t)k * per_filter + i];
            w_out[(size_t)k * per_filter + i] = p;
        }
        volatile float m = omega * mean[k];
        volatile float lam = beta[k] - m;
        b_out[k] = lam;
        if (omega_out) omega_out[k] = omega;
    }
}

/*
 * Filter score (Eq. 6 without the monotone square root for the l2 norm; the l1 norm is
 * the sum of magnitudes).  Each term |w| or w*w is exact in fp64 because w is fp32.
 * The sum is taken in a fixed order so that the result is one well-defined double:
 * the filter is flattened in (c,r,s) order, 32 partial sums take elements
 * t = l, l+32, l+64, ... in increasing t, and the partial sums are combined pairwise
 * with partners at distance 16, 8, 4, 2, 1 (p[l] += p[l^d], all l at once).
 */
double fpo_score_filter(const float* w, int count, int norm_l2) {
    double part[32];
    for (int l = 0; l < 32; ++l) {
        double s = 0.0;
        for (int t = l; t < count; t += 32) {
            const double v = (double)w[t];
            s += norm_l2 ? v * v : fabs(v);
        }
        part[l] = s;
    }
    for (int d = 16; d >= 1; d >>= 1) {
        double next[32];
        for (int l = 0; l < 32; ++l) next[l] = part[l] + part[l ^ d];
        for (int l = 0; l < 32; ++l) part[l] = next[l];
    }
    return part[0];
}

void fpo_score(const float* w, int K, int per_filter, int norm_l2, double* scores) {
    for (int k = 0; k < K; ++k) scores[k] = fpo_score_filter(w + (size_t)k * per_filter, per_filter, norm_l2);
}

int fpo_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
