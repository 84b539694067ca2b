/*
 * fp64 CPU oracle for the per-replica CNN training step (Algorithm 1: forward pass,
 * loss, backward pass, gradient averaging, parameter update).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain definition of every operation on the
 * step, written so that it can be checked against the formulas by eye.  It shares no code,
 * header, table or constant with the CUDA library; only tests, the smoke check and the
 * CPU-baseline leg of the benchmark may call it.
 *
 * Conventions: activations NHWC, weights KRSC (K output channels, R x S taps, C input
 * channels), everything double.  "Convolution" is cross-correlation (no kernel flip):
 *     y[n,p,q,k] = sum_{r,s,c} x[n, p*stride + r - pad, q*stride + s - pad, c] * w[k,r,s,c]
 * with x taken as zero outside the image.  P = floor((H + 2 pad - R)/stride) + 1, same for Q.
 *
 * No blocking, fusion or reordering beyond the loops the definitions state; OpenMP splits
 * only independent outer iterations.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

static int out_dim(int in, int taps, int stride, int pad) { return (in + 2 * pad - taps) / stride + 1; }

/* ---------------------------------------------------------------------------------------
 * Round-to-nearest-even onto the bfloat16 grid (1 sign, 8 exponent, 7 mantissa bits),
 * done directly from double so that no double rounding through float occurs.
 * Normal range: spacing is 2^(e-7) for |x| in [2^e, 2^(e+1)); below 2^-126 the spacing is
 * the subnormal quantum 2^-133.  rint() rounds half to even in the default rounding mode,
 * and scaling by a power of two is exact.
 * ------------------------------------------------------------------------------------ */
double orc_bf16_rne(double x)
{
    if (x == 0.0 || isnan(x) || isinf(x)) return x;
    double ax = fabs(x);
    int e;
    (void)frexp(ax, &e);          /* ax = m * 2^e with m in [0.5,1)  =>  ax in [2^(e-1), 2^e) */
    int exp2 = e - 1;             /* floor(log2(ax)) */
    if (exp2 < -126) exp2 = -126; /* subnormal range shares the quantum of the smallest normal binade */
    double quantum = ldexp(1.0, exp2 - 7);
    double r = rint(ax / quantum) * quantum;
    if (r >= ldexp(1.0, 128)) r = INFINITY;
    return x < 0 ? -r : r;
}

void orc_round_bf16(const double* in, double* out, long n)
{
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n; ++i) out[i] = orc_bf16_rne(in[i]);
}

/* ---------------------------------------------------------------------------------------
 * Forward convolution (the defining sum, gather form).
 * ------------------------------------------------------------------------------------ */
void orc_conv2d_fwd(const double* x, const double* w, double* y,
                    int N, int H, int W, int C, int K, int R, int S, int stride, int pad)
{
    const int P = out_dim(H, R, stride, pad), Q = out_dim(W, S, stride, pad);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int k = 0; k < K; ++k) {
                    double acc = 0.0;
                    for (int r = 0; r < R; ++r) {
                        const int h = p * stride + r - pad;
                        if (h < 0 || h >= H) continue;
                        for (int s = 0; s < S; ++s) {
                            const int ww = q * stride + s - pad;
                            if (ww < 0 || ww >= W) continue;
                            const double* xp = x + (((size_t)n * H + h) * W + ww) * C;
                            const double* wp = w + (((size_t)k * R + r) * S + s) * C;
                            double part = 0.0;
#pragma omp simd reduction(+ : part)
                            for (int c = 0; c < C; ++c) part += xp[c] * wp[c];
                            acc += part;
                        }
                    }
                    y[(((size_t)n * P + p) * Q + q) * K + k] = acc;
                }
}

/* ---------------------------------------------------------------------------------------
 * Data gradient, scatter form: every (output pixel, tap) pair pushes dy * w onto the
 * input pixel it read in the forward pass.  dx[n,h,w,c] = sum over (p,q,r,s,k) with
 * p*stride + r - pad = h and q*stride + s - pad = w of dy[n,p,q,k] * w[k,r,s,c].
 * ------------------------------------------------------------------------------------ */
void orc_conv2d_dgrad(const double* dy, const double* w, double* dx,
                      int N, int H, int W, int C, int K, int R, int S, int stride, int pad)
{
    const int P = out_dim(H, R, stride, pad), Q = out_dim(W, S, stride, pad);
    memset(dx, 0, sizeof(double) * (size_t)N * H * W * C);
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) /* images are independent, so no two threads touch the same dx */
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int k = 0; k < K; ++k) {
                    const double g = dy[(((size_t)n * P + p) * Q + q) * K + k];
                    for (int r = 0; r < R; ++r) {
                        const int h = p * stride + r - pad;
                        if (h < 0 || h >= H) continue;
                        for (int s = 0; s < S; ++s) {
                            const int ww = q * stride + s - pad;
                            if (ww < 0 || ww >= W) continue;
                            double* dxp = dx + (((size_t)n * H + h) * W + ww) * C;
                            const double* wp = w + (((size_t)k * R + r) * S + s) * C;
#pragma omp simd
                            for (int c = 0; c < C; ++c) dxp[c] += g * wp[c];
                        }
                    }
                }
}

/* ---------------------------------------------------------------------------------------
 * Weight gradient: dw[k,r,s,c] = sum_{n,p,q} dy[n,p,q,k] * x[n, p*stride+r-pad, q*stride+s-pad, c].
 * ------------------------------------------------------------------------------------ */
void orc_conv2d_wgrad(const double* dy, const double* x, double* dw,
                      int N, int H, int W, int C, int K, int R, int S, int stride, int pad)
{
    const int P = out_dim(H, R, stride, pad), Q = out_dim(W, S, stride, pad);
    memset(dw, 0, sizeof(double) * (size_t)K * R * S * C);
#pragma omp parallel for schedule(static)
    for (int k = 0; k < K; ++k) /* each thread owns dw[k,:,:,:] */
        for (int n = 0; n < N; ++n)
            for (int p = 0; p < P; ++p)
                for (int q = 0; q < Q; ++q) {
                    const double g = dy[(((size_t)n * P + p) * Q + q) * K + k];
                    for (int r = 0; r < R; ++r) {
                        const int h = p * stride + r - pad;
                        if (h < 0 || h >= H) continue;
                        for (int s = 0; s < S; ++s) {
                            const int ww = q * stride + s - pad;
                            if (ww < 0 || ww >= W) continue;
                            const double* xp = x + (((size_t)n * H + h) * W + ww) * C;
                            double* dwp = dw + (((size_t)k * R + r) * S + s) * C;
#pragma omp simd
                            for (int c = 0; c < C; ++c) dwp[c] += g * xp[c];
                        }
                    }
                }
}

/* ---------------------------------------------------------------------------------------
 * Training-mode batch normalisation + optional residual + optional ReLU over M = N*P*Q rows
 * of C channels.  Per channel: mean = sum(y)/M; var = sum((y-mean)^2)/M (biased, two-pass);
 * invstd = 1/sqrt(var+eps); z = gamma*(y-mean)*invstd + beta (+ residual); a = relu ? max(z,0) : z.
 * Outputs mean, invstd and the biased variance (the caller derives running statistics).
 * ------------------------------------------------------------------------------------ */
void orc_bn_stats(const double* y, long M, int C, double eps, double* mean, double* var, double* invstd)
{
#pragma omp parallel for schedule(static)
    for (int c = 0; c < C; ++c) {
        double s = 0.0;
        for (long m = 0; m < M; ++m) s += y[m * C + c];
        const double mu = s / (double)M;
        double ss = 0.0;
        for (long m = 0; m < M; ++m) {
            const double d = y[m * C + c] - mu;
            ss += d * d;
        }
        mean[c] = mu;
        var[c] = ss / (double)M;
        invstd[c] = 1.0 / sqrt(var[c] + eps);
    }
}

void orc_bn_relu_apply(const double* y, const double* mean, const double* invstd,
                       const double* gamma, const double* beta, const double* residual /* may be NULL */,
                       int relu, long M, int C, double* a)
{
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m)
        for (int c = 0; c < C; ++c) {
            double z = gamma[c] * (y[m * C + c] - mean[c]) * invstd[c] + beta[c];
            if (residual) z += residual[m * C + c];
            a[m * C + c] = (relu && z < 0.0) ? 0.0 : z;
        }
}

/* ---------------------------------------------------------------------------------------
 * Backward of the above.  dz = (da1 + da2) * [a > 0] (mask only if relu; ReLU'(0) = 0);
 * dbeta = sum dz; dgamma = sum dz*xhat, xhat = (y-mean)*invstd;
 * dy = gamma*invstd*(dz - dbeta/M - xhat*dgamma/M); dres = dz (gradient of the residual input).
 * ------------------------------------------------------------------------------------ */
void orc_bn_relu_bwd(const double* da1, const double* da2 /* may be NULL */, const double* y, const double* a,
                     const double* gamma, const double* mean, const double* invstd, int relu, long M, int C,
                     double* dy, double* dres /* may be NULL */, double* dgamma, double* dbeta)
{
#pragma omp parallel for schedule(static)
    for (int c = 0; c < C; ++c) {
        double sb = 0.0, sg = 0.0;
        for (long m = 0; m < M; ++m) {
            double dz = da1[m * C + c] + (da2 ? da2[m * C + c] : 0.0);
            if (relu && !(a[m * C + c] > 0.0)) dz = 0.0;
            const double xhat = (y[m * C + c] - mean[c]) * invstd[c];
            sb += dz;
            sg += dz * xhat;
        }
        dbeta[c] = sb;
        dgamma[c] = sg;
        for (long m = 0; m < M; ++m) {
            double dz = da1[m * C + c] + (da2 ? da2[m * C + c] : 0.0);
            if (relu && !(a[m * C + c] > 0.0)) dz = 0.0;
            const double xhat = (y[m * C + c] - mean[c]) * invstd[c];
            dy[m * C + c] = gamma[c] * invstd[c] * (dz - sb / (double)M - xhat * sg / (double)M);
            if (dres) dres[m * C + c] = dz;
        }
    }
}

/* Global average pool over the HW positions of each image, and its gradient. */
void orc_avgpool_fwd(const double* a, int N, int HW, int C, double* pooled)
{
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c) {
            double s = 0.0;
            for (int i = 0; i < HW; ++i) s += a[((size_t)n * HW + i) * C + c];
            pooled[(size_t)n * C + c] = s / (double)HW;
        }
}

void orc_avgpool_bwd(const double* dpooled, int N, int HW, int C, double* da)
{
    for (int n = 0; n < N; ++n)
        for (int i = 0; i < HW; ++i)
            for (int c = 0; c < C; ++c) da[((size_t)n * HW + i) * C + c] = dpooled[(size_t)n * C + c] / (double)HW;
}

/* ---------------------------------------------------------------------------------------
 * Softmax cross-entropy head.  loss = (1/N) sum_i (logsumexp(z_i) - z_i[label_i]);
 * dz[i,j] = (softmax(z_i)[j] - [j == label_i]) * grad_scale.  Max-subtracted logsumexp.
 * Returns -1 if a label is outside [0, classes).
 * ------------------------------------------------------------------------------------ */
int orc_softmax_xent(const double* z, const int32_t* labels, int N, int classes, double grad_scale,
                     double* loss, double* dz)
{
    double total = 0.0;
    for (int i = 0; i < N; ++i) {
        const double* zi = z + (size_t)i * classes;
        if (labels[i] < 0 || labels[i] >= classes) return -1;
        double mx = zi[0];
        for (int j = 1; j < classes; ++j) mx = zi[j] > mx ? zi[j] : mx;
        double se = 0.0;
        for (int j = 0; j < classes; ++j) se += exp(zi[j] - mx);
        const double lse = mx + log(se);
        total += lse - zi[labels[i]];
        for (int j = 0; j < classes; ++j)
            dz[(size_t)i * classes + j] = (exp(zi[j] - lse) - (j == labels[i] ? 1.0 : 0.0)) * grad_scale;
    }
    *loss = total / (double)N;
    return 0;
}

/* ---------------------------------------------------------------------------------------
 * Gradient averaging fused with the SGD-momentum update (Algorithm 1, the gradient
 * synchronisation and parameter update steps):
 * g = g_sum * inv_n + wd*w;  v = mu*v + g;  w = w - lr*v.   In place on w and v.
 * ------------------------------------------------------------------------------------ */
void orc_sgd_momentum(double* w, double* v, const double* g_sum, long count,
                      double inv_n, double lr, double mu, double wd)
{
    for (long i = 0; i < count; ++i) {
        const double g = g_sum[i] * inv_n + wd * w[i];
        v[i] = mu * v[i] + g;
        w[i] = w[i] - lr * v[i];
    }
}
