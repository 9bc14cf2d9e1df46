/*
 * fp64 CPU oracle for the Conv2d -> BatchNorm(training-mode batch statistics) -> SiLU block,
 * forward and backward.  TEST INFRASTRUCTURE ONLY: nothing in the product path links, loads
 * or calls this file; only tests, the smoke check and the benchmark's cpu_baseline leg do.
 * It shares no code with the CUDA library.
 *
 * The paper names the operators of its detector (convolutions, batch normalisation kept in
 * F32, SiLU activations: Sec. 3.2 "mixed precision", Sec. 6 "case study", Table 2 rows 2-3)
 * but prints no formula; the definitions are the ones of the works it cites for them, with
 * the dominant framework's defaults the paper says it adopts.  Because the method is exact,
 * every function below is the plain definition written out as direct loops in double
 * precision: no im2col, no blocking, no transform-domain convolution, no BLAS.
 *
 * Layouts: activations NHWC, weights [Cout][k][k][Cin] ("KRSC"), everything row-major
 * double.  pad = k/2 (integer division), out = (in + 2*pad - k)/stride + 1.
 *
 * Pins (tests/test_oracle_pins.py): 1x1 conv == matrix product; identity and shift kernels;
 * all-ones closed form; brute-force re-derivation on tiny tensors; adjoint identities
 * <conv(x,w),g> = <x,dgrad(g,w)> = <w,wgrad(x,g)>; BN zero-mean / mean(xhat^2) = 1-eps*invstd^2;
 * SiLU closed-form values; central finite differences of the whole block; sum(dy)=0 and
 * sum(dy*xhat) = gamma*dgamma*eps*invstd^3 per channel.  Evaluation-mode and plain variants (end of
 * the file): a hand-worked value; running statistics set to the batch statistics reproduce the
 * training-mode forward; gamma = 0 and huge-variance limits; conv + bias against a library
 * correlation; folded filter + bias reproduces the unfolded evaluation-mode block.
 * No function here is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define IDX4(a, b, c, d, B, C, D) ((((size_t)(a) * (size_t)(B) + (size_t)(b)) * (size_t)(C) + (size_t)(c)) * (size_t)(D) + (size_t)(d))

static int out_extent(int in, int k, int stride) { return (in + 2 * (k / 2) - k) / stride + 1; }

int oracle_out_extent(int in, int k, int stride) { return out_extent(in, k, stride); }

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Direct cross-correlation (no kernel flip), zero padding:
 *   y[n,p,q,c'] = sum_{r,t,c} x[n, p*s-P+r, q*s-P+t, c] * w[c',r,t,c],  terms outside the image are 0. */
void oracle_conv_fwd(const double* x, const double* w, double* y,
                     int N, int H, int W, int Cin, int Cout, int k, int stride)
{
    const int P = k / 2, Ho = out_extent(H, k, stride), Wo = out_extent(W, k, stride);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int p = 0; p < Ho; ++p)
            for (int q = 0; q < Wo; ++q)
                for (int co = 0; co < Cout; ++co) {
                    double acc = 0.0;
                    for (int r = 0; r < k; ++r) {
                        const int h = p * stride - P + r;
                        if (h < 0 || h >= H) continue;
                        for (int t = 0; t < k; ++t) {
                            const int ww = q * stride - P + t;
                            if (ww < 0 || ww >= W) continue;
                            const double* xp = x + IDX4(n, h, ww, 0, H, W, Cin);
                            const double* wp = w + IDX4(co, r, t, 0, k, k, Cin);
                            double s = 0.0;
#pragma omp simd reduction(+ : s)
                            for (int c = 0; c < Cin; ++c) s += xp[c] * wp[c];
                            acc += s;
                        }
                    }
                    y[IDX4(n, p, q, co, Ho, Wo, Cout)] = acc;
                }
}

/* Data gradient of the above: dx[n,h,w,c] = sum over (p,q,r,t,c') with p*s-P+r=h, q*s-P+t=w of dy[n,p,q,c']*w[c',r,t,c].
 * Written as a gather over the input pixel so that rows can be computed in parallel without races. */
void oracle_conv_dgrad(const double* dy, const double* w, double* dx,
                       int N, int H, int W, int Cin, int Cout, int k, int stride)
{
    const int P = k / 2, Ho = out_extent(H, k, stride), Wo = out_extent(W, k, stride);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int h = 0; h < H; ++h)
            for (int ww = 0; ww < W; ++ww) {
                double* dxp = dx + IDX4(n, h, ww, 0, H, W, Cin);
                for (int c = 0; c < Cin; ++c) dxp[c] = 0.0;
                for (int r = 0; r < k; ++r) {
                    const int hp = h + P - r;
                    if (hp < 0 || hp % stride != 0) continue;
                    const int p = hp / stride;
                    if (p >= Ho) continue;
                    for (int t = 0; t < k; ++t) {
                        const int wq = ww + P - t;
                        if (wq < 0 || wq % stride != 0) continue;
                        const int q = wq / stride;
                        if (q >= Wo) continue;
                        const double* dyp = dy + IDX4(n, p, q, 0, Ho, Wo, Cout);
                        for (int co = 0; co < Cout; ++co) {
                            const double gv = dyp[co];
                            const double* wp = w + IDX4(co, r, t, 0, k, k, Cin);
#pragma omp simd
                            for (int c = 0; c < Cin; ++c) dxp[c] += gv * wp[c];
                        }
                    }
                }
            }
}

/* Weight gradient: dw[c',r,t,c] = sum_{n,p,q} dy[n,p,q,c'] * x[n, p*s-P+r, q*s-P+t, c] (zero outside). */
void oracle_conv_wgrad(const double* x, const double* dy, double* dw,
                       int N, int H, int W, int Cin, int Cout, int k, int stride)
{
    const int P = k / 2, Ho = out_extent(H, k, stride), Wo = out_extent(W, k, stride);
#pragma omp parallel for collapse(2) schedule(static)
    for (int co = 0; co < Cout; ++co)
        for (int r = 0; r < k; ++r)
            for (int t = 0; t < k; ++t) {
                double* dwp = dw + IDX4(co, r, t, 0, k, k, Cin);
                for (int c = 0; c < Cin; ++c) dwp[c] = 0.0;
                for (int n = 0; n < N; ++n)
                    for (int p = 0; p < Ho; ++p) {
                        const int h = p * stride - P + r;
                        if (h < 0 || h >= H) continue;
                        for (int q = 0; q < Wo; ++q) {
                            const int ww = q * stride - P + t;
                            if (ww < 0 || ww >= W) continue;
                            const double gv = dy[IDX4(n, p, q, co, Ho, Wo, Cout)];
                            const double* xp = x + IDX4(n, h, ww, 0, H, W, Cin);
#pragma omp simd
                            for (int c = 0; c < Cin; ++c) dwp[c] += gv * xp[c];
                        }
                    }
            }
}

/* Training-mode batch statistics over the M = N*Ho*Wo rows of y[M][C]: two-pass mean and BIASED variance,
 * invstd = 1/sqrt(var + eps).  Optional running statistics use momentum m and the unbiased variance:
 *   rm <- (1-m) rm + m mean ;  rv <- (1-m) rv + m var*M/(M-1). */
void oracle_bn_stats(const double* y, long long M, int C, double eps,
                     double* mean, double* var, double* invstd,
                     double* running_mean, double* running_var, double momentum)
{
#pragma omp parallel for schedule(static)
    for (int c = 0; c < C; ++c) {
        double s = 0.0;
        for (long long i = 0; i < M; ++i) s += y[(size_t)i * C + c];
        const double mu = s / (double)M;
        double v = 0.0;
        for (long long i = 0; i < M; ++i) {
            const double d = y[(size_t)i * C + c] - mu;
            v += d * d;
        }
        v /= (double)M;
        mean[c] = mu;
        var[c] = v;
        invstd[c] = 1.0 / sqrt(v + eps);
        if (running_mean) running_mean[c] = (1.0 - momentum) * running_mean[c] + momentum * mu;
        if (running_var) running_var[c] = (1.0 - momentum) * running_var[c] + momentum * v * (double)M / (double)(M - 1);
    }
}

static double sigmoid(double z) { return 1.0 / (1.0 + exp(-z)); }

/* Normalise, affine, SiLU:  xhat = (y-mean)*invstd ; z = gamma*xhat + beta ; a = z*sigmoid(z). */
void oracle_bn_silu_fwd(const double* y, long long M, int C,
                        const double* mean, const double* invstd, const double* gamma, const double* beta,
                        double* a)
{
#pragma omp parallel for schedule(static)
    for (long long i = 0; i < M; ++i)
        for (int c = 0; c < C; ++c) {
            const double xhat = (y[(size_t)i * C + c] - mean[c]) * invstd[c];
            const double z = gamma[c] * xhat + beta[c];
            a[(size_t)i * C + c] = z * sigmoid(z);
        }
}

/* Backward of SiLU and of batch-statistics BN, given g = dL/da:
 *   s = sigmoid(z) ; dz = g*s*(1 + z*(1-s))
 *   dbeta = sum dz ; dgamma = sum dz*xhat
 *   dy = gamma*invstd*(dz - dbeta/M - xhat*dgamma/M) */
void oracle_bn_silu_bwd(const double* g, const double* y, long long M, int C,
                        const double* mean, const double* invstd, const double* gamma, const double* beta,
                        double* dy, double* dgamma, double* dbeta)
{
#pragma omp parallel for schedule(static)
    for (int c = 0; c < C; ++c) {
        double sb = 0.0, sg = 0.0;
        for (long long i = 0; i < M; ++i) {
            const double xhat = (y[(size_t)i * C + c] - mean[c]) * invstd[c];
            const double z = gamma[c] * xhat + beta[c];
            const double s = sigmoid(z);
            const double dz = g[(size_t)i * C + c] * s * (1.0 + z * (1.0 - s));
            sb += dz;
            sg += dz * xhat;
        }
        dbeta[c] = sb;
        dgamma[c] = sg;
    }
#pragma omp parallel for schedule(static)
    for (long long i = 0; i < M; ++i)
        for (int c = 0; c < C; ++c) {
            const double xhat = (y[(size_t)i * C + c] - mean[c]) * invstd[c];
            const double z = gamma[c] * xhat + beta[c];
            const double s = sigmoid(z);
            const double dz = g[(size_t)i * C + c] * s * (1.0 + z * (1.0 - s));
            dy[(size_t)i * C + c] = gamma[c] * invstd[c] * (dz - dbeta[c] / (double)M - xhat * dgamma[c] / (double)M);
        }
}

/* ---------------------------------------------------------------------------------------------
 * Evaluation-mode and plain variants (the paper's Table 2 row 9 fix: validation must normalise
 * with the running statistics, not with batch statistics; Table 2 row 3: the detection head's
 * output convolutions carry a bias and no normalisation).
 * ------------------------------------------------------------------------------------------- */

/* Evaluation-mode BN then optional SiLU: the stored running mean and running variance take the
 * place of the batch statistics; nothing is updated.
 *   z = gamma*(y - rmean)/sqrt(rvar + eps) + beta ;  a = act ? z*sigmoid(z) : z. */
void oracle_bn_eval_act(const double* y, long long M, int C,
                        const double* gamma, const double* beta, const double* rmean, const double* rvar,
                        double eps, int act, double* a)
{
#pragma omp parallel for schedule(static)
    for (long long i = 0; i < M; ++i)
        for (int c = 0; c < C; ++c) {
            const double xhat = (y[(size_t)i * C + c] - rmean[c]) / sqrt(rvar[c] + eps);
            const double z = gamma[c] * xhat + beta[c];
            a[(size_t)i * C + c] = act ? z * sigmoid(z) : z;
        }
}

/* Per-channel bias then optional SiLU:  z = y + bias[c] ;  out = act ? z*sigmoid(z) : z.  bias may be NULL (zero). */
void oracle_bias_act(const double* y, long long M, int C, const double* bias, int act, double* out)
{
#pragma omp parallel for schedule(static)
    for (long long i = 0; i < M; ++i)
        for (int c = 0; c < C; ++c) {
            const double z = y[(size_t)i * C + c] + (bias ? bias[c] : 0.0);
            out[(size_t)i * C + c] = act ? z * sigmoid(z) : z;
        }
}

/* Folding evaluation-mode BN into the convolution that feeds it: with s_c = gamma_c/sqrt(rvar_c + eps),
 *   w'[c',r,t,c] = s_c' * w[c',r,t,c] ;  bias'[c'] = beta_c' - rmean_c' * s_c',
 * so that conv(x, w') + bias' equals the BN output for every x.  K = k*k*Cin filter taps per output channel. */
void oracle_bn_fold(const double* w, int Cout, long long K,
                    const double* gamma, const double* beta, const double* rmean, const double* rvar, double eps,
                    double* w_folded, double* bias_folded)
{
    for (int co = 0; co < Cout; ++co) {
        const double s = gamma[co] / sqrt(rvar[co] + eps);
        for (long long t = 0; t < K; ++t) w_folded[(size_t)co * K + t] = s * w[(size_t)co * K + t];
        bias_folded[co] = beta[co] - rmean[co] * s;
    }
}
