/*
 * PruneTrain hot-path ORACLE  --  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of what the GPU library computes. It shares
 * no code, header, table or helper with the CUDA path and must never be called
 * from it. Only the tests, the smoke check and the bench's cpu_baseline /
 * reference legs execute it.
 *
 * Every function is the textbook definition of its operation written out as
 * nested loops (OpenMP over one outer independent loop, nothing else: no
 * blocking, no reordering, no fusion).
 *
 * Layouts (all dense, host memory):
 *   activations  x  [N][H][W][C]      (channels innermost)
 *   outputs      y  [N][P][Q][K]
 *   weights      w  [K][R][S][C]
 * with P = floor((H + 2*pad - R)/stride) + 1 and Q likewise from W and S.
 *
 * Paper passages followed:
 *   conv forward / backward          Sec. 2.1 (convolution layers), Eq. 4 (weight gradient)
 *   group-lasso regulariser          Eq. 1, Eq. 2
 *   optimiser                        Algorithm 1 (Optimizer step), momentum SGD
 *   threshold zeroing                Sec. 4.1 ("threshold of 1e-4"), Sec. 4.2 / Fig. 4 (max-abs per channel)
 *   gather of surviving channels     Sec. 4.2 (the surviving channels keep their weights and momentum unchanged)
 *
 * Parity pins: every function below is pinned by tests/test_oracle_*.py
 * (closed forms, adjoint identities, finite differences, hand examples,
 * brute force). Learning dynamics (accuracy, how many channels die) are
 * "parity unpinned": they need the datasets and are out of scope.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int pto_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Round an fp32 value to the nearest bf16 (ties to even) and widen to fp64.
 * bf16 keeps the top 16 bits of the fp32 pattern. NaN stays NaN. */
static double bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u && (u & 0x007fffffu)) {
        u |= 0x00400000u;               /* quiet NaN, keep it NaN */
        u &= 0xffff0000u;
    } else {
        uint32_t lsb = (u >> 16) & 1u;
        u += 0x7fffu + lsb;
        u &= 0xffff0000u;
    }
    float r;
    memcpy(&r, &u, 4);
    return (double)r;
}

void pto_round_bf16(const float *in, double *out, size_t n)
{
    for (size_t i = 0; i < n; ++i) out[i] = bf16_rne(in[i]);
}

/* bf16-round a whole tensor once and widen it, so the loops below are pure fp64. */
static double *widen_bf16(const float *in, size_t n)
{
    double *d = (double *)malloc((n ? n : 1) * sizeof(double));
    if (d) for (size_t i = 0; i < n; ++i) d[i] = bf16_rne(in[i]);
    return d;
}

static int out_dim(int H, int R, int stride, int pad)
{
    int t = H + 2 * pad - R;
    if (t < 0) return 0;
    return t / stride + 1;
}

int pto_out_dim(int H, int R, int stride, int pad) { return out_dim(H, R, stride, pad); }

/* ------------------------------------------------------------------ conv */
/* Forward (cross-correlation, zero outside the image, no bias):
 *   y[n,p,q,k] = sum_{r,s,c} x[n, p*stride-pad+r, q*stride-pad+s, c] * w[k,r,s,c]
 * Inputs are rounded to bf16 first (the GPU path's operand precision) and
 * everything after that is fp64. */
int pto_conv_fwd(const float *x, const float *w, double *y,
                 int N, int H, int W, int C, int K, int R, int S, int stride, int pad)
{
    const int P = out_dim(H, R, stride, pad), Q = out_dim(W, S, stride, pad);
    if (P <= 0 || Q <= 0) return 1;
    double *xd = widen_bf16(x, (size_t)N * H * W * C), *wd = widen_bf16(w, (size_t)K * R * S * C);
    if (!xd || !wd) { free(xd); free(wd); return 2; }
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int k = 0; k < K; ++k) {
                    double acc = 0.0;
                    for (int r = 0; r < R; ++r) {
                        const int h = p * stride - pad + r;
                        if (h < 0 || h >= H) continue;
                        for (int s = 0; s < S; ++s) {
                            const int ww = q * stride - pad + s;
                            if (ww < 0 || ww >= W) continue;
                            const double *xp = xd + (((size_t)n * H + h) * W + ww) * C;
                            const double *wp = wd + (((size_t)k * R + r) * S + s) * C;
                            for (int c = 0; c < C; ++c) acc += xp[c] * wp[c];
                        }
                    }
                    y[(((size_t)n * P + p) * Q + q) * K + k] = acc;
                }
    free(xd); free(wd);
    return 0;
}

/* Data gradient, scatter form of the forward's adjoint:
 *   for every (n,p,q,k,r,s,c): dx[n, p*stride-pad+r, q*stride-pad+s, c] += dy[n,p,q,k] * w[k,r,s,c]
 * Input pixels no tap reaches stay exactly 0. */
int pto_conv_dgrad(const float *dy, const float *w, double *dx,
                   int N, int H, int W, int C, int K, int R, int S, int stride, int pad)
{
    const int P = out_dim(H, R, stride, pad), Q = out_dim(W, S, stride, pad);
    if (P <= 0 || Q <= 0) return 1;
    double *gd = widen_bf16(dy, (size_t)N * P * Q * K), *wd = widen_bf16(w, (size_t)K * R * S * C);
    if (!gd || !wd) { free(gd); free(wd); return 2; }
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        double *dxn = dx + (size_t)n * H * W * C;
        for (size_t i = 0; i < (size_t)H * W * C; ++i) dxn[i] = 0.0;
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q)
                for (int k = 0; k < K; ++k) {
                    const double g = gd[(((size_t)n * P + p) * Q + q) * K + k];
                    for (int r = 0; r < R; ++r) {
                        const int h = p * stride - pad + r;
                        if (h < 0 || h >= H) continue;
                        for (int s = 0; s < S; ++s) {
                            const int ww = q * stride - pad + s;
                            if (ww < 0 || ww >= W) continue;
                            double *dp = dxn + ((size_t)h * W + ww) * C;
                            const double *wp = wd + (((size_t)k * R + r) * S + s) * C;
                            for (int c = 0; c < C; ++c) dp[c] += g * wp[c];
                        }
                    }
                }
    }
    free(gd); free(wd);
    return 0;
}

/* Weight gradient (Eq. 4), plain sum over the batch and all output pixels:
 *   dw[k,r,s,c] = sum_{n,p,q} dy[n,p,q,k] * x[n, p*stride-pad+r, q*stride-pad+s, c] */
int pto_conv_wgrad(const float *x, const float *dy, double *dw,
                   int N, int H, int W, int C, int K, int R, int S, int stride, int pad)
{
    const int P = out_dim(H, R, stride, pad), Q = out_dim(W, S, stride, pad);
    if (P <= 0 || Q <= 0) return 1;
    double *xd = widen_bf16(x, (size_t)N * H * W * C), *gd = widen_bf16(dy, (size_t)N * P * Q * K);
    if (!xd || !gd) { free(xd); free(gd); return 2; }
#pragma omp parallel for collapse(2) schedule(static)
    for (int k = 0; k < K; ++k)
        for (int r = 0; r < R; ++r)
            for (int s = 0; s < S; ++s)
                for (int c = 0; c < C; ++c) {
                    double acc = 0.0;
                    for (int n = 0; n < N; ++n)
                        for (int p = 0; p < P; ++p) {
                            const int h = p * stride - pad + r;
                            if (h < 0 || h >= H) continue;
                            for (int q = 0; q < Q; ++q) {
                                const int ww = q * stride - pad + s;
                                if (ww < 0 || ww >= W) continue;
                                acc += gd[(((size_t)n * P + p) * Q + q) * K + k] *
                                       xd[(((size_t)n * H + h) * W + ww) * C + c];
                            }
                        }
                    dw[(((size_t)k * R + r) * S + s) * C + c] = acc;
                }
    free(xd); free(gd);
    return 0;
}

/* One-element versions, for checking sampled outputs of full-size problems.
 * idx[i] is the flat index into the dense output tensor of the matching
 * full function; each element is the same defining sum, evaluated alone. */
int pto_conv_fwd_samples(const float *x, const float *w, const int64_t *idx, int64_t n_idx, double *out,
                         int N, int H, int W, int C, int K, int R, int S, int stride, int pad)
{
    const int P = out_dim(H, R, stride, pad), Q = out_dim(W, S, stride, pad);
    if (P <= 0 || Q <= 0) return 1;
    (void)N;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t i = 0; i < n_idx; ++i) {
        int64_t t = idx[i];
        const int k = (int)(t % K); t /= K;
        const int q = (int)(t % Q); t /= Q;
        const int p = (int)(t % P); t /= P;
        const int n = (int)t;
        double acc = 0.0;
        for (int r = 0; r < R; ++r) {
            const int h = p * stride - pad + r;
            if (h < 0 || h >= H) continue;
            for (int s = 0; s < S; ++s) {
                const int ww = q * stride - pad + s;
                if (ww < 0 || ww >= W) continue;
                const float *xp = x + (((size_t)n * H + h) * W + ww) * C;
                const float *wp = w + (((size_t)k * R + r) * S + s) * C;
                for (int c = 0; c < C; ++c) acc += bf16_rne(xp[c]) * bf16_rne(wp[c]);
            }
        }
        out[i] = acc;
    }
    return 0;
}

/* dx[n,h,w,c] = sum over (p,r) with p*stride-pad+r == h, (q,s) with q*stride-pad+s == w, and k. */
int pto_conv_dgrad_samples(const float *dy, const float *w, const int64_t *idx, int64_t n_idx, double *out,
                           int N, int H, int W, int C, int K, int R, int S, int stride, int pad)
{
    const int P = out_dim(H, R, stride, pad), Q = out_dim(W, S, stride, pad);
    if (P <= 0 || Q <= 0) return 1;
    (void)N;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t i = 0; i < n_idx; ++i) {
        int64_t t = idx[i];
        const int c = (int)(t % C); t /= C;
        const int ww = (int)(t % W); t /= W;
        const int h = (int)(t % H); t /= H;
        const int n = (int)t;
        double acc = 0.0;
        for (int p = 0; p < P; ++p) {
            const int r = h - (p * stride - pad);
            if (r < 0 || r >= R) continue;
            for (int q = 0; q < Q; ++q) {
                const int s = ww - (q * stride - pad);
                if (s < 0 || s >= S) continue;
                const float *dyp = dy + (((size_t)n * P + p) * Q + q) * K;
                for (int k = 0; k < K; ++k)
                    acc += bf16_rne(dyp[k]) * bf16_rne(w[(((size_t)k * R + r) * S + s) * C + c]);
            }
        }
        out[i] = acc;
    }
    return 0;
}

int pto_conv_wgrad_samples(const float *x, const float *dy, const int64_t *idx, int64_t n_idx, double *out,
                           int N, int H, int W, int C, int K, int R, int S, int stride, int pad)
{
    const int P = out_dim(H, R, stride, pad), Q = out_dim(W, S, stride, pad);
    if (P <= 0 || Q <= 0) return 1;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < n_idx; ++i) {
        int64_t t = idx[i];
        const int c = (int)(t % C); t /= C;
        const int s = (int)(t % S); t /= S;
        const int r = (int)(t % R); t /= R;
        const int k = (int)t;
        double acc = 0.0;
        for (int n = 0; n < N; ++n)
            for (int p = 0; p < P; ++p) {
                const int h = p * stride - pad + r;
                if (h < 0 || h >= H) continue;
                for (int q = 0; q < Q; ++q) {
                    const int ww = q * stride - pad + s;
                    if (ww < 0 || ww >= W) continue;
                    acc += bf16_rne(dy[(((size_t)n * P + p) * Q + q) * K + k]) *
                           bf16_rne(x[(((size_t)n * H + h) * W + ww) * C + c]);
                }
            }
        out[i] = acc;
    }
    return 0;
}

/* ------------------------------------------------- group lasso + SGD */
/* Per layer, weights w[K][RS][C] (fp32 widened to fp64):
 *   s_out[k] = sum_{rs,c} w^2          (output-channel group, Eq. 2 second sum)
 *   s_in[c]  = sum_{k,rs} w^2          (input-channel group,  Eq. 2 first sum)
 *   d R / d w = w * ( [reg_out][s_out>tiny]/sqrt(s_out[k]) + [reg_in][s_in>tiny]/sqrt(s_in[c]) )
 *   g~ = g + wd*w + lambda * dR/dw     (Eq. 1: the regulariser is part of the loss)
 *   v' = mu*v + g~ ;  w' = w - lr*v'   (momentum SGD, dampening 0, no Nesterov)
 * The subgradient of an all-zero group is taken as 0 (guard: sumsq > 1e-24).
 * reg_sum gets sum_k sqrt(s_out) + sum_c sqrt(s_in) over the regularised groups
 * (Eq. 2 without lambda), from the PRE-update weights (Algorithm 1: GroupLassoReg(W_i)). */
void pto_lasso_sgd(const float *w, const float *g, const float *v,
                   int K, int C, int RS, int reg_in, int reg_out,
                   double lambda, double lr, double mu, double wd,
                   double *w_new, double *v_new, double *s_out, double *s_in, double *reg_sum)
{
    for (int k = 0; k < K; ++k) s_out[k] = 0.0;
    for (int c = 0; c < C; ++c) s_in[c] = 0.0;
    for (int k = 0; k < K; ++k)
        for (int rs = 0; rs < RS; ++rs)
            for (int c = 0; c < C; ++c) {
                const double a = (double)w[((size_t)k * RS + rs) * C + c];
                s_out[k] += a * a;
                s_in[c] += a * a;
            }
    double reg = 0.0;
    if (reg_out) for (int k = 0; k < K; ++k) reg += sqrt(s_out[k]);
    if (reg_in)  for (int c = 0; c < C; ++c) reg += sqrt(s_in[c]);
    *reg_sum = reg;
    for (int k = 0; k < K; ++k)
        for (int rs = 0; rs < RS; ++rs)
            for (int c = 0; c < C; ++c) {
                const size_t i = ((size_t)k * RS + rs) * C + c;
                const double a = (double)w[i];
                double term = 0.0;
                if (reg_out && s_out[k] > 1e-24) term += 1.0 / sqrt(s_out[k]);
                if (reg_in && s_in[c] > 1e-24) term += 1.0 / sqrt(s_in[c]);
                const double gt = (double)g[i] + wd * a + lambda * a * term;
                const double vn = mu * (double)v[i] + gt;
                v_new[i] = vn;
                w_new[i] = a - lr * vn;
            }
}

/* ------------------------------------------------ zero-group detection */
/* A group is "zero" iff every member satisfies |w| < thr, compared in fp32
 * (strict <; a NaN member fails the comparison, so the group is kept). */
void pto_find_zero_groups(const float *w, int K, int C, int RS, float thr,
                          uint8_t *zero_out, uint8_t *zero_in)
{
    for (int k = 0; k < K; ++k) {
        int all = 1;
        for (int rs = 0; rs < RS && all; ++rs)
            for (int c = 0; c < C; ++c)
                if (!(fabsf(w[((size_t)k * RS + rs) * C + c]) < thr)) { all = 0; break; }
        zero_out[k] = (uint8_t)all;
    }
    for (int c = 0; c < C; ++c) {
        int all = 1;
        for (int k = 0; k < K && all; ++k)
            for (int rs = 0; rs < RS; ++rs)
                if (!(fabsf(w[((size_t)k * RS + rs) * C + c]) < thr)) { all = 0; break; }
        zero_in[c] = (uint8_t)all;
    }
}

/* --------------------------------------------------------------- gather */
/* new[k',rs,c'] = old[mapK[k'], rs, mapC[c']]  -- a copy, bit for bit. */
void pto_gather_f32(const float *old, int C_old, int RS,
                    const int32_t *mapK, int K_new, const int32_t *mapC, int C_new, float *out)
{
    for (int k = 0; k < K_new; ++k)
        for (int rs = 0; rs < RS; ++rs)
            for (int c = 0; c < C_new; ++c)
                out[((size_t)k * RS + rs) * C_new + c] =
                    old[((size_t)mapK[k] * RS + rs) * C_old + mapC[c]];
}
