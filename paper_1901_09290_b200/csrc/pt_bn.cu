// Batch normalisation + residual add + ReLU on ragged channel counts, forward and backward (Sec. 2.1: the normalisation
// layers read their inputs several times and are bound by memory bandwidth). NHWC bf16 activations with channel pitch ld,
// fp32 statistics and parameters. Four streaming kernels and two small finishing kernels:
//   forward : reduce (per-channel sum and sum of squares about a pivot) -> finish (mean, 1/std, moving statistics)
//             -> apply (y = relu(gamma*xhat + beta + residual))
//   backward: reduce (dbeta = sum dz, dgamma = sum dz*xhat) -> finish -> apply (dx, dresidual)
// The tensor is one contiguous array of 16-byte vectors (8 channels each); a thread keeps one vector column and walks
// the pixels, so a warp always reads consecutive vectors whatever the channel count is. Partial sums are combined in a
// fixed order (run-to-run identical); no atomics.
#include "pt_internal.h"

namespace {

constexpr int kBnThreads = 256;
constexpr int kBnMaxBlocks = 148 * 4;

struct BnP {
    long long M;            // pixels
    int C, ld, LV;          // channels, pitch, vectors per pixel (ld / 8)
    int ppb;                // pixels a block covers per iteration (kBnThreads / LV)
    int blocks;             // blocks of the reduce kernels
    long long chunk;        // pixels per block (multiple of ppb)
    float eps, momentum;
    int relu;
};

__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8])
{
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 t = __bfloat1622float2(h[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}

__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    uint4 v;
    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return v;
}

// MODE 0: a0 = sum(x - pivot), a1 = sum((x - pivot)^2), pivot = the channel's value at pixel 0 (keeps the variance free of
//         the cancellation a large mean would cause in sum(x^2) - sum(x)^2/M).
// MODE 1: a0 = sum(dz), a1 = sum(dz * xhat), dz = dy where y > 0 (ReLU) else 0.
// partial layout: [block][2][LV*8] floats.
template <int MODE>
__global__ void __launch_bounds__(kBnThreads) bn_reduce_kernel(const BnP p, const uint4 *__restrict__ x, const uint4 *__restrict__ y,
                                                               const uint4 *__restrict__ dy, const float *__restrict__ mean,
                                                               const float *__restrict__ invstd, float *__restrict__ partial)
{
    __shared__ float red[kBnThreads][17];
    const int t = threadIdx.x;
    const int cv = t % p.LV, pr = t / p.LV;
    const bool active = pr < p.ppb;
    float a0[8], a1[8], piv[8], mu[8], is[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { a0[j] = 0.f; a1[j] = 0.f; piv[j] = 0.f; mu[j] = 0.f; is[j] = 0.f; }
    if (active) {
        if (MODE == 0) {
            unpack8(x[cv], piv);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int c = cv * 8 + j;
                if (c < p.C) { mu[j] = mean[c]; is[j] = invstd[c]; }
            }
        }
        const long long m0 = (long long)blockIdx.x * p.chunk;
        const long long m1 = m0 + p.chunk < p.M ? m0 + p.chunk : p.M;
        constexpr int U = MODE == 0 ? 4 : 2;          // pixels per iteration: all their loads are issued before any arithmetic
        for (long long m = m0 + pr; m < m1; m += (long long)U * p.ppb) {
            uint4 vx[U], vg[U], vy[U];
            bool live[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long mu_ = m + (long long)u * p.ppb;
                live[u] = mu_ < m1;
                const size_t i = (size_t)(live[u] ? mu_ : m) * p.LV + cv;
                vx[u] = x[i];
                if (MODE == 1) { vg[u] = dy[i]; vy[u] = y[i]; }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float xv[8];
                unpack8(vx[u], xv);
                if (MODE == 0) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float dd = live[u] ? xv[j] - piv[j] : 0.f;
                        a0[j] += dd; a1[j] += dd * dd;
                    }
                } else {
                    float dv[8], fv[8];
                    unpack8(vg[u], dv);
                    unpack8(vy[u], fv);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float z = (live[u] && (!p.relu || fv[j] > 0.f)) ? dv[j] : 0.f;
                        a0[j] += z; a1[j] += z * ((xv[j] - mu[j]) * is[j]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) { red[t][j] = a0[j]; red[t][8 + j] = a1[j]; }
    __syncthreads();
    // thread (cv, j) with t < LV*... : each of the first LV threads sums its column over the pixel rows, in order
    if (t < p.LV) {
        float s[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) s[j] = 0.f;
        for (int r = 0; r < p.ppb; ++r)
#pragma unroll
            for (int j = 0; j < 16; ++j) s[j] += red[r * p.LV + t][j];
        float *dst = partial + (size_t)blockIdx.x * 2 * p.ld;
#pragma unroll
        for (int j = 0; j < 8; ++j) { dst[t * 8 + j] = s[j]; dst[p.ld + t * 8 + j] = s[8 + j]; }
    }
}

// Sums the block partials of kFinC channels per CTA: thread (tx, ty) adds the rows ty, ty + kFinS, ... of channel tx in ascending
// order in fp64 (eight loads in flight: a chain of dependent L2 loads is what costs time here), then the kFinS slices are added
// in a fixed order in two steps. 8 channels x 128 slices: a convolution's epilogue warps leave up to 1776 rows, 14 per slice
// (32 channels x 32 slices took 9 us per call, 55 rows per slice). Returns the two sums to the threads with ty == 0.
constexpr int kFinC = 8, kFinS = 128;
__device__ __forceinline__ bool bn_sum_partials(const BnP &p, const float *__restrict__ partial, int c, double &s0, double &s1)
{
    __shared__ double sh[2][kFinS][kFinC];
    __shared__ double sh2[2][16][kFinC];
    const int tx = threadIdx.x & (kFinC - 1), ty = threadIdx.x / kFinC;
    double a0 = 0.0, a1 = 0.0;
    if (c < p.C) {
        int b = ty;
        for (; b + 7 * kFinS < p.blocks; b += 8 * kFinS) {
            float v0[8], v1[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                v0[u] = partial[(size_t)(b + kFinS * u) * 2 * p.ld + c];
                v1[u] = partial[(size_t)(b + kFinS * u) * 2 * p.ld + p.ld + c];
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) { a0 += (double)v0[u]; a1 += (double)v1[u]; }
        }
        {
            // the remaining rows (fewer than eight): loaded together, added in the same ascending order
            float v0[8], v1[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int bb = b + kFinS * u;
                v0[u] = bb < p.blocks ? partial[(size_t)bb * 2 * p.ld + c] : 0.f;
                v1[u] = bb < p.blocks ? partial[(size_t)bb * 2 * p.ld + p.ld + c] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (b + kFinS * u < p.blocks) { a0 += (double)v0[u]; a1 += (double)v1[u]; }
        }
    }
    sh[0][ty][tx] = a0;
    sh[1][ty][tx] = a1;
    __syncthreads();
    if (ty < 16) {
        double t0 = 0.0, t1 = 0.0;
#pragma unroll
        for (int r = 0; r < kFinS / 16; ++r) { t0 += sh[0][ty * (kFinS / 16) + r][tx]; t1 += sh[1][ty * (kFinS / 16) + r][tx]; }
        sh2[0][ty][tx] = t0;
        sh2[1][ty][tx] = t1;
    }
    __syncthreads();
    if (ty != 0 || c >= p.C) return false;
    s0 = 0.0; s1 = 0.0;
#pragma unroll
    for (int r = 0; r < 16; ++r) { s0 += sh2[0][r][tx]; s1 += sh2[1][r][tx]; }
    return true;
}

__global__ void __launch_bounds__(1024) bn_fwd_finish_kernel(const BnP p, const __nv_bfloat16 *__restrict__ x, const float *__restrict__ partial,
                                                            float *__restrict__ save_mean, float *__restrict__ save_invstd,
                                                            float *__restrict__ running_mean, float *__restrict__ running_var)
{
    const int c = blockIdx.x * kFinC + (threadIdx.x & (kFinC - 1));
    double s0, s1;
    if (!bn_sum_partials(p, partial, c, s0, s1)) return;
    const double M = (double)p.M;
    const double d = s0 / M;
    double var = s1 / M - d * d;
    if (var < 0.0) var = 0.0;
    const double mean = (x ? (double)__bfloat162float(x[c]) : 0.0) + d;     // sums about a pivot (the channel's first value) or about 0
    save_mean[c] = (float)mean;
    save_invstd[c] = (float)(1.0 / sqrt(var + (double)p.eps));
    if (running_mean && running_var) {
        const double mom = (double)p.momentum;
        running_mean[c] = (float)((1.0 - mom) * (double)running_mean[c] + mom * mean);
        running_var[c] = (float)((1.0 - mom) * (double)running_var[c] + mom * var * (p.M > 1 ? M / (M - 1.0) : 1.0));
    }
}

__global__ void __launch_bounds__(1024) bn_bwd_finish_kernel(const BnP p, const float *__restrict__ partial, float *__restrict__ dgamma,
                                                            float *__restrict__ dbeta)
{
    const int c = blockIdx.x * kFinC + (threadIdx.x & (kFinC - 1));
    double s0, s1;
    if (!bn_sum_partials(p, partial, c, s0, s1)) return;
    dbeta[c] = (float)s0;
    dgamma[c] = (float)s1;
}

// MODE 0: y = relu(x*scale + shift + residual), scale = gamma*invstd, shift = beta - mean*scale.
// MODE 1: dz = dy where y > 0; dresidual = dz; dx = gamma*invstd * (dz - dbeta/M - xhat*dgamma/M).
// Pad lanes (channel >= C) of the outputs are written as zeros.
template <int MODE>
__global__ void __launch_bounds__(kBnThreads) bn_apply_kernel(const BnP p, const uint4 *__restrict__ x, const uint4 *__restrict__ y_in,
                                                              const uint4 *__restrict__ aux /* residual | dy */,
                                                              const float *__restrict__ gamma, const float *__restrict__ beta,
                                                              const float *__restrict__ mean, const float *__restrict__ invstd,
                                                              const float *__restrict__ dgamma, const float *__restrict__ dbeta,
                                                              uint4 *__restrict__ out, uint4 *__restrict__ out2 /* dresidual */)
{
    const int t = threadIdx.x;
    const int cv = t % p.LV, pr = t / p.LV;
    if (pr >= p.ppb) return;
    float k0[8], k1[8], k2[8];       // MODE 0: scale, shift, valid ; MODE 1: gamma*invstd, mean, invstd*dgamma/M (k3 = dbeta/M below)
    float k3[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int c = cv * 8 + j;
        const bool ok = c < p.C;
        if (MODE == 0) {
            const float sc = ok ? gamma[c] * invstd[c] : 0.f;
            k0[j] = sc;
            k1[j] = ok ? beta[c] - mean[c] * sc : 0.f;
            k2[j] = ok ? 1.f : 0.f;
            k3[j] = 0.f;
        } else {
            const float is = ok ? invstd[c] : 0.f;
            k0[j] = ok ? gamma[c] * is : 0.f;
            k1[j] = ok ? mean[c] : 0.f;
            k2[j] = ok ? is * dgamma[c] / (float)p.M : 0.f;      // xhat * dgamma / M = (x - mean) * (invstd * dgamma / M)
            k3[j] = ok ? dbeta[c] / (float)p.M : 0.f;
        }
    }
    const long long m0 = (long long)blockIdx.x * p.chunk;
    const long long m1 = m0 + p.chunk < p.M ? m0 + p.chunk : p.M;
    for (long long m = m0 + pr; m < m1; m += 2 * p.ppb) {
        const bool two = m + p.ppb < m1;
        const size_t i0 = (size_t)m * p.LV + cv, i1 = two ? (size_t)(m + p.ppb) * p.LV + cv : i0;
        // both pixels' loads go out before any arithmetic
        uint4 vx[2], va[2], vy[2];
        vx[0] = x[i0]; vx[1] = x[i1];
        if (aux) { va[0] = aux[i0]; va[1] = aux[i1]; }
        if (MODE == 1) { vy[0] = y_in[i0]; vy[1] = y_in[i1]; }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (u == 1 && !two) break;
            const size_t i = u ? i1 : i0;
            float xv[8], av[8], r[8];
            unpack8(vx[u], xv);
            if (MODE == 0) {
                if (aux) unpack8(va[u], av);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float z = xv[j] * k0[j] + k1[j];
                    if (aux) z += av[j];
                    if (p.relu) z = fmaxf(z, 0.f);
                    r[j] = k2[j] != 0.f ? z : 0.f;
                }
                out[i] = pack8(r);
            } else {
                float yv[8], dz[8];
                unpack8(va[u], av);
                unpack8(vy[u], yv);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const bool ok = cv * 8 + j < p.C;       // pad lanes may hold anything, NaN included: never let them through
                    dz[j] = ok ? ((!p.relu || yv[j] > 0.f) ? av[j] : 0.f) : 0.f;
                    r[j] = ok ? k0[j] * (dz[j] - k3[j] - (xv[j] - k1[j]) * k2[j]) : 0.f;
                }
                out[i] = pack8(r);
                if (out2) out2[i] = pack8(dz);
            }
        }
    }
}

pt_status bn_params(const pt_ctx *c, const pt_bn_desc *d, BnP *p)
{
    if (!c || !d) return PT_ERR_INVALID_ARG;
    if (d->N < 1 || d->H < 1 || d->W < 1 || d->C < 1 || d->ld < d->C || (d->ld & 7)) return PT_ERR_INVALID_ARG;
    if (!(d->eps >= 0.f) || !(d->momentum >= 0.f && d->momentum <= 1.f)) return PT_ERR_INVALID_ARG;
    if (d->ld > 8 * kBnThreads) return PT_ERR_UNSUPPORTED;
    memset(p, 0, sizeof(*p));
    p->M = (long long)d->N * d->H * d->W;
    p->C = d->C; p->ld = d->ld; p->LV = d->ld / 8;
    p->ppb = kBnThreads / p->LV;
    p->eps = d->eps; p->momentum = d->momentum; p->relu = d->relu ? 1 : 0;
    // at least 4 of a block's pixel rows per block, at most kBnMaxBlocks blocks (four per SM)
    long long blocks = (p->M + (long long)p->ppb * 4 - 1) / ((long long)p->ppb * 4);
    if (blocks > kBnMaxBlocks) blocks = kBnMaxBlocks;
    if (blocks < 1) blocks = 1;
    long long chunk = (p->M + blocks - 1) / blocks;
    chunk = (chunk + p->ppb - 1) / p->ppb * p->ppb;
    p->chunk = chunk;
    p->blocks = (int)((p->M + chunk - 1) / chunk);
    return PT_OK;
}

}  // namespace

extern "C" size_t pt_bn_workspace_bytes(const pt_ctx *c, const pt_bn_desc *d)
{
    BnP p;
    if (bn_params(c, d, &p) != PT_OK) return 0;
    return (size_t)p.blocks * 2 * p.ld * sizeof(float);
}

static bool aligned16(const void *q) { return ((uintptr_t)q & 15) == 0; }

extern "C" pt_status pt_bn_relu_fwd(pt_ctx *c, const pt_bn_desc *d, const void *x, const void *residual, const float *gamma,
                                    const float *beta, float *running_mean, float *running_var, float *save_mean,
                                    float *save_invstd, void *y, void *ws, size_t ws_bytes, void *stream)
{
    BnP p;
    pt_status r = bn_params(c, d, &p);
    if (r != PT_OK) return r;
    if (!x || !gamma || !beta || !save_mean || !save_invstd || !y || (running_mean == nullptr) != (running_var == nullptr))
        return PT_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y) || (residual && !aligned16(residual))) return PT_ERR_INVALID_ARG;
    if (!ws || ws_bytes < pt_bn_workspace_bytes(c, d)) return PT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    float *partial = (float *)ws;
    bn_reduce_kernel<0><<<p.blocks, kBnThreads, 0, st>>>(p, (const uint4 *)x, nullptr, nullptr, nullptr, nullptr, partial);
    bn_fwd_finish_kernel<<<pt_ceil_div(p.C, kFinC), kFinC * kFinS, 0, st>>>(p, (const __nv_bfloat16 *)x, partial, save_mean, save_invstd, running_mean,
                                                               running_var);
    bn_apply_kernel<0><<<p.blocks, kBnThreads, 0, st>>>(p, (const uint4 *)x, nullptr, (const uint4 *)residual, gamma, beta, save_mean,
                                                        save_invstd, nullptr, nullptr, (uint4 *)y, nullptr);
    c->launches += 3;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

extern "C" pt_status pt_bn_relu_bwd(pt_ctx *c, const pt_bn_desc *d, const void *x, const void *y, const void *dy, const float *gamma,
                                    const float *save_mean, const float *save_invstd, void *dx, void *dresidual, float *dgamma,
                                    float *dbeta, void *ws, size_t ws_bytes, void *stream)
{
    BnP p;
    pt_status r = bn_params(c, d, &p);
    if (r != PT_OK) return r;
    if (!x || !dy || !gamma || !save_mean || !save_invstd || !dx || !dgamma || !dbeta || (p.relu && !y)) return PT_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dx) || (y && !aligned16(y)) || (dresidual && !aligned16(dresidual)))
        return PT_ERR_INVALID_ARG;
    if (!ws || ws_bytes < pt_bn_workspace_bytes(c, d)) return PT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    float *partial = (float *)ws;
    const uint4 *yv = (const uint4 *)(y ? y : dy);          // without ReLU the mask input is never looked at
    bn_reduce_kernel<1><<<p.blocks, kBnThreads, 0, st>>>(p, (const uint4 *)x, yv, (const uint4 *)dy, save_mean, save_invstd, partial);
    bn_bwd_finish_kernel<<<pt_ceil_div(p.C, kFinC), kFinC * kFinS, 0, st>>>(p, partial, dgamma, dbeta);
    bn_apply_kernel<1><<<p.blocks, kBnThreads, 0, st>>>(p, (const uint4 *)x, yv, (const uint4 *)dy, gamma, nullptr, save_mean, save_invstd,
                                                        dgamma, dbeta, (uint4 *)dx, (uint4 *)dresidual);
    c->launches += 3;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

// The forward pass when the convolution that produced x already took the channel sums (pt_conv_fwd_stats): no reduction pass
// over x, only the short finish over the convolution's rows of partial sums and the apply pass.
extern "C" pt_status pt_bn_relu_fwd_stats(pt_ctx *c, const pt_bn_desc *d, const void *x, const void *residual, const float *gamma,
                                          const float *beta, float *running_mean, float *running_var, float *save_mean,
                                          float *save_invstd, void *y, const float *stats, int32_t n_parts, void *stream)
{
    BnP p;
    pt_status r = bn_params(c, d, &p);
    if (r != PT_OK) return r;
    if (!x || !gamma || !beta || !save_mean || !save_invstd || !y || !stats || n_parts < 1 ||
        (running_mean == nullptr) != (running_var == nullptr))
        return PT_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y) || (residual && !aligned16(residual))) return PT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    BnP pf = p;
    pf.blocks = n_parts;                            // rows of [2][ld] partial sums, taken about 0
    bn_fwd_finish_kernel<<<pt_ceil_div(p.C, kFinC), kFinC * kFinS, 0, st>>>(pf, nullptr, stats, save_mean, save_invstd, running_mean, running_var);
    bn_apply_kernel<0><<<p.blocks, kBnThreads, 0, st>>>(p, (const uint4 *)x, nullptr, (const uint4 *)residual, gamma, beta, save_mean,
                                                        save_invstd, nullptr, nullptr, (uint4 *)y, nullptr);
    c->launches += 2;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}
