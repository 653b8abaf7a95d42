// Max pooling on ragged channel counts, forward and backward (Sec. 2.1 lists the pooling layers among the cheap, bandwidth-
// bound layers of a CNN; ResNet has one, after the stem). It is here so that a training step can be chained from the image to
// the last feature map; NHWC bf16 activations with channel pitch ld, one 16-byte vector (8 channels) per thread.
//   forward : y[n,p,q,c] = max over the window of x[n, p*stride - pad + r, q*stride - pad + s, c]; positions outside the image
//             are never selected; of equal maxima the first in scan order (r, then s) is the selected one.
//   backward: dx[n,h,w,c] = sum of dy[n,p,q,c] over the windows whose selected position is (h,w). Each input position lies in
//             at most ceil(R/stride)^2 windows; the thread of an input position looks at those windows, so nothing is added
//             atomically (run-to-run identical). The selections come from the index tensor the forward pass can leave (one
//             byte per output element: the selected position r*R + s of the window, 255 where no position was valid), or are
//             recomputed from x when there is none (R*R loads per window instead of one: 644 us against 70 us for the
//             pooling after the ResNet-50 stem at batch 64).
#include "pt_internal.h"

namespace {

struct PoolP { int N, H, W, C, ld, LV, R, stride, pad, P, Q; };

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

// Maximum and the scan-order index of its first occurrence, per channel, of the window of output position (p, q).
__device__ __forceinline__ void window_max(const PoolP &p, const uint4 *__restrict__ x, int n, int po, int qo, int cv, float (&m)[8], int (&at)[8])
{
#pragma unroll
    for (int j = 0; j < 8; ++j) { m[j] = -INFINITY; at[j] = -1; }
    for (int r = 0; r < p.R; ++r) {
        const int h = po * p.stride - p.pad + r;
        if (h < 0 || h >= p.H) continue;
        for (int s = 0; s < p.R; ++s) {
            const int w = qo * p.stride - p.pad + s;
            if (w < 0 || w >= p.W) continue;
            float f[8];
            unpack8(x[((size_t)(n * p.H + h) * p.W + w) * p.LV + cv], f);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (f[j] > m[j] || at[j] < 0) { m[j] = f[j]; at[j] = h * p.W + w; }     // strictly greater: the first maximum stays
        }
    }
}

__global__ void __launch_bounds__(256) maxpool_fwd_kernel(const PoolP p, const uint4 *__restrict__ x, uint4 *__restrict__ y,
                                                          uint2 *__restrict__ index)
{
    const size_t total = (size_t)p.N * p.P * p.Q * p.LV;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int cv = (int)(i % p.LV);
        size_t t = i / p.LV;
        const int q = (int)(t % p.Q); t /= p.Q;
        const int po = (int)(t % p.P), n = (int)(t / p.P);
        float m[8];
        int at[8];
        window_max(p, x, n, po, q, cv, m, at);
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (cv * 8 + j >= p.C || at[j] < 0) m[j] = 0.f;
        y[i] = pack8(m);
        if (index) {
            // the selected position inside the window, one byte per channel
            unsigned b[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                b[j] = 255u;
                if (cv * 8 + j < p.C && at[j] >= 0) {
                    const int h = at[j] / p.W, w = at[j] - h * p.W;
                    b[j] = (unsigned)((h - (po * p.stride - p.pad)) * p.R + (w - (q * p.stride - p.pad)));
                }
            }
            index[i] = make_uint2(b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24), b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24));
        }
    }
}

// Backward from the stored selections: one 8-byte index vector and one 16-byte dy vector per window.
__global__ void __launch_bounds__(256) maxpool_bwd_index_kernel(const PoolP p, const uint2 *__restrict__ index,
                                                                const uint4 *__restrict__ dy, uint4 *__restrict__ dx)
{
    const size_t total = (size_t)p.N * p.H * p.W * p.LV;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int cv = (int)(i % p.LV);
        size_t t = i / p.LV;
        const int w = (int)(t % p.W); t /= p.W;
        const int h = (int)(t % p.H), n = (int)(t / p.H);
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.f;
        int p_lo = h + p.pad - p.R + 1;
        p_lo = p_lo <= 0 ? 0 : (p_lo + p.stride - 1) / p.stride;
        int p_hi = (h + p.pad) / p.stride;
        if (p_hi > p.P - 1) p_hi = p.P - 1;
        int q_lo = w + p.pad - p.R + 1;
        q_lo = q_lo <= 0 ? 0 : (q_lo + p.stride - 1) / p.stride;
        int q_hi = (w + p.pad) / p.stride;
        if (q_hi > p.Q - 1) q_hi = p.Q - 1;
        for (int po = p_lo; po <= p_hi; ++po)            // ascending windows: the order of the additions is fixed
            for (int q = q_lo; q <= q_hi; ++q) {
                const size_t o = ((size_t)(n * p.P + po) * p.Q + q) * p.LV + cv;
                const uint2 ix = index[o];
                float g[8];
                unpack8(dy[o], g);
                const unsigned me = (unsigned)((h - (po * p.stride - p.pad)) * p.R + (w - (q * p.stride - p.pad)));
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const unsigned b = ((j < 4 ? ix.x : ix.y) >> (8 * (j & 3))) & 255u;
                    if (b == me) acc[j] += g[j];
                }
            }
        dx[i] = pack8(acc);                              // pad lanes carry index 255: they stay zero
    }
}

__global__ void __launch_bounds__(256) maxpool_bwd_kernel(const PoolP p, const uint4 *__restrict__ x, const uint4 *__restrict__ dy,
                                                          uint4 *__restrict__ dx)
{
    const size_t total = (size_t)p.N * p.H * p.W * p.LV;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int cv = (int)(i % p.LV);
        size_t t = i / p.LV;
        const int w = (int)(t % p.W); t /= p.W;
        const int h = (int)(t % p.H), n = (int)(t / p.H);
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.f;
        // windows that contain (h, w): p*stride - pad <= h <= p*stride - pad + R - 1
        int p_lo = h + p.pad - p.R + 1;
        p_lo = p_lo <= 0 ? 0 : (p_lo + p.stride - 1) / p.stride;
        int p_hi = (h + p.pad) / p.stride;
        if (p_hi > p.P - 1) p_hi = p.P - 1;
        int q_lo = w + p.pad - p.R + 1;
        q_lo = q_lo <= 0 ? 0 : (q_lo + p.stride - 1) / p.stride;
        int q_hi = (w + p.pad) / p.stride;
        if (q_hi > p.Q - 1) q_hi = p.Q - 1;
        const int me = h * p.W + w;
        for (int po = p_lo; po <= p_hi; ++po)
            for (int q = q_lo; q <= q_hi; ++q) {
                float m[8], g[8];
                int at[8];
                window_max(p, x, n, po, q, cv, m, at);
                unpack8(dy[((size_t)(n * p.P + po) * p.Q + q) * p.LV + cv], g);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (at[j] == me) acc[j] += g[j];
            }
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (cv * 8 + j >= p.C) acc[j] = 0.f;
        dx[i] = pack8(acc);
    }
}

pt_status pool_params(const pt_ctx *c, const pt_pool_desc *d, PoolP *p)
{
    if (!c || !d) return PT_ERR_INVALID_ARG;
    if (d->N < 1 || d->H < 1 || d->W < 1 || d->C < 1 || d->ld < d->C || (d->ld & 7)) return PT_ERR_INVALID_ARG;
    if (d->R < 1 || d->stride < 1 || d->pad < 0 || d->pad >= d->R) return PT_ERR_INVALID_ARG;
    p->N = d->N; p->H = d->H; p->W = d->W; p->C = d->C; p->ld = d->ld; p->LV = d->ld / 8;
    p->R = d->R; p->stride = d->stride; p->pad = d->pad;
    p->P = pt_out_dim(d->H, d->R, d->stride, d->pad);
    p->Q = pt_out_dim(d->W, d->R, d->stride, d->pad);
    if (p->P < 1 || p->Q < 1) return PT_ERR_INVALID_ARG;
    if ((long long)d->N * d->H * d->W >= (1ll << 31)) return PT_ERR_UNSUPPORTED;
    return PT_OK;
}

unsigned pool_grid(const pt_ctx *c, size_t total)
{
    size_t b = (total + 255) / 256, cap = (size_t)c->sm_count * 16;
    return (unsigned)(b < cap ? (b ? b : 1) : cap);
}

}  // namespace

static bool pool_aligned16(const void *q) { return ((uintptr_t)q & 15) == 0; }

extern "C" pt_status pt_maxpool_fwd(pt_ctx *c, const pt_pool_desc *d, const void *x, void *y, void *index, void *stream)
{
    PoolP p;
    pt_status r = pool_params(c, d, &p);
    if (r != PT_OK) return r;
    if (!x || !y || !pool_aligned16(x) || !pool_aligned16(y)) return PT_ERR_INVALID_ARG;
    if (index && (((uintptr_t)index & 7) || p.R * p.R > 255)) return PT_ERR_INVALID_ARG;
    const size_t total = (size_t)p.N * p.P * p.Q * p.LV;
    maxpool_fwd_kernel<<<pool_grid(c, total), 256, 0, (cudaStream_t)stream>>>(p, (const uint4 *)x, (uint4 *)y, (uint2 *)index);
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

extern "C" pt_status pt_maxpool_bwd(pt_ctx *c, const pt_pool_desc *d, const void *x, const void *dy, const void *index, void *dx,
                                    void *stream)
{
    PoolP p;
    pt_status r = pool_params(c, d, &p);
    if (r != PT_OK) return r;
    if ((!x && !index) || !dy || !dx || (x && !pool_aligned16(x)) || !pool_aligned16(dy) || !pool_aligned16(dx)) return PT_ERR_INVALID_ARG;
    if (index && (((uintptr_t)index & 7) || p.R * p.R > 255)) return PT_ERR_INVALID_ARG;
    const size_t total = (size_t)p.N * p.H * p.W * p.LV;
    if (index)
        maxpool_bwd_index_kernel<<<pool_grid(c, total), 256, 0, (cudaStream_t)stream>>>(p, (const uint2 *)index, (const uint4 *)dy,
                                                                                       (uint4 *)dx);
    else
        maxpool_bwd_kernel<<<pool_grid(c, total), 256, 0, (cudaStream_t)stream>>>(p, (const uint4 *)x, (const uint4 *)dy, (uint4 *)dx);
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}
