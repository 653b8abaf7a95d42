// CUDA-core implicit-GEMM convolutions (fwd, dgrad, wgrad) for every legal shape.
// They are the general path for shapes the tcgen05 kernels do not take, and an
// independent GPU cross-check of them. bf16 operands, fp32 accumulation.
#include "pt_internal.h"

namespace {

struct ConvP {
    int N, H, W, C, K, R, S, stride, pad, P, Q;
    int ldx, ldy, ldw, out_f32;
    int M, Nn, Kred;            // implicit GEMM extents
    int kred_per_split;         // wgrad: reduction elements per grid.z slice
};

constexpr int BM = 64, BN = 64, BK = 16;

// MODE 0: fwd    M = N*P*Q (pixels) , Nn = K        , Kred = R*S*C   (kk = (r*S+s)*C + c)
// MODE 1: dgrad  M = N*H*W (pixels) , Nn = C        , Kred = R*S*K   (kk = (r*S+s)*K + k)
// MODE 2: wgrad  M = K              , Nn = R*S*C    , Kred = N*P*Q   (kk = output pixel)
template <int MODE>
__device__ __forceinline__ float load_a(const ConvP &p, const __nv_bfloat16 *a, int m, int kk)
{
    if (m >= p.M || kk >= p.Kred) return 0.f;
    if (MODE == 0) {
        int c = kk % p.C, rs = kk / p.C, s = rs % p.S, r = rs / p.S;
        int q = m % p.Q, t = m / p.Q, pp = t % p.P, n = t / p.P;
        int h = pp * p.stride - p.pad + r, w = q * p.stride - p.pad + s;
        if (h < 0 || h >= p.H || w < 0 || w >= p.W) return 0.f;
        return __bfloat162float(a[((size_t)(n * p.H + h) * p.W + w) * p.ldx + c]);
    } else if (MODE == 1) {
        int k = kk % p.K, rs = kk / p.K, s = rs % p.S, r = rs / p.S;
        int w = m % p.W, t = m / p.W, h = t % p.H, n = t / p.H;
        int hp = h + p.pad - r, wq = w + p.pad - s;
        if (hp < 0 || wq < 0 || hp % p.stride || wq % p.stride) return 0.f;
        int pp = hp / p.stride, q = wq / p.stride;
        if (pp >= p.P || q >= p.Q) return 0.f;
        return __bfloat162float(a[((size_t)(n * p.P + pp) * p.Q + q) * p.ldy + k]);
    } else {
        return __bfloat162float(a[(size_t)kk * p.ldy + m]);      // dy[pixel][k]
    }
}

template <int MODE>
__device__ __forceinline__ float load_b(const ConvP &p, const __nv_bfloat16 *b, int kk, int j)
{
    if (j >= p.Nn || kk >= p.Kred) return 0.f;
    if (MODE == 0) {
        int c = kk % p.C, rs = kk / p.C;
        return __bfloat162float(b[((size_t)j * p.R * p.S + rs) * p.ldw + c]);
    } else if (MODE == 1) {
        int k = kk % p.K, rs = kk / p.K;
        return __bfloat162float(b[((size_t)k * p.R * p.S + rs) * p.ldw + j]);
    } else {
        int c = j % p.C, rs = j / p.C, s = rs % p.S, r = rs / p.S;
        int q = kk % p.Q, t = kk / p.Q, pp = t % p.P, n = t / p.P;
        int h = pp * p.stride - p.pad + r, w = q * p.stride - p.pad + s;
        if (h < 0 || h >= p.H || w < 0 || w >= p.W) return 0.f;
        return __bfloat162float(b[((size_t)(n * p.H + h) * p.W + w) * p.ldx + c]);
    }
}

template <int MODE>
__global__ void __launch_bounds__(256) simt_conv_kernel(ConvP p, const __nv_bfloat16 *__restrict__ a,
                                                        const __nv_bfloat16 *__restrict__ b, void *__restrict__ out,
                                                        float *__restrict__ partial)
{
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int t = threadIdx.x, tx = t % 16, ty = t / 16;
    const int m0 = blockIdx.x * BM, j0 = blockIdx.y * BN;
    int kbeg = 0, kend = p.Kred;
    if (MODE == 2) {
        kbeg = blockIdx.z * p.kred_per_split;
        kend = min(p.Kred, kbeg + p.kred_per_split);
    }
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = kbeg; k0 < kend; k0 += BK) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int idx = t + 256 * e;
            int ml, kl;
            if (MODE == 2) { ml = idx % BM; kl = idx / BM; } else { kl = idx % BK; ml = idx / BK; }
            int kk = k0 + kl;
            As[kl][ml] = (kk < kend) ? load_a<MODE>(p, a, m0 + ml, kk) : 0.f;
            int jl, kl2;
            if (MODE == 0) { kl2 = idx % BK; jl = idx / BK; } else { jl = idx % BN; kl2 = idx / BN; }
            int kk2 = k0 + kl2;
            Bs[kl2][jl] = (kk2 < kend) ? load_b<MODE>(p, b, kk2, j0 + jl) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kl = 0; kl < BK; ++kl) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) av[i] = As[kl][ty + 16 * i];
#pragma unroll
            for (int j = 0; j < 4; ++j) bv[j] = Bs[kl][tx + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + ty + 16 * i;
        if (m >= p.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int jj = j0 + tx + 16 * j;
            if (jj >= p.Nn) continue;
            if (MODE == 2) {
                partial[((size_t)blockIdx.z * p.M + m) * p.Nn + jj] = acc[i][j];
            } else {
                size_t o = (size_t)m * (MODE == 0 ? p.ldy : p.ldx) + jj;
                if (p.out_f32) ((float *)out)[o] = acc[i][j];
                else ((__nv_bfloat16 *)out)[o] = __float2bfloat16_rn(acc[i][j]);
            }
        }
    }
}

// dw[i] = sum over splits, ascending: fixed order, so the result is run-to-run identical.
__global__ void splitk_reduce_kernel(const float *__restrict__ partial, float *__restrict__ dw, size_t n, int splits)
{
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = 0.f;
    for (int z = 0; z < splits; ++z) s += partial[(size_t)z * n + i];
    dw[i] = s;
}

int simt_wgrad_splits(const pt_ctx *c, const pt_conv_desc *d, int P, int Q)
{
    int tiles = pt_ceil_div(d->K, BM) * pt_ceil_div(d->R * d->S * d->C, BN);
    long long kred = (long long)d->N * P * Q;
    int want = pt_ceil_div(4 * c->sm_count, tiles);
    long long maxs = (kred + 255) / 256;
    if (want > maxs) want = (int)maxs;
    if (want < 1) want = 1;
    if (want > 1024) want = 1024;
    return want;
}

}  // namespace

size_t pt_simt_conv_workspace(const pt_ctx *c, const pt_conv_desc *d, int which)
{
    if (which != PT_CONV_WGRAD) return 0;
    int P = pt_out_dim(d->H, d->R, d->stride, d->pad), Q = pt_out_dim(d->W, d->S, d->stride, d->pad);
    return (size_t)simt_wgrad_splits(c, d, P, Q) * d->K * d->R * d->S * d->C * sizeof(float);
}

pt_status pt_simt_conv(pt_ctx *c, const pt_conv_desc *d, int which, const void *a, const void *b, void *out,
                       void *ws, size_t ws_bytes, cudaStream_t st)
{
    ConvP p;
    p.N = d->N; p.H = d->H; p.W = d->W; p.C = d->C; p.K = d->K; p.R = d->R; p.S = d->S;
    p.stride = d->stride; p.pad = d->pad;
    p.P = pt_out_dim(d->H, d->R, d->stride, d->pad);
    p.Q = pt_out_dim(d->W, d->S, d->stride, d->pad);
    p.ldx = d->ldx; p.ldy = d->ldy; p.ldw = d->ldw; p.out_f32 = d->out_f32;
    p.kred_per_split = 0;
    const __nv_bfloat16 *A = (const __nv_bfloat16 *)a, *B = (const __nv_bfloat16 *)b;
    if (which == PT_CONV_FWD) {
        p.M = d->N * p.P * p.Q; p.Nn = d->K; p.Kred = d->R * d->S * d->C;
        dim3 grid(pt_ceil_div(p.M, BM), pt_ceil_div(p.Nn, BN));
        simt_conv_kernel<0><<<grid, 256, 0, st>>>(p, A, B, out, nullptr);
        c->launches += 1;
    } else if (which == PT_CONV_DGRAD) {
        p.M = d->N * d->H * d->W; p.Nn = d->C; p.Kred = d->R * d->S * d->K;
        dim3 grid(pt_ceil_div(p.M, BM), pt_ceil_div(p.Nn, BN));
        simt_conv_kernel<1><<<grid, 256, 0, st>>>(p, A, B, out, nullptr);
        c->launches += 1;
    } else {
        p.M = d->K; p.Nn = d->R * d->S * d->C; p.Kred = d->N * p.P * p.Q;
        int splits = simt_wgrad_splits(c, d, p.P, p.Q);
        size_t n = (size_t)p.M * p.Nn;
        if (ws_bytes < (size_t)splits * n * sizeof(float)) return PT_ERR_WORKSPACE;
        p.kred_per_split = pt_ceil_div(pt_ceil_div(p.Kred, splits), BK) * BK;
        dim3 grid(pt_ceil_div(p.M, BM), pt_ceil_div(p.Nn, BN), splits);
        // operands: A = dy, B = x
        simt_conv_kernel<2><<<grid, 256, 0, st>>>(p, B, A, nullptr, (float *)ws);
        splitk_reduce_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>((const float *)ws, (float *)out, n, splits);
        c->launches += 2;
    }
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}
