// Penalty-coefficient set-up (Eq. 3): softmax cross-entropy of the first forward pass and lambda from the penalty ratio.
// Tiny kernels: one warp per logits row, fp32 row arithmetic with the row maximum subtracted, fp64 batch mean summed in a
// fixed order by a single block (run-to-run identical).
#include "pt_internal.h"
#include <math.h>

namespace {

constexpr int kRowsPerBlock = 8;        // one warp per row

__global__ void xent_rows_kernel(const float *__restrict__ logits, const int *__restrict__ labels, int n, int classes, int ld,
                                 float *__restrict__ row_loss)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * kRowsPerBlock + warp;
    if (row >= n) return;
    const float *z = logits + (size_t)row * ld;
    float m = -INFINITY;
    for (int c = lane; c < classes; c += 32) m = fmaxf(m, z[c]);
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float s = 0.f;
    for (int c = lane; c < classes; c += 32) s += expf(z[c] - m);
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);    // butterfly: every lane ends with the same sum
    if (lane == 0) {
        const int lab = labels[row];
        row_loss[row] = (lab >= 0 && lab < classes) ? (m + logf(s)) - z[lab] : NAN;
    }
}

// One block: thread t sums rows t, t + 256, ... in ascending order, then a fixed tree over the 256 partial sums.
__global__ void xent_mean_kernel(const float *__restrict__ row_loss, int n, double *__restrict__ loss_out)
{
    __shared__ double part[256];
    double acc = 0.0;
    for (int i = threadIdx.x; i < n; i += 256) acc += (double)row_loss[i];
    part[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) loss_out[0] = part[0] / (double)n;
}

__global__ void set_coeff_kernel(const double *__restrict__ loss, const double *__restrict__ reg_sum, double ratio,
                                 float *__restrict__ lambda_out)
{
    const double r = reg_sum[0];
    lambda_out[0] = r == 0.0 ? 0.f : (float)(ratio * loss[0] / ((1.0 - ratio) * r));
}

}  // namespace

extern "C" size_t pt_cross_entropy_workspace_bytes(int32_t n) { return n > 0 ? (size_t)n * sizeof(float) : 0; }

extern "C" pt_status pt_cross_entropy(pt_ctx *c, const float *logits, const int32_t *labels, int32_t n, int32_t classes, int32_t ld,
                                      double *loss_out, void *ws, size_t ws_bytes, void *stream)
{
    if (!c || !logits || !labels || !loss_out || n < 1 || classes < 1 || ld < classes) return PT_ERR_INVALID_ARG;
    if (!ws || ws_bytes < pt_cross_entropy_workspace_bytes(n)) return PT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    float *rows = (float *)ws;
    xent_rows_kernel<<<pt_ceil_div(n, kRowsPerBlock), kRowsPerBlock * 32, 0, st>>>(logits, labels, n, classes, ld, rows);
    xent_mean_kernel<<<1, 256, 0, st>>>(rows, n, loss_out);
    c->launches += 2;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

extern "C" pt_status pt_set_coeff(pt_ctx *c, const double *loss, const double *reg_sum, float ratio, float *lambda_out, void *stream)
{
    if (!c || !loss || !reg_sum || !lambda_out || !(ratio > 0.f && ratio < 1.f)) return PT_ERR_INVALID_ARG;
    set_coeff_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(loss, reg_sum, (double)ratio, lambda_out);
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}
