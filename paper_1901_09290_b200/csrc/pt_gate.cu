// Channel gating (Sec. 4.2, the alternative to channel union): a residual branch reads only the dense input channels of
// its first convolution out of the shared node tensor (gather) and its last convolution's dense output channels are put
// back at their positions in the node where the residual add happens (scatter-add). Both are pure data movement over
// NHWC bf16 tensors -- the tensor reshaping whose memory traffic the paper measured -- plus the list of dense channels.
// The gradient of the gather is the scatter-add and vice versa, so the two kernels serve both passes.
#include "pt_internal.h"

namespace {

constexpr int kGateMax = 4096;          // channels of a node / of a selection (index tables live in shared memory)
constexpr int kGateThreads = 256;

// An index outside the tensor is skipped (nothing is read or written there) and reported through the status word.
__device__ __forceinline__ void bad_index(unsigned int *status, unsigned int where)
{
    if (atomicCAS(&status[0], 0u, (unsigned)PT_DEV_BAD_INDEX) == 0u) status[1] = where;
}

// Ascending list of the indices whose flag is zero; one block, chunks of 1024 flags, ballot + warp totals.
__global__ void __launch_bounds__(1024) dense_list_kernel(const uint8_t *__restrict__ zero, int n, int *__restrict__ idx, int *__restrict__ count)
{
    __shared__ int warp_tot[32];
    __shared__ int base;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) base = 0;
    __syncthreads();
    for (int start = 0; start < n; start += 1024) {
        const int i = start + tid;
        const bool keep = i < n && zero[i] == 0;
        const unsigned b = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) warp_tot[warp] = __popc(b);
        __syncthreads();
        int off = base;
        for (int w = 0; w < warp; ++w) off += warp_tot[w];
        if (keep) idx[off + __popc(b & ((1u << lane) - 1u))] = i;
        __syncthreads();
        if (tid == 0) {
            int t = 0;
            for (int w = 0; w < 32; ++w) t += warp_tot[w];
            base += t;
        }
        __syncthreads();
    }
    for (int i = base + tid; i < n; i += 1024) idx[i] = -1;
    if (tid == 0) *count = base;
}

// dst[p][j] = src[p][idx[j]] (j < n_sel), 0 in the pad lanes. A thread produces 8 consecutive output channels (one 16-byte
// store); the threads of a block walk a contiguous range of pixels, so a source row is fetched once and then hit in L1.
__global__ void __launch_bounds__(kGateThreads) gather_kernel(const unsigned short *__restrict__ src, int ld_src, int c_src,
                                                              const int *__restrict__ idx, int n_sel, unsigned short *__restrict__ dst,
                                                              int ld_dst, long long npix, long long pix_per_block, unsigned int *status)
{
    __shared__ int s_idx[kGateMax];
    for (int j = threadIdx.x; j < ld_dst; j += kGateThreads) {
        int id = j < n_sel ? idx[j] : -1;
        if (j < n_sel && (id < 0 || id >= c_src)) { bad_index(status, 40u); id = -1; }
        s_idx[j] = id;
    }
    __syncthreads();
    const long long p_beg = (long long)blockIdx.x * pix_per_block;
    const long long p_end = p_beg + pix_per_block < npix ? p_beg + pix_per_block : npix;
    if (p_beg >= p_end) return;
    const int groups = ld_dst >> 3;
    const int items = (int)(p_end - p_beg) * groups;
    const unsigned short *s0 = src + (size_t)p_beg * ld_src;
    unsigned short *d0 = dst + (size_t)p_beg * ld_dst;
    for (int it = threadIdx.x; it < items; it += kGateThreads) {
        const int p = it / groups, g = it - p * groups;
        const unsigned short *row = s0 + (size_t)p * ld_src;
        __align__(16) unsigned short o[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int id = s_idx[g * 8 + e];
            o[e] = id >= 0 ? __ldg(row + id) : (unsigned short)0;
        }
        *reinterpret_cast<uint4 *>(d0 + (size_t)p * ld_dst + g * 8) = *reinterpret_cast<const uint4 *>(o);
    }
}

__device__ __forceinline__ float bf16_bits_to_float(unsigned short h) { return __uint_as_float((unsigned)h << 16); }

// node_out[p][c] = act(node_in[p][c] + branch[p][j] where idx[j] == c), fp32 add, one rounding to bf16; 0 in the pad lanes.
__global__ void __launch_bounds__(kGateThreads) scatter_add_kernel(const unsigned short *__restrict__ branch, int ld_b,
                                                                   const int *__restrict__ idx, int n_sel,
                                                                   const unsigned short *node_in,
                                                                   unsigned short *node_out, int ld_node, int c_node,
                                                                   long long npix, long long pix_per_block, int relu, unsigned int *status)
{
    __shared__ short s_inv[kGateMax];
    for (int c = threadIdx.x; c < ld_node; c += kGateThreads) s_inv[c] = -1;
    __syncthreads();
    for (int j = threadIdx.x; j < n_sel; j += kGateThreads) {
        const int id = idx[j];
        if (id < 0 || id >= c_node) bad_index(status, 41u);
        else s_inv[id] = (short)j;
    }
    __syncthreads();
    const long long p_beg = (long long)blockIdx.x * pix_per_block;
    const long long p_end = p_beg + pix_per_block < npix ? p_beg + pix_per_block : npix;
    if (p_beg >= p_end) return;
    const int groups = ld_node >> 3;
    const int items = (int)(p_end - p_beg) * groups;
    const unsigned short *b0 = branch + (size_t)p_beg * ld_b;
    const unsigned short *i0 = node_in ? node_in + (size_t)p_beg * ld_node : nullptr;
    unsigned short *o0 = node_out + (size_t)p_beg * ld_node;
    for (int it = threadIdx.x; it < items; it += kGateThreads) {
        const int p = it / groups, g = it - p * groups;
        uint4 in = make_uint4(0u, 0u, 0u, 0u);
        // node_in may be the tensor node_out (in-place merge): a plain load, not the read-only path, and no restrict
        if (i0) in = *reinterpret_cast<const uint4 *>(i0 + (size_t)p * ld_node + g * 8);
        const unsigned short *ie = reinterpret_cast<const unsigned short *>(&in);
        const unsigned short *brow = b0 + (size_t)p * ld_b;
        __align__(16) unsigned short o[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int c = g * 8 + e;
            float v = bf16_bits_to_float(ie[e]);
            const int j = s_inv[c];
            if (j >= 0) v += bf16_bits_to_float(__ldg(brow + j));
            if (relu) v = v > 0.f ? v : 0.f;
            const __nv_bfloat16 r = __float2bfloat16_rn(v);
            o[e] = c < c_node ? *reinterpret_cast<const unsigned short *>(&r) : (unsigned short)0;
        }
        *reinterpret_cast<uint4 *>(o0 + (size_t)p * ld_node + g * 8) = *reinterpret_cast<const uint4 *>(o);
    }
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

// Blocks walk contiguous pixel ranges; a few blocks per SM, and no range so long that its item count overflows an int.
void gate_grid(const pt_ctx *c, long long npix, int groups, unsigned *blocks, long long *pix_per_block)
{
    long long nb = (long long)c->sm_count * 8;
    long long ppb = (npix + nb - 1) / nb;
    if (ppb < 8) ppb = 8;
    const long long cap = (long long)(1 << 30) / (groups > 0 ? groups : 1);
    if (ppb > cap) ppb = cap;
    *pix_per_block = ppb;
    *blocks = (unsigned)((npix + ppb - 1) / ppb);
}

}  // namespace

extern "C" pt_status pt_dense_channel_list(pt_ctx *ctx, const uint8_t *zero_flags, int32_t n, int32_t *idx, int32_t *count, void *stream)
{
    if (!ctx || !zero_flags || !idx || !count || n < 0) return PT_ERR_INVALID_ARG;
    dense_list_kernel<<<1, 1024, 0, (cudaStream_t)stream>>>(zero_flags, n, idx, count);
    ctx->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

extern "C" pt_status pt_channel_gather(pt_ctx *ctx, const void *src, int32_t ld_src, int32_t c_src, const int32_t *idx, int32_t n_sel,
                                       void *dst, int32_t ld_dst, int64_t npix, void *stream)
{
    if (!ctx || !src || !dst || !idx || npix < 0 || n_sel < 0 || c_src < 1) return PT_ERR_INVALID_ARG;
    if (ld_src < c_src || ld_dst < n_sel || ld_dst < 8 || (ld_src & 7) || (ld_dst & 7) || !aligned16(src) || !aligned16(dst))
        return PT_ERR_INVALID_ARG;
    if (ld_dst > kGateMax) return PT_ERR_UNSUPPORTED;
    if (npix == 0) return PT_OK;
    unsigned blocks;
    long long ppb;
    gate_grid(ctx, npix, ld_dst >> 3, &blocks, &ppb);
    gather_kernel<<<blocks, kGateThreads, 0, (cudaStream_t)stream>>>((const unsigned short *)src, ld_src, c_src, idx, n_sel,
                                                                     (unsigned short *)dst, ld_dst, npix, ppb, ctx->d_status);
    ctx->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

extern "C" pt_status pt_channel_scatter_add(pt_ctx *ctx, const void *branch, int32_t ld_branch, const int32_t *idx, int32_t n_sel,
                                            const void *node_in, void *node_out, int32_t ld_node, int32_t c_node, int64_t npix,
                                            int32_t relu, void *stream)
{
    if (!ctx || !branch || !node_out || !idx || npix < 0 || n_sel < 0 || c_node < 1) return PT_ERR_INVALID_ARG;
    if (ld_node < c_node || ld_branch < n_sel || ld_branch < 8 || n_sel > c_node || (ld_node & 7) || (ld_branch & 7) ||
        !aligned16(branch) || !aligned16(node_out) || (node_in && !aligned16(node_in)))
        return PT_ERR_INVALID_ARG;
    if (ld_node > kGateMax || n_sel > 32767) return PT_ERR_UNSUPPORTED;
    if (npix == 0) return PT_OK;
    unsigned blocks;
    long long ppb;
    gate_grid(ctx, npix, ld_node >> 3, &blocks, &ppb);
    scatter_add_kernel<<<blocks, kGateThreads, 0, (cudaStream_t)stream>>>((const unsigned short *)branch, ld_branch, idx, n_sel,
                                                                          (const unsigned short *)node_in, (unsigned short *)node_out,
                                                                          ld_node, c_node, npix, ppb, relu ? 1 : 0, ctx->d_status);
    ctx->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}
