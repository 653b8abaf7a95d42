// Zero-group detection for ONE conv weight tensor that allocates nothing, anywhere.
//
// Who needs this: code that runs where a device allocation is not allowed or not possible -- inside a
// framework that owns the whole device heap through its own caching allocator and forbids raw cudaMalloc,
// in a latency-critical loop where the implicit device synchronisation of an allocation is not acceptable,
// or in a long-lived service that must never fail with "out of memory" half-way through a reconfiguration.
// Such a caller can pass its inputs and outputs but has no workspace to hand over.
//
// The scratch the detection needs (one 32-bit max-|w| slot per output channel and per input channel) lives in
// a file-scope __device__ array instead. Consequences, all documented in include/pt.h as well:
//   * K + C is limited to PT_NOALLOC_MAX_GROUPS; larger layers are rejected with PT_ERR_UNSUPPORTED;
//   * every GPU that loads the library carries the array (256 KiB) until the process exits;
//   * all calls on a device share it and it keeps the previous call's contents, so each call first clears the
//     slots it is going to use, and two calls that overlap on the GPU (different streams) race;
//   * the first call on a device looks the array's device address up (cudaGetSymbolAddress); make that first
//     call outside any stream capture.
#include "pt_internal.h"
#include <mutex>

namespace {

constexpr int kMaxGroups = 65536;
constexpr int kMaxDevices = 64;

// The array's name is only a host-side handle here; the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned int g_noalloc_scratch[kMaxGroups];

std::mutex g_setup_mutex;
unsigned int *g_scratch_addr[kMaxDevices] = {nullptr};

// Once per device, with that device current: resolve the device address of the static scratch array.
pt_status scratch_for_current_device(unsigned int **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { (void)cudaGetLastError(); return PT_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) { (void)cudaGetLastError(); return PT_ERR_CUDA; }
        g_scratch_addr[dev] = (unsigned int *)p;
    }
    *out = g_scratch_addr[dev];
    return PT_OK;
}

// Block = TY line groups x TX columns; thread (tx, ty) owns column col0 + tx and lines ty, ty + TY, ... of its block's
// run of lines. |w| is compared through its bit pattern (ordered like the value; a NaN sorts above +inf).
__global__ void __launch_bounds__(256) noalloc_absmax_kernel(const float *__restrict__ w, int lines, int C, int RS, int tx_log2,
                                                             int lines_per_block, unsigned int *__restrict__ mk,
                                                             unsigned int *__restrict__ mc)
{
    const int TX = 1 << tx_log2, TY = 256 >> tx_log2;
    const int tx = threadIdx.x & (TX - 1), ty = threadIdx.x >> tx_log2, lane = threadIdx.x & 31;
    const int c = blockIdx.y * TX + tx;
    const bool cv = c < C;
    const int line0 = blockIdx.x * lines_per_block;
    const int line_end = min(lines, line0 + lines_per_block);
    unsigned int cm = 0u;
    for (int l = line0 + ty; l < line_end; l += TY) {       // the trip count is uniform within a warp (same ty)
        unsigned int b = cv ? (__float_as_uint(w[(size_t)l * C + c]) & 0x7fffffffu) : 0u;
        cm = max(cm, b);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) b = max(b, __shfl_xor_sync(0xffffffffu, b, o));
        if (lane == 0 && b) atomicMax(&mk[l / RS], b);
    }
    if (cv && cm) atomicMax(&mc[c], cm);
}

__global__ void noalloc_masks_kernel(const unsigned int *__restrict__ mk, const unsigned int *__restrict__ mc, int K, int C,
                                     float thr, uint8_t *__restrict__ zero_out, uint8_t *__restrict__ zero_in)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    // strict "<" in fp32; a NaN compares false and keeps its group
    if (i < K) zero_out[i] = (__uint_as_float(mk[i]) < thr) ? 1 : 0;
    else if (i < K + C) zero_in[i - K] = (__uint_as_float(mc[i - K]) < thr) ? 1 : 0;
}

}  // namespace

extern "C" pt_status pt_find_zero_groups_noalloc(const float *w, int32_t K, int32_t C, int32_t RS, float threshold,
                                                 uint8_t *zero_out, uint8_t *zero_in, void *stream)
{
    if (!w || !zero_out || !zero_in || K <= 0 || C <= 0 || RS <= 0 || !(threshold >= 0.f)) return PT_ERR_INVALID_ARG;
    if ((long long)K + C > kMaxGroups) return PT_ERR_UNSUPPORTED;          // beyond the static scratch: use pt_find_zero_groups
    if ((long long)K * RS * C >= (1ll << 31)) return PT_ERR_UNSUPPORTED;
    unsigned int *scratch = nullptr;
    pt_status s = scratch_for_current_device(&scratch);
    if (s != PT_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned int *mk = scratch, *mc = scratch + K;
    // the array still holds the previous call's maxima: clear the slots this call uses
    PT_CUDA_OK(cudaMemsetAsync(scratch, 0, (size_t)(K + C) * sizeof(unsigned int), st));
    int lg = 5;
    while ((1 << lg) < C && lg < 8) ++lg;
    const int TX = 1 << lg, TY = 256 / TX;
    const int lines = K * RS, lines_per_block = TY * 32;
    dim3 grid((unsigned)pt_ceil_div(lines, lines_per_block), (unsigned)pt_ceil_div(C, TX));
    noalloc_absmax_kernel<<<grid, 256, 0, st>>>(w, lines, C, RS, lg, lines_per_block, mk, mc);
    noalloc_masks_kernel<<<pt_ceil_div(K + C, 256), 256, 0, st>>>(mk, mc, K, C, threshold, zero_out, zero_in);
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}
