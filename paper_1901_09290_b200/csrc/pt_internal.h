// Internal declarations shared by the translation units of the library (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <string.h>
#include <vector>

#include "../../include/pt.h"

// The CUDA call that last failed on this thread: kept for pt_last_cuda_error.
void pt_note_cuda_error(cudaError_t e, const char *call, const char *file, int line);

#define PT_CUDA_OK(call)                                   \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) {                          \
            pt_note_cuda_error(e__, #call, __FILE__, __LINE__); \
            (void)cudaGetLastError();                      \
            return PT_ERR_CUDA;                            \
        }                                                  \
    } while (0)

// Device status word layout: [0] = first error code recorded (0 = none), [1] = detail (where), [2] = ticket of the
// keep-set scan (self-resetting), [3] spare.
enum { PT_DEV_OK = 0, PT_DEV_TIMEOUT = 1, PT_DEV_BAD_INDEX = 2 };

struct pt_region {              // one cached table in the arena
    size_t off = 0, cap = 0;    // byte range inside the arena
    std::vector<char> key;      // host bytes the current device copy was built from
    bool valid = false;
};

struct pt_ctx {
    int device = 0;
    int sm_count = 0;
    int cc_major = 0, cc_minor = 0;
    unsigned int *d_status = nullptr;   // 4 words, device
    unsigned int *h_status = nullptr;   // 4 words, pinned host
    char *d_arena = nullptr;            // table arena, device
    char *h_stage = nullptr;            // pinned staging copy of the arena
    size_t arena_bytes = 0;
    cudaEvent_t upload_done = nullptr;  // last staging->arena copy
    bool upload_pending = false;
    // Cached device tables. A captured CUDA graph embeds the device address of the table its kernels read, so tables of
    // different callers must not evict each other: the lasso step and the detection have their own slot sets.
    pt_region lasso_tab[3], detect_tab[2], graph_tab;
    int lasso_next = 0, detect_next = 0;
    // pt_reconfigure: four cached gather tables, each with the argument bytes it was built from and its launch shape. A call
    // with the same arguments (every reconfiguration of a fixed pair of models, or of a fixed part of them) launches straight
    // from its table; a caller that gathers a model in two parts keeps both tables alive.
    struct GatherSlot {
        pt_region reg;
        std::vector<char> args;
        unsigned chunks = 0, grid = 0;
        size_t jobs_bytes = 0, first_off = 0;
    } gather_slot[4];
    int gather_next = 0;
    int32_t *h_counts = nullptr;        // pinned, for pt_reconfigure_plan: [0] = flag the kernel raises, [16..] = counts
    unsigned int plan_seq = 0;          // sequence number the next plan's flag carries
    unsigned int *d_sync = nullptr;     // zero-initialised, self-resetting arrival counters of the split weight gradient
    unsigned int sync_next = 0;         // ring position in d_sync
    uint64_t launches = 0;
    int wgrad_ctas = 0;                 // CTA limit of a weight-gradient launch (0 = all SMs)
    // pt_conv_fwd_stats: non-zero while that call runs: the forward kernels also leave per-warp channel sums in stats_out
    // (stats_cap bytes) and the launcher records how many rows of partial sums there are
    int stats_mode = 0;
    int stats_parts = 0;
    float *stats_out = nullptr;
    size_t stats_cap = 0;
    int test_skip = 0;                  // pt_test_skip_next_arrive: 1 = next split weight gradient, 2 = next fwd/dgrad GEMM-form launch
    // Helper streams for independent launches inside one call (the parity classes of a stride-2 data gradient): the caller's
    // stream forks to them and joins them back through events, which a stream capture records as graph edges.
    cudaStream_t fork_stream[3] = {nullptr, nullptr, nullptr};
    cudaEvent_t fork_ev = nullptr, join_ev[3] = {nullptr, nullptr, nullptr};
    // tcgen05 conv path
    void *encode_tiled = nullptr;       // cuTensorMapEncodeTiled
    void *encode_im2col = nullptr;      // cuTensorMapEncodeIm2col
};

static inline int pt_ceil_div(int a, int b) { return (a + b - 1) / b; }
static inline size_t pt_align_up(size_t a, size_t b) { return (a + b - 1) / b * b; }
static inline int pt_out_dim(int H, int R, int stride, int pad) {
    int t = H + 2 * pad - R;
    return t < 0 ? 0 : t / stride + 1;
}

// Copies `bytes` of host data into the region's slot of the arena if it differs from what is there.
// Returns the device address of the slot.
pt_status pt_upload_table(pt_ctx *ctx, pt_region *reg, const void *host, size_t bytes, cudaStream_t st, char **dev);
// Same over a set of slots: a slot already holding these bytes is reused, otherwise the oldest one is overwritten.
pt_status pt_upload_table_slots(pt_ctx *ctx, pt_region *slots, int n_slots, int *next, const void *host, size_t bytes,
                                cudaStream_t st, char **dev);

// Validation shared by the conv entry points. Fills P, Q.
pt_status pt_conv_validate(const pt_ctx *ctx, const pt_conv_desc *d, int *P, int *Q);

// SIMT (CUDA-core) convolution kernels: every legal shape.
pt_status pt_simt_conv(pt_ctx *ctx, const pt_conv_desc *d, int which, const void *a, const void *b, void *out,
                       void *ws, size_t ws_bytes, cudaStream_t st);
size_t pt_simt_conv_workspace(const pt_ctx *ctx, const pt_conv_desc *d, int which);

// tcgen05 / TMEM / TMA convolution kernels: returns PT_ERR_UNSUPPORTED for shapes they do not cover.
bool pt_sm100_conv_supported(const pt_ctx *ctx, const pt_conv_desc *d, int which);
pt_status pt_sm100_conv(pt_ctx *ctx, const pt_conv_desc *d, int which, const void *a, const void *b, void *out,
                        void *ws, size_t ws_bytes, cudaStream_t st);
size_t pt_sm100_conv_workspace(const pt_ctx *ctx, const pt_conv_desc *d, int which);
int pt_sm100_wgrad_ctas(const pt_ctx *ctx, const pt_conv_desc *d, int *waits);
pt_status pt_sm100_set_wait_limit_ns(unsigned long long ns, cudaStream_t st);
