// Context management, status handling, table upload and the conv entry points' dispatch.
#include "pt_internal.h"
#include <stdio.h>

static const size_t kArenaBytes = 5u << 20;     // 5 MiB of tables: ten slots of 512 KiB
static const size_t kSlotBytes = 512u << 10;
static const size_t kSyncWords = 16384;         // arrival counters of the split weight gradients

static thread_local char g_last_cuda[384] = "";

void pt_note_cuda_error(cudaError_t e, const char *call, const char *file, int line)
{
    const char *base = strrchr(file, '/');
    snprintf(g_last_cuda, sizeof(g_last_cuda), "%s (%d) from %.200s at %s:%d", cudaGetErrorName(e), (int)e, call,
             base ? base + 1 : file, line);
}

extern "C" const char *pt_last_cuda_error(void) { return g_last_cuda; }

extern "C" const char *pt_status_string(pt_status s)
{
    switch (s) {
    case PT_OK: return "PT_OK";
    case PT_ERR_INVALID_ARG: return "PT_ERR_INVALID_ARG";
    case PT_ERR_UNSUPPORTED: return "PT_ERR_UNSUPPORTED";
    case PT_ERR_WORKSPACE: return "PT_ERR_WORKSPACE";
    case PT_ERR_CUDA: return "PT_ERR_CUDA";
    case PT_ERR_TIMEOUT: return "PT_ERR_TIMEOUT";
    case PT_ERR_ARCH: return "PT_ERR_ARCH";
    }
    return "PT_ERR_UNKNOWN";
}

extern "C" pt_status pt_create(pt_ctx **out, int device)
{
    if (!out) return PT_ERR_INVALID_ARG;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) { (void)cudaGetLastError(); return PT_ERR_CUDA; }
    PT_CUDA_OK(cudaSetDevice(device));
    cudaDeviceProp prop;
    PT_CUDA_OK(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return PT_ERR_ARCH;
    pt_ctx *c = new pt_ctx();
    c->device = device;
    c->sm_count = prop.multiProcessorCount;
    c->cc_major = prop.major;
    c->cc_minor = prop.minor;
    c->arena_bytes = kArenaBytes;
    bool ok = cudaMalloc(&c->d_status, 16) == cudaSuccess && cudaMemset(c->d_status, 0, 16) == cudaSuccess &&
              cudaMallocHost(&c->h_status, 16) == cudaSuccess && cudaMalloc(&c->d_arena, kArenaBytes) == cudaSuccess &&
              cudaMallocHost(&c->h_stage, kArenaBytes) == cudaSuccess &&
              cudaMallocHost(&c->h_counts, (65536 + 16) * sizeof(int32_t)) == cudaSuccess &&
              cudaMalloc(&c->d_sync, kSyncWords * sizeof(unsigned int)) == cudaSuccess &&
              cudaMemset(c->d_sync, 0, kSyncWords * sizeof(unsigned int)) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->upload_done, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { (void)cudaGetLastError(); pt_destroy(c); return PT_ERR_CUDA; }
    size_t off = 0;
    for (int i = 0; i < 3; ++i) { c->lasso_tab[i].off = off; c->lasso_tab[i].cap = kSlotBytes; off += kSlotBytes; }
    for (int i = 0; i < 2; ++i) { c->detect_tab[i].off = off; c->detect_tab[i].cap = kSlotBytes; off += kSlotBytes; }
    c->graph_tab.off = off;  c->graph_tab.cap = kSlotBytes; off += kSlotBytes;
    for (int i = 0; i < 4; ++i) { c->gather_slot[i].reg.off = off; c->gather_slot[i].reg.cap = kSlotBytes; off += kSlotBytes; }
    // Driver entry points for tensor-map encoding, looked up at run time so the library loads without libcuda.
    cudaDriverEntryPointQueryResult qr;
    void *fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess) c->encode_tiled = fn;
    fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess) c->encode_im2col = fn;
    (void)cudaGetLastError();
    *out = c;
    return PT_OK;
}

extern "C" pt_status pt_destroy(pt_ctx *c)
{
    if (!c) return PT_OK;
    (void)cudaSetDevice(c->device);
    if (c->upload_done) cudaEventDestroy(c->upload_done);
    for (int i = 0; i < 3; ++i) {
        if (c->fork_stream[i]) cudaStreamDestroy(c->fork_stream[i]);
        if (c->join_ev[i]) cudaEventDestroy(c->join_ev[i]);
    }
    if (c->fork_ev) cudaEventDestroy(c->fork_ev);
    if (c->d_status) cudaFree(c->d_status);
    if (c->h_status) cudaFreeHost(c->h_status);
    if (c->d_arena) cudaFree(c->d_arena);
    if (c->h_stage) cudaFreeHost(c->h_stage);
    if (c->h_counts) cudaFreeHost(c->h_counts);
    if (c->d_sync) cudaFree(c->d_sync);
    (void)cudaGetLastError();
    delete c;
    return PT_OK;
}

extern "C" uint64_t pt_launch_count(const pt_ctx *c) { return c ? c->launches : 0; }

extern "C" pt_status pt_set_wgrad_cta_limit(pt_ctx *c, int max_ctas)
{
    if (!c || max_ctas < 0) return PT_ERR_INVALID_ARG;
    c->wgrad_ctas = max_ctas;
    return PT_OK;
}

extern "C" pt_status pt_test_set_wait_limit(pt_ctx *c, uint32_t milliseconds)
{
    if (!c) return PT_ERR_INVALID_ARG;
    PT_CUDA_OK(cudaSetDevice(c->device));
    return pt_sm100_set_wait_limit_ns(milliseconds ? (unsigned long long)milliseconds * 1000000ull : 2000000000ull, nullptr);
}

extern "C" pt_status pt_test_skip_next_arrive(pt_ctx *c, int32_t which)
{
    if (!c || which < 0 || which > 2) return PT_ERR_INVALID_ARG;
    c->test_skip = which;
    return PT_OK;
}

extern "C" pt_status pt_poll_device_status(pt_ctx *c, void *stream)
{
    if (!c) return PT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    PT_CUDA_OK(cudaMemcpyAsync(c->h_status, c->d_status, 16, cudaMemcpyDeviceToHost, st));
    PT_CUDA_OK(cudaStreamSynchronize(st));
    unsigned int code = c->h_status[0];
    if (code != PT_DEV_OK) {
        PT_CUDA_OK(cudaMemsetAsync(c->d_status, 0, 16, st));
        if (code == PT_DEV_TIMEOUT) {
            // A split weight gradient that gave up leaves its arrival counters non-zero (only the normal path resets them):
            // clear the whole ring, or a later launch that gets the same slots would see its splits as already arrived.
            PT_CUDA_OK(cudaMemsetAsync(c->d_sync, 0, kSyncWords * sizeof(unsigned int), st));
            c->sync_next = 0;
        }
        PT_CUDA_OK(cudaStreamSynchronize(st));
        return code == PT_DEV_TIMEOUT ? PT_ERR_TIMEOUT : code == PT_DEV_BAD_INDEX ? PT_ERR_INVALID_ARG : PT_ERR_CUDA;
    }
    return PT_OK;
}

pt_status pt_upload_table(pt_ctx *c, pt_region *reg, const void *host, size_t bytes, cudaStream_t st, char **dev)
{
    if (bytes > reg->cap) return PT_ERR_UNSUPPORTED;
    *dev = c->d_arena + reg->off;
    if (reg->valid && reg->key.size() == bytes && memcmp(reg->key.data(), host, bytes) == 0) return PT_OK;
    if (c->upload_pending) {                       // the staging buffer may still be the source of a copy
        PT_CUDA_OK(cudaEventSynchronize(c->upload_done));
        c->upload_pending = false;
    }
    memcpy(c->h_stage + reg->off, host, bytes);
    PT_CUDA_OK(cudaMemcpyAsync(c->d_arena + reg->off, c->h_stage + reg->off, bytes, cudaMemcpyHostToDevice, st));
    PT_CUDA_OK(cudaEventRecord(c->upload_done, st));
    c->upload_pending = true;
    reg->key.assign((const char *)host, (const char *)host + bytes);
    reg->valid = true;
    return PT_OK;
}

pt_status pt_upload_table_slots(pt_ctx *c, pt_region *slots, int n_slots, int *next, const void *host, size_t bytes,
                                cudaStream_t st, char **dev)
{
    for (int i = 0; i < n_slots; ++i)
        if (slots[i].valid && slots[i].key.size() == bytes && memcmp(slots[i].key.data(), host, bytes) == 0)
            return pt_upload_table(c, &slots[i], host, bytes, st, dev);
    pt_region *victim = &slots[*next % n_slots];
    *next = (*next + 1) % n_slots;
    return pt_upload_table(c, victim, host, bytes, st, dev);
}

// ------------------------------------------------------------------------------------------ conv dispatch
pt_status pt_conv_validate(const pt_ctx *c, const pt_conv_desc *d, int *P, int *Q)
{
    if (!c || !d) return PT_ERR_INVALID_ARG;
    if (d->N <= 0 || d->H <= 0 || d->W <= 0 || d->C <= 0 || d->K <= 0 || d->R <= 0 || d->S <= 0) return PT_ERR_INVALID_ARG;
    if (d->stride <= 0 || d->pad < 0 || d->pad >= d->R + d->S) return PT_ERR_INVALID_ARG;
    if (d->ldx < d->C || d->ldx % 8 || d->ldy < d->K || d->ldy % 8 || d->ldw < d->C || d->ldw % 8) return PT_ERR_INVALID_ARG;
    if (d->algo < 0 || d->algo > 2) return PT_ERR_INVALID_ARG;
    *P = pt_out_dim(d->H, d->R, d->stride, d->pad);
    *Q = pt_out_dim(d->W, d->S, d->stride, d->pad);
    if (*P <= 0 || *Q <= 0) return PT_ERR_INVALID_ARG;
    // index arithmetic inside the kernels is 64-bit for addresses and 32-bit for pixel counts
    if ((int64_t)d->N * d->H * d->W >= (1ll << 31) || (int64_t)d->N * *P * *Q >= (1ll << 31)) return PT_ERR_UNSUPPORTED;
    if ((int64_t)d->K * d->R * d->S * d->ldw >= (1ll << 31)) return PT_ERR_UNSUPPORTED;
    return PT_OK;
}

static bool aligned16(const void *p) { return ((uintptr_t)p & 15) == 0; }

extern "C" size_t pt_conv_workspace_bytes(const pt_ctx *c, const pt_conv_desc *d, int which)
{
    int P, Q;
    if (which < 0 || which > 2 || pt_conv_validate(c, d, &P, &Q) != PT_OK) return 0;
    size_t a = pt_simt_conv_workspace(c, d, which);
    size_t b = pt_sm100_conv_supported(c, d, which) ? pt_sm100_conv_workspace(c, d, which) : 0;
    if (d->algo == 1) return a;
    if (d->algo == 2) return b;
    return a > b ? a : b;
}

extern "C" int32_t pt_conv_wgrad_ctas(const pt_ctx *c, const pt_conv_desc *d, int32_t *waits)
{
    int P, Q;
    if (waits) *waits = 0;
    if (pt_conv_validate(c, d, &P, &Q) != PT_OK) return 0;
    if (d->algo == 1 || !pt_sm100_conv_supported(c, d, PT_CONV_WGRAD)) return 0;
    int w = 0;
    const int n = pt_sm100_wgrad_ctas(c, d, &w);
    if (waits) *waits = w;
    return n;
}

static pt_status conv_dispatch(pt_ctx *c, const pt_conv_desc *d, int which, const void *a, const void *b, void *out,
                               void *ws, size_t ws_bytes, void *stream)
{
    int P, Q;
    pt_status s = pt_conv_validate(c, d, &P, &Q);
    if (s != PT_OK) return s;
    if (!a || !b || !out) return PT_ERR_INVALID_ARG;
    if (!aligned16(a) || !aligned16(b) || !aligned16(out) || (ws && !aligned16(ws))) return PT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    bool fast = d->algo != 1 && pt_sm100_conv_supported(c, d, which);
    if (d->algo == 2 && !fast) return PT_ERR_UNSUPPORTED;
    if (fast) {
        if (pt_sm100_conv_workspace(c, d, which) > ws_bytes || (pt_sm100_conv_workspace(c, d, which) && !ws)) return PT_ERR_WORKSPACE;
        pt_status r = pt_sm100_conv(c, d, which, a, b, out, ws, ws_bytes, st);
        if (r != PT_ERR_UNSUPPORTED || d->algo == 2) return r;     // a shape the tcgen05 path declines goes to the SIMT kernels
    }
    if (pt_simt_conv_workspace(c, d, which) > ws_bytes || (pt_simt_conv_workspace(c, d, which) && !ws)) return PT_ERR_WORKSPACE;
    return pt_simt_conv(c, d, which, a, b, out, ws, ws_bytes, st);
}

extern "C" pt_status pt_conv_fwd(pt_ctx *c, const pt_conv_desc *d, const void *x, const void *w, void *y,
                                 void *ws, size_t ws_bytes, void *stream)
{
    return conv_dispatch(c, d, PT_CONV_FWD, x, w, y, ws, ws_bytes, stream);
}

extern "C" size_t pt_conv_fwd_stats_bytes(const pt_ctx *c, const pt_conv_desc *d)
{
    int P, Q;
    if (pt_conv_validate(c, d, &P, &Q) != PT_OK) return 0;
    return (size_t)c->sm_count * 12 * 2 * (size_t)d->ldy * sizeof(float);      // at most twelve epilogue warps per SM
}

extern "C" pt_status pt_conv_fwd_stats(pt_ctx *c, const pt_conv_desc *d, const void *x, const void *w, void *y, float *stats,
                                       size_t stats_bytes, int32_t *n_parts, void *ws, size_t ws_bytes, void *stream)
{
    if (!c || !d || !stats || !n_parts) return PT_ERR_INVALID_ARG;
    if (d->out_f32 || d->algo == 1) return PT_ERR_UNSUPPORTED;
    pt_conv_desc dd = *d;
    dd.algo = 2;                                    // the statistics come out of the tcgen05 kernels' epilogues only
    c->stats_mode = 2; c->stats_out = stats; c->stats_cap = stats_bytes; c->stats_parts = 0;
    const pt_status r = conv_dispatch(c, &dd, PT_CONV_FWD, x, w, y, ws, ws_bytes, stream);
    c->stats_mode = 0; c->stats_out = nullptr; c->stats_cap = 0;
    *n_parts = r == PT_OK ? c->stats_parts : 0;
    return r;
}

extern "C" pt_status pt_conv_dgrad(pt_ctx *c, const pt_conv_desc *d, const void *dy, const void *w, void *dx,
                                   void *ws, size_t ws_bytes, void *stream)
{
    return conv_dispatch(c, d, PT_CONV_DGRAD, dy, w, dx, ws, ws_bytes, stream);
}

extern "C" pt_status pt_conv_wgrad(pt_ctx *c, const pt_conv_desc *d, const void *x, const void *dy, float *dw,
                                   void *ws, size_t ws_bytes, void *stream)
{
    return conv_dispatch(c, d, PT_CONV_WGRAD, x, dy, dw, ws, ws_bytes, stream);
}

// ------------------------------------------------------------------ dynamic mini-batch adjustment (Sec. 4.3), host arithmetic
static bool shape_ok(const pt_layer_shape &l)
{
    return l.H > 0 && l.W > 0 && l.C > 0 && l.K > 0 && l.R > 0 && l.S > 0 && l.stride > 0 && l.pad >= 0 &&
           pt_out_dim(l.H, l.R, l.stride, l.pad) > 0 && pt_out_dim(l.W, l.S, l.stride, l.pad) > 0;
}

static void memory_terms(const pt_layer_shape *layers, int32_t n, size_t *fixed, size_t *per_sample)
{
    size_t f = 0, a = 0;
    for (int i = 0; i < n; ++i) {
        const pt_layer_shape &l = layers[i];
        const size_t P = (size_t)pt_out_dim(l.H, l.R, l.stride, l.pad), Q = (size_t)pt_out_dim(l.W, l.S, l.stride, l.pad);
        const size_t ldc = pt_align_up((size_t)l.C, 8), ldk = pt_align_up((size_t)l.K, 8);
        f += (size_t)l.K * l.R * l.S * l.C * 12 + (size_t)l.K * l.R * l.S * ldc * 2;     // w, g, v fp32; bf16 shadow at its pitch
        a += ((size_t)l.H * l.W * ldc + P * Q * ldk) * 2 * 2;                             // x, dx, y, dy in bf16
    }
    *fixed = f;
    *per_sample = a;
}

extern "C" size_t pt_training_memory_bytes(const pt_layer_shape *layers, int32_t n, int32_t batch)
{
    if (!layers || n < 1 || batch < 1) return 0;
    for (int i = 0; i < n; ++i)
        if (!shape_ok(layers[i])) return 0;
    size_t f, a;
    memory_terms(layers, n, &f, &a);
    return f + a * (size_t)batch;
}

extern "C" pt_status pt_update_mini_batch(const pt_layer_shape *layers, int32_t n, size_t capacity_bytes, int32_t cur_batch,
                                          float cur_lr, int32_t granularity, int32_t *new_batch, float *new_lr)
{
    if (!layers || n < 1 || cur_batch < 1 || granularity < 1 || !new_batch || !new_lr) return PT_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i)
        if (!shape_ok(layers[i])) return PT_ERR_INVALID_ARG;
    size_t f, a;
    memory_terms(layers, n, &f, &a);
    int32_t nb = cur_batch;
    const size_t now = f + a * (size_t)cur_batch;
    if (now <= capacity_bytes) {
        const size_t steps = (capacity_bytes - now) / (a * (size_t)granularity);
        const size_t cap_steps = (size_t)(0x7fffffff - cur_batch) / (size_t)granularity;
        nb = cur_batch + (int32_t)(steps < cap_steps ? steps : cap_steps) * granularity;
    }
    *new_batch = nb;
    *new_lr = (float)((double)cur_lr * (double)nb / (double)cur_batch);
    return PT_OK;
}
