// Group-lasso regularised momentum SGD over all conv weights (Eq. 1-2, Algorithm 1) and
// zero-group detection (Sec. 4.1 threshold, Sec. 4.2 max-abs per channel).
//
// All layers are processed by one launch per phase through a chunk table. A weight tensor
// [K][RS][C] is seen as K*RS "lines" of C contiguous floats; a chunk is a run of lines of one
// layer. Inside a block, thread (tx, ty) owns the columns c = tx + TX*j and the lines
// ty, ty+TY, ... of its chunk, so every access is a coalesced run of a line and per-column
// quantities stay in registers.
//
// Phases of the step:
//   1. norms_partial : per line sum of squares, per chunk column sums of squares   (reads w)
//   2. norms_finish  : fixed-order reduction to s_out[k], s_in[c]; 1/norm factors; per-layer Eq. 2 sum
//   3. reg_total     : fixed-order sum of the per-layer sums -> reg_sum_out
//   4. update        : g~, v, w, bf16 shadow                                        (reads w,g,v; writes w,v,shadow)
// No floating-point atomics: results are run-to-run identical.
#include "pt_internal.h"

namespace {

struct LayerDev {
    float *w; const float *g; float *v; __nv_bfloat16 *wb;
    float *sumsq_out, *sumsq_in;
    uint8_t *zero_out, *zero_in;
    int K, C, RS, ldw;
    int reg_in, reg_out;
    int chunk0, n_chunks;       // this layer's chunks in the chunk table
    int tx_log2;                // TX = 1 << tx_log2 column lanes (32..256)
    int pad_;
    long long line_off;         // offset of this layer's lines in the per-line scratch
    long long col_off;          // offset of this layer's column partials (n_chunks * C floats)
    long long k_off, c_off;     // offsets into the per-K / per-C scratch arrays
};

struct Chunk { int layer, line0, nlines, idx; };

struct WsLayout {
    size_t linesum, colpart, inv_out, inv_in, layer_reg, maxbits, total;
};

constexpr int kThreads = 256;
constexpr int kMaxColsPerThread = 8;      // columns are walked in passes of TX*8

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---- phase 1
__global__ void __launch_bounds__(kThreads) norms_partial_kernel(const LayerDev *__restrict__ layers,
                                                                 const Chunk *__restrict__ chunks,
                                                                 float *__restrict__ linesum, float *__restrict__ colpart)
{
    __shared__ float s_line[8];                 // per-warp partials of one line pass
    __shared__ float s_col[kThreads];
    const Chunk ch = chunks[blockIdx.x];
    const LayerDev L = layers[ch.layer];
    const int TX = 1 << L.tx_log2, TY = kThreads >> L.tx_log2;
    const int tx = threadIdx.x & (TX - 1), ty = threadIdx.x >> L.tx_log2;
    const int lane = threadIdx.x & 31;
    const int wx = tx >> 5, nwx = TX >> 5;      // warp index along the line, warps per line
    (void)s_line;
    float *cp = colpart + L.col_off + (size_t)ch.idx * L.C;
    float *ls = linesum + L.line_off;
    const int passes = (L.C + TX * kMaxColsPerThread - 1) / (TX * kMaxColsPerThread);
    for (int pass = 0; pass < passes; ++pass) {
        const int cbase = pass * TX * kMaxColsPerThread + tx;
        float cacc[kMaxColsPerThread];
#pragma unroll
        for (int j = 0; j < kMaxColsPerThread; ++j) cacc[j] = 0.f;
        for (int l = ty; l < ch.nlines; l += TY) {
            const float *row = L.w + (size_t)(ch.line0 + l) * L.C;
            float racc = 0.f;
#pragma unroll
            for (int j = 0; j < kMaxColsPerThread; ++j) {
                int c = cbase + j * TX;
                if (c < L.C) {
                    float a = row[c];
                    float sq = a * a;
                    cacc[j] += sq;
                    racc += sq;
                }
            }
            racc = warp_sum(racc);
            // one partial per (line, warp-along-line, pass): summed in fixed order by phase 2
            if (lane == 0) ls[((size_t)(ch.line0 + l) * passes + pass) * nwx + wx] = racc;
        }
        // combine the TY line-groups' column partials in fixed order through shared memory
#pragma unroll
        for (int j = 0; j < kMaxColsPerThread; ++j) {
            __syncthreads();
            s_col[threadIdx.x] = cacc[j];
            __syncthreads();
            int c = cbase + j * TX;
            if (ty == 0 && c < L.C) {
                float s = 0.f;
                for (int y = 0; y < TY; ++y) s += s_col[y * TX + tx];
                cp[c] = s;
            }
        }
    }
}

// ---- phase 2: one block per layer
__global__ void __launch_bounds__(kThreads) norms_finish_kernel(const LayerDev *__restrict__ layers,
                                                                const float *__restrict__ linesum,
                                                                const float *__restrict__ colpart,
                                                                float *__restrict__ inv_out, float *__restrict__ inv_in,
                                                                double *__restrict__ layer_reg)
{
    __shared__ double s_red[kThreads];
    const LayerDev L = layers[blockIdx.x];
    const int TX = 1 << L.tx_log2;
    const int nwx = TX >> 5;
    const int passes = (L.C + TX * kMaxColsPerThread - 1) / (TX * kMaxColsPerThread);
    const int per_line = passes * nwx;
    double reg = 0.0;
    for (int k = threadIdx.x; k < L.K; k += kThreads) {
        const float *p = linesum + L.line_off + (size_t)k * L.RS * per_line;
        float s = 0.f;
        for (int i = 0; i < L.RS * per_line; ++i) s += p[i];
        L.sumsq_out[k] = s;
        float inv = (L.reg_out && s > 1e-24f) ? rsqrtf(s) : 0.f;
        inv_out[L.k_off + k] = inv;
        if (L.reg_out) reg += (double)sqrtf(s);
    }
    for (int c = threadIdx.x; c < L.C; c += kThreads) {
        const float *p = colpart + L.col_off + c;
        float s = 0.f;
        for (int i = 0; i < L.n_chunks; ++i) s += p[(size_t)i * L.C];
        L.sumsq_in[c] = s;
        float inv = (L.reg_in && s > 1e-24f) ? rsqrtf(s) : 0.f;
        inv_in[L.c_off + c] = inv;
        if (L.reg_in) reg += (double)sqrtf(s);
    }
    s_red[threadIdx.x] = reg;
    __syncthreads();
    for (int o = kThreads / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) s_red[threadIdx.x] += s_red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) layer_reg[blockIdx.x] = s_red[0];
}

// ---- phase 3
__global__ void reg_total_kernel(const double *__restrict__ layer_reg, int n, double *__restrict__ out)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        double s = 0.0;
        for (int i = 0; i < n; ++i) s += layer_reg[i];
        *out = s;
    }
}

// ---- phase 4
__global__ void __launch_bounds__(kThreads) update_kernel(const LayerDev *__restrict__ layers,
                                                          const Chunk *__restrict__ chunks,
                                                          const float *__restrict__ inv_out,
                                                          const float *__restrict__ inv_in, pt_sgd_hparams hp)
{
    const Chunk ch = chunks[blockIdx.x];
    const LayerDev L = layers[ch.layer];
    const int TX = 1 << L.tx_log2, TY = kThreads >> L.tx_log2;
    const int tx = threadIdx.x & (TX - 1), ty = threadIdx.x >> L.tx_log2;
    const float *io = inv_out + L.k_off;
    const float *ii = inv_in + L.c_off;
    const int passes = (L.C + TX * kMaxColsPerThread - 1) / (TX * kMaxColsPerThread);
    for (int pass = 0; pass < passes; ++pass) {
        const int cbase = pass * TX * kMaxColsPerThread + tx;
        float ci[kMaxColsPerThread];
#pragma unroll
        for (int j = 0; j < kMaxColsPerThread; ++j) {
            int c = cbase + j * TX;
            ci[j] = (c < L.C) ? ii[c] : 0.f;
        }
        for (int l = ty; l < ch.nlines; l += TY) {
            const int line = ch.line0 + l;
            const float ko = io[line / L.RS];
            const size_t base = (size_t)line * L.C;
            const size_t sbase = (size_t)line * L.ldw;
#pragma unroll
            for (int j = 0; j < kMaxColsPerThread; ++j) {
                int c = cbase + j * TX;
                if (c < L.C) {
                    float w = L.w[base + c], g = L.g[base + c], v = L.v[base + c];
                    float gt = g + hp.weight_decay * w + hp.lambda * w * (ko + ci[j]);
                    float vn = hp.momentum * v + gt;
                    float wn = w - hp.lr * vn;
                    L.v[base + c] = vn;
                    L.w[base + c] = wn;
                    if (L.wb) L.wb[sbase + c] = __float2bfloat16_rn(wn);
                }
            }
        }
    }
}

// ---- detection
__global__ void __launch_bounds__(kThreads) absmax_kernel(const LayerDev *__restrict__ layers,
                                                          const Chunk *__restrict__ chunks, unsigned int *__restrict__ maxbits)
{
    const Chunk ch = chunks[blockIdx.x];
    const LayerDev L = layers[ch.layer];
    const int TX = 1 << L.tx_log2, TY = kThreads >> L.tx_log2;
    const int tx = threadIdx.x & (TX - 1), ty = threadIdx.x >> L.tx_log2;
    const int lane = threadIdx.x & 31;
    unsigned int *mk = maxbits + L.k_off + L.c_off;         // this layer's K entries, then its C entries
    unsigned int *mc = mk + L.K;
    const int passes = (L.C + TX * kMaxColsPerThread - 1) / (TX * kMaxColsPerThread);
    for (int pass = 0; pass < passes; ++pass) {
        const int cbase = pass * TX * kMaxColsPerThread + tx;
        unsigned int cm[kMaxColsPerThread];
#pragma unroll
        for (int j = 0; j < kMaxColsPerThread; ++j) cm[j] = 0u;
        for (int l = ty; l < ch.nlines; l += TY) {
            const int line = ch.line0 + l;
            const float *row = L.w + (size_t)line * L.C;
            unsigned int rm = 0u;
#pragma unroll
            for (int j = 0; j < kMaxColsPerThread; ++j) {
                int c = cbase + j * TX;
                if (c < L.C) {
                    // |w| as its bit pattern: ordered like the value for finite numbers, and any NaN sorts above +inf
                    unsigned int bits = __float_as_uint(row[c]) & 0x7fffffffu;
                    cm[j] = max(cm[j], bits);
                    rm = max(rm, bits);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) rm = max(rm, __shfl_xor_sync(0xffffffffu, rm, o));
            if (lane == 0 && rm) atomicMax(&mk[line / L.RS], rm);
        }
#pragma unroll
        for (int j = 0; j < kMaxColsPerThread; ++j) {
            int c = cbase + j * TX;
            if (c < L.C && cm[j]) atomicMax(&mc[c], cm[j]);
        }
    }
}

__global__ void masks_kernel(const LayerDev *__restrict__ layers, const unsigned int *__restrict__ maxbits, float thr)
{
    const LayerDev L = layers[blockIdx.x];
    const unsigned int *mk = maxbits + L.k_off + L.c_off;
    const unsigned int *mc = mk + L.K;
    // strict "<" on the fp32 value; a NaN compares false, so its groups are kept
    for (int k = threadIdx.x; k < L.K; k += blockDim.x) L.zero_out[k] = (__uint_as_float(mk[k]) < thr) ? 1 : 0;
    for (int c = threadIdx.x; c < L.C; c += blockDim.x) L.zero_in[c] = (__uint_as_float(mc[c]) < thr) ? 1 : 0;
}

__global__ void __launch_bounds__(kThreads) zero_groups_kernel(const LayerDev *__restrict__ layers, const Chunk *__restrict__ chunks)
{
    const Chunk ch = chunks[blockIdx.x];
    const LayerDev L = layers[ch.layer];
    const int TX = 1 << L.tx_log2, TY = kThreads >> L.tx_log2;
    const int tx = threadIdx.x & (TX - 1), ty = threadIdx.x >> L.tx_log2;
    for (int l = ty; l < ch.nlines; l += TY) {
        const int line = ch.line0 + l;
        const bool zk = L.zero_out[line / L.RS] != 0;
        for (int c = tx; c < L.C; c += TX) {
            if (zk || L.zero_in[c]) {
                L.w[(size_t)line * L.C + c] = 0.f;
                L.v[(size_t)line * L.C + c] = 0.f;
                if (L.wb) L.wb[(size_t)line * L.ldw + c] = __float2bfloat16_rn(0.f);
            }
        }
    }
}

// ---------------------------------------------------------------------------------- host side
struct Tables {
    std::vector<LayerDev> layers;
    std::vector<Chunk> chunks;
    WsLayout ws;
};

constexpr int kChunkElems = 32768;

pt_status build_tables(const pt_layer *layers, int n, Tables *t)
{
    if (!layers || n <= 0) return PT_ERR_INVALID_ARG;
    t->layers.resize(n);
    t->chunks.clear();
    long long line_off = 0, col_off = 0, k_off = 0, c_off = 0;
    for (int i = 0; i < n; ++i) {
        const pt_layer &s = layers[i];
        if (!s.w || !s.v || s.K <= 0 || s.C <= 0 || s.RS <= 0) return PT_ERR_INVALID_ARG;
        if (s.w_bf16 && (s.ldw < s.C || s.ldw % 8)) return PT_ERR_INVALID_ARG;
        if ((long long)s.K * s.RS * (long long)(s.ldw > s.C ? s.ldw : s.C) >= (1ll << 31)) return PT_ERR_UNSUPPORTED;
        LayerDev &d = t->layers[i];
        d.w = s.w; d.g = s.g; d.v = s.v; d.wb = (__nv_bfloat16 *)s.w_bf16;
        d.sumsq_out = s.sumsq_out; d.sumsq_in = s.sumsq_in; d.zero_out = s.zero_out; d.zero_in = s.zero_in;
        d.K = s.K; d.C = s.C; d.RS = s.RS; d.ldw = s.ldw;
        d.reg_in = s.reg_in; d.reg_out = s.reg_out;
        int lg = 5;
        while ((1 << lg) < s.C && lg < 8) ++lg;
        d.tx_log2 = lg;
        d.pad_ = 0;
        const int TX = 1 << lg, TY = kThreads / TX;
        const int lines = s.K * s.RS;
        int lines_per_chunk = kChunkElems / s.C;
        if (lines_per_chunk < TY) lines_per_chunk = TY;
        lines_per_chunk = pt_ceil_div(lines_per_chunk, TY) * TY;
        d.chunk0 = (int)t->chunks.size();
        d.n_chunks = pt_ceil_div(lines, lines_per_chunk);
        for (int c = 0; c < d.n_chunks; ++c) {
            Chunk ch;
            ch.layer = i; ch.line0 = c * lines_per_chunk;
            ch.nlines = lines - ch.line0 < lines_per_chunk ? lines - ch.line0 : lines_per_chunk;
            ch.idx = c;
            t->chunks.push_back(ch);
        }
        const int passes = pt_ceil_div(s.C, TX * kMaxColsPerThread);
        d.line_off = line_off; line_off += (long long)lines * passes * (TX / 32);
        d.col_off = col_off;   col_off += (long long)d.n_chunks * s.C;
        d.k_off = k_off;       k_off += s.K;
        d.c_off = c_off;       c_off += s.C;
    }
    WsLayout &w = t->ws;
    size_t o = 0;
    w.linesum = o;   o = pt_align_up(o + (size_t)line_off * 4, 256);
    w.colpart = o;   o = pt_align_up(o + (size_t)col_off * 4, 256);
    w.inv_out = o;   o = pt_align_up(o + (size_t)k_off * 4, 256);
    w.inv_in = o;    o = pt_align_up(o + (size_t)c_off * 4, 256);
    w.layer_reg = o; o = pt_align_up(o + (size_t)n * 8, 256);
    w.maxbits = o;   o = pt_align_up(o + (size_t)(k_off + c_off) * 4, 256);
    w.total = o;
    return PT_OK;
}

// Uploads [LayerDev * n][Chunk * m] and returns device pointers.
pt_status upload(pt_ctx *c, const Tables &t, cudaStream_t st, const LayerDev **dl, const Chunk **dc)
{
    size_t lb = pt_align_up(t.layers.size() * sizeof(LayerDev), 256), cb = t.chunks.size() * sizeof(Chunk);
    std::vector<char> buf(lb + cb, 0);
    memcpy(buf.data(), t.layers.data(), t.layers.size() * sizeof(LayerDev));
    memcpy(buf.data() + lb, t.chunks.data(), cb);
    char *dev = nullptr;
    pt_status s = pt_upload_table(c, &c->lasso_tab, buf.data(), buf.size(), st, &dev);
    if (s != PT_OK) return s;
    *dl = (const LayerDev *)dev;
    *dc = (const Chunk *)(dev + lb);
    return PT_OK;
}

}  // namespace

extern "C" size_t pt_group_lasso_workspace_bytes(const pt_ctx *c, const pt_layer *layers, int32_t n)
{
    (void)c;
    Tables t;
    if (build_tables(layers, n, &t) != PT_OK) return 0;
    return t.ws.total;
}

extern "C" pt_status pt_group_lasso_sgd_step(pt_ctx *c, const pt_layer *layers, int32_t n, const pt_sgd_hparams *hp,
                                             double *reg_sum_out, void *ws, size_t ws_bytes, void *stream)
{
    if (!c || !hp) return PT_ERR_INVALID_ARG;
    Tables t;
    pt_status s = build_tables(layers, n, &t);
    if (s != PT_OK) return s;
    for (int i = 0; i < n; ++i)
        if (!layers[i].g || !layers[i].sumsq_out || !layers[i].sumsq_in) return PT_ERR_INVALID_ARG;
    if (!ws || ws_bytes < t.ws.total || ((uintptr_t)ws & 255)) return PT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const LayerDev *dl; const Chunk *dc;
    s = upload(c, t, st, &dl, &dc);
    if (s != PT_OK) return s;
    char *b = (char *)ws;
    float *linesum = (float *)(b + t.ws.linesum), *colpart = (float *)(b + t.ws.colpart);
    float *inv_out = (float *)(b + t.ws.inv_out), *inv_in = (float *)(b + t.ws.inv_in);
    double *layer_reg = (double *)(b + t.ws.layer_reg);
    const unsigned nch = (unsigned)t.chunks.size();
    norms_partial_kernel<<<nch, kThreads, 0, st>>>(dl, dc, linesum, colpart);
    norms_finish_kernel<<<n, kThreads, 0, st>>>(dl, linesum, colpart, inv_out, inv_in, layer_reg);
    c->launches += 2;
    if (reg_sum_out) { reg_total_kernel<<<1, 32, 0, st>>>(layer_reg, n, reg_sum_out); c->launches += 1; }
    update_kernel<<<nch, kThreads, 0, st>>>(dl, dc, inv_out, inv_in, *hp);
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

extern "C" pt_status pt_find_zero_groups(pt_ctx *c, const pt_layer *layers, int32_t n, float threshold,
                                         int32_t zero_in_place, void *ws, size_t ws_bytes, void *stream)
{
    if (!c || !(threshold >= 0.f)) return PT_ERR_INVALID_ARG;
    Tables t;
    pt_status s = build_tables(layers, n, &t);
    if (s != PT_OK) return s;
    for (int i = 0; i < n; ++i)
        if (!layers[i].zero_out || !layers[i].zero_in) return PT_ERR_INVALID_ARG;
    if (!ws || ws_bytes < t.ws.total || ((uintptr_t)ws & 255)) return PT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const LayerDev *dl; const Chunk *dc;
    s = upload(c, t, st, &dl, &dc);
    if (s != PT_OK) return s;
    unsigned int *maxbits = (unsigned int *)((char *)ws + t.ws.maxbits);
    PT_CUDA_OK(cudaMemsetAsync(maxbits, 0, t.ws.total - t.ws.maxbits, st));
    const unsigned nch = (unsigned)t.chunks.size();
    absmax_kernel<<<nch, kThreads, 0, st>>>(dl, dc, maxbits);
    masks_kernel<<<n, 256, 0, st>>>(dl, maxbits, threshold);
    c->launches += 2;
    if (zero_in_place) { zero_groups_kernel<<<nch, kThreads, 0, st>>>(dl, dc); c->launches += 1; }
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}
