// Group-lasso regularised momentum SGD over all conv weights (Eq. 1-2, Algorithm 1) and
// zero-group detection (Sec. 4.1 threshold, Sec. 4.2 max-abs per channel).
//
// All layers are processed by one launch per phase through a chunk table. A weight tensor
// [K][RS][C] is seen as K*RS "lines" of C contiguous floats; a chunk is a run of lines of one
// layer restricted to a block of TX <= 256 columns. Inside a block, thread (tx, ty) owns column
// col0 + tx and the lines ty, ty+TY, ... of its chunk (four lines in flight per thread), so every
// access is a coalesced run of a line and per-column quantities stay in registers.
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
    int tx_log2;                // TX = 1 << tx_log2 threads along a line (32..256): one column per thread
    int n_cb;                   // column blocks of TX columns
    int n_lc;                   // line chunks
    int pad_;
    long long line_off;         // offset of this layer's per-line partials (lines * n_cb floats)
    long long col_off;          // offset of this layer's column partials (n_lc * C floats)
    long long k_off, c_off;     // offsets into the per-K / per-C scratch arrays
};

// A chunk is a run of lines of one layer restricted to one block of TX columns.
struct Chunk { int layer, line0, nlines, col0, lc, cb, pad0, pad1; };

struct WsLayout {
    size_t linesum, colpart, inv_out, inv_in, layer_reg, maxbits, total;
};

constexpr int kThreads = 256;
constexpr int kUnroll = 8;                // lines in flight per thread
constexpr int kSweeps = 4;                // unrolled sweeps per chunk: every block does the same number of iterations
constexpr int kUpdateSplit = 2;           // blocks per chunk in the update kernel

// Eight per-lane values (one per line) are reduced over the 32 lanes with 9 shuffles instead of 40: three
// halving exchanges leave lane l with the partial of line (l >> 2) & 7 over its 4-lane group's share, two more
// add the four lanes of a group. The tree is fixed, so the result is run-to-run identical.
// Returns the total of line ((lane >> 2) & 7), valid in every lane.
template <typename T, typename Op>
__device__ __forceinline__ T warp_reduce8(T (&v)[8], int lane, Op op)
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const bool hi = lane & 16;
        const T send = hi ? v[i] : v[i + 4], keep = hi ? v[i + 4] : v[i];
        v[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, 16));
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const bool hi = lane & 8;
        const T send = hi ? v[i] : v[i + 2], keep = hi ? v[i + 2] : v[i];
        v[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, 8));
    }
    {
        const bool hi = lane & 4;
        const T send = hi ? v[0] : v[1], keep = hi ? v[1] : v[0];
        v[0] = op(keep, __shfl_xor_sync(0xffffffffu, send, 4));
    }
    v[0] = op(v[0], __shfl_xor_sync(0xffffffffu, v[0], 2));
    v[0] = op(v[0], __shfl_xor_sync(0xffffffffu, v[0], 1));
    return v[0];
}
struct OpAdd { __device__ __forceinline__ float operator()(float a, float b) const { return a + b; } };
struct OpMax { __device__ __forceinline__ unsigned int operator()(unsigned int a, unsigned int b) const { return a > b ? a : b; } };

// ---- phase 1
__global__ void __launch_bounds__(kThreads) norms_partial_kernel(const LayerDev *__restrict__ layers,
                                                                 const Chunk *__restrict__ chunks,
                                                                 float *__restrict__ linesum, float *__restrict__ colpart)
{
    __shared__ float s_col[kThreads];
    __shared__ float s_line[2 * kThreads];       // [line in chunk][warp along the line]: at most 64 lines per TY x 8 warps
    const Chunk ch = chunks[blockIdx.x];
    const LayerDev L = layers[ch.layer];
    const int TX = 1 << L.tx_log2, TY = kThreads >> L.tx_log2;
    const int tx = threadIdx.x & (TX - 1), ty = threadIdx.x >> L.tx_log2;
    const int lane = threadIdx.x & 31;
    const int wx = tx >> 5, nwx = TX >> 5;
    const int c = ch.col0 + tx;
    const bool cv = c < L.C;
    const float *wbase = L.w + (size_t)ch.line0 * L.C + c;
    float cacc = 0.f;
    for (int l = ty; l < ch.nlines; l += kUnroll * TY) {
        float a[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int ll = l + u * TY;
            a[u] = (cv && ll < ch.nlines) ? wbase[(size_t)ll * L.C] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            a[u] *= a[u];
            cacc += a[u];
        }
        const float tot = warp_reduce8(a, lane, OpAdd());
        if ((lane & 3) == 0) {
            const int ll = l + ((lane >> 2) & 7) * TY;      // the lane's 4-lane group holds this line's total
            if (ll < ch.nlines) s_line[ll * nwx + wx] = tot;
        }
    }
    s_col[threadIdx.x] = cacc;
    __syncthreads();
    // one partial per (line, column block): the warps along a line are added in ascending order
    for (int ln = threadIdx.x; ln < ch.nlines; ln += kThreads) {
        float s = 0.f;
        for (int x = 0; x < nwx; ++x) s += s_line[ln * nwx + x];
        linesum[L.line_off + (size_t)(ch.line0 + ln) * L.n_cb + ch.cb] = s;
    }
    // combine the TY line groups' column partials in fixed order
    if (ty == 0 && cv) {
        float s = 0.f;
        for (int y = 0; y < TY; ++y) s += s_col[y * TX + tx];
        colpart[L.col_off + (size_t)ch.lc * L.C + c] = s;
    }
}

// ---- phase 2: one block per 256 groups of one layer (kind 0: output-channel groups, kind 1: input-channel groups)
struct FinishJob { int layer, kind, start, pad; };

__global__ void __launch_bounds__(kThreads) norms_finish_kernel(const LayerDev *__restrict__ layers,
                                                                const FinishJob *__restrict__ jobs,
                                                                const float *__restrict__ linesum,
                                                                const float *__restrict__ colpart,
                                                                float *__restrict__ inv_out, float *__restrict__ inv_in,
                                                                double *__restrict__ job_reg)
{
    __shared__ double s_red[kThreads];
    const FinishJob J = jobs[blockIdx.x];
    const LayerDev L = layers[J.layer];
    const int per_line = L.n_cb;
    double reg = 0.0;
    const int i = J.start + threadIdx.x;
    if (J.kind == 0) {
        if (i < L.K) {
            const float *p = linesum + L.line_off + (size_t)i * L.RS * per_line;
            float s = 0.f;
#pragma unroll 8
            for (int e = 0; e < L.RS * per_line; ++e) s += p[e];           // fixed order
            L.sumsq_out[i] = s;
            inv_out[L.k_off + i] = (L.reg_out && s > 1e-24f) ? rsqrtf(s) : 0.f;
            if (L.reg_out) reg = (double)sqrtf(s);
        }
    } else {
        if (i < L.C) {
            const float *p = colpart + L.col_off + i;
            float s = 0.f;
#pragma unroll 8
            for (int e = 0; e < L.n_lc; ++e) s += p[(size_t)e * L.C];        // fixed order
            L.sumsq_in[i] = s;
            inv_in[L.c_off + i] = (L.reg_in && s > 1e-24f) ? rsqrtf(s) : 0.f;
            if (L.reg_in) reg = (double)sqrtf(s);
        }
    }
    s_red[threadIdx.x] = reg;
    __syncthreads();
    for (int o = kThreads / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) s_red[threadIdx.x] += s_red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) job_reg[blockIdx.x] = s_red[0];
}

// ---- phase 3
__global__ void reg_total_kernel(const double *__restrict__ job_reg, int n, double *__restrict__ out)
{
    // 32 lanes take strided slices, then a fixed shuffle tree: the same order on every run
    double s = 0.0;
    for (int i = threadIdx.x; i < n; i += 32) s += job_reg[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (threadIdx.x == 0) *out = s;
}

// ---- phase 4
__global__ void __launch_bounds__(kThreads) update_kernel(const LayerDev *__restrict__ layers,
                                                          const Chunk *__restrict__ chunks,
                                                          const float *__restrict__ inv_out,
                                                          const float *__restrict__ inv_in, pt_sgd_hparams hp)
{
    // kUpdateSplit blocks share a chunk (alternate sweeps): the update has no per-chunk results to combine, and the finer
    // grain wastes less of the last wave
    const Chunk ch = chunks[blockIdx.x / kUpdateSplit];
    const int sub = blockIdx.x % kUpdateSplit;
    const LayerDev L = layers[ch.layer];
    const int TX = 1 << L.tx_log2, TY = kThreads >> L.tx_log2;
    const int tx = threadIdx.x & (TX - 1), ty = threadIdx.x >> L.tx_log2;
    const int c = ch.col0 + tx;
    if (c >= L.C) return;
    const float ci = inv_in[L.c_off + c];
    const float *io = inv_out + L.k_off;
    for (int l = ty + sub * kUnroll * TY; l < ch.nlines; l += kUpdateSplit * kUnroll * TY) {
        float w[kUnroll], g[kUnroll], v[kUnroll], ko[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int line = ch.line0 + l + u * TY;
            if (l + u * TY < ch.nlines) {
                const size_t i = (size_t)line * L.C + c;
                w[u] = L.w[i]; g[u] = L.g[i]; v[u] = L.v[i];
                ko[u] = io[line / L.RS];
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int line = ch.line0 + l + u * TY;
            if (l + u * TY < ch.nlines) {
                const size_t i = (size_t)line * L.C + c;
                const float gt = g[u] + hp.weight_decay * w[u] + hp.lambda * w[u] * (ko[u] + ci);
                const float vn = hp.momentum * v[u] + gt;
                const float wn = w[u] - hp.lr * vn;
                L.v[i] = vn;
                L.w[i] = wn;
                if (L.wb) L.wb[(size_t)line * L.ldw + c] = __float2bfloat16_rn(wn);
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
    __shared__ unsigned int s_line[2 * kThreads];
    unsigned int *mk = maxbits + L.k_off + L.c_off;         // this layer's K entries, then its C entries
    unsigned int *mc = mk + L.K;
    const int wx = tx >> 5, nwx = TX >> 5;
    const int c = ch.col0 + tx;
    const bool cv = c < L.C;
    const float *wbase = L.w + (size_t)ch.line0 * L.C + c;
    unsigned int cm = 0u;
    for (int l = ty; l < ch.nlines; l += kUnroll * TY) {
        unsigned int b[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int ll = l + u * TY;
            // |w| as its bit pattern: ordered like the value for finite numbers, and any NaN sorts above +inf
            b[u] = (cv && ll < ch.nlines) ? (__float_as_uint(wbase[(size_t)ll * L.C]) & 0x7fffffffu) : 0u;
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) cm = max(cm, b[u]);
        const unsigned int tot = warp_reduce8(b, lane, OpMax());
        if ((lane & 3) == 0) {
            const int ll = l + ((lane >> 2) & 7) * TY;
            if (ll < ch.nlines) s_line[ll * nwx + wx] = tot;
        }
    }
    __syncthreads();
    for (int ln = threadIdx.x; ln < ch.nlines; ln += kThreads) {
        unsigned int m = 0u;
        for (int x = 0; x < nwx; ++x) m = max(m, s_line[ln * nwx + x]);
        if (m) atomicMax(&mk[(ch.line0 + ln) / L.RS], m);
    }
    if (cv && cm) atomicMax(&mc[c], cm);
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
    const int c = ch.col0 + tx;
    if (c >= L.C) return;
    const bool zc = L.zero_in[c] != 0;
    for (int l = ty; l < ch.nlines; l += TY) {
        const int line = ch.line0 + l;
        if (zc || L.zero_out[line / L.RS]) {
            L.w[(size_t)line * L.C + c] = 0.f;
            L.v[(size_t)line * L.C + c] = 0.f;
            if (L.wb) L.wb[(size_t)line * L.ldw + c] = __float2bfloat16_rn(0.f);
        }
    }
}

// ---------------------------------------------------------------------------------- host side
struct Tables {
    std::vector<LayerDev> layers;
    std::vector<Chunk> chunks;
    std::vector<FinishJob> jobs;
    WsLayout ws;
};


pt_status build_tables(const pt_layer *layers, int n, Tables *t)
{
    if (!layers || n <= 0) return PT_ERR_INVALID_ARG;
    t->layers.resize(n);
    t->chunks.clear();
    t->jobs.clear();
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
        // a chunk is TY*kUnroll*sweeps lines x TX columns; sweeps = 4 (8192 thread slots), more for tall tensors so that no
        // column has more than ~32 chunk partials to add up in phase 2 (the s_line staging holds at most 256 lines x warps)
        int sweeps = kSweeps;
        while (sweeps < 8 && lines > 32 * TY * kUnroll * sweeps) sweeps *= 2;
        const int lines_per_chunk = TY * kUnroll * sweeps;
        d.n_cb = pt_ceil_div(s.C, TX);
        d.n_lc = pt_ceil_div(lines, lines_per_chunk);
        for (int lc = 0; lc < d.n_lc; ++lc)
            for (int cb = 0; cb < d.n_cb; ++cb) {
                Chunk ch;
                ch.layer = i; ch.line0 = lc * lines_per_chunk;
                ch.nlines = lines - ch.line0 < lines_per_chunk ? lines - ch.line0 : lines_per_chunk;
                ch.col0 = cb * TX; ch.lc = lc; ch.cb = cb; ch.pad0 = ch.pad1 = 0;
                t->chunks.push_back(ch);
            }
        for (int k0 = 0; k0 < s.K; k0 += kThreads) t->jobs.push_back(FinishJob{i, 0, k0, 0});
        for (int c0 = 0; c0 < s.C; c0 += kThreads) t->jobs.push_back(FinishJob{i, 1, c0, 0});
        d.line_off = line_off; line_off += (long long)lines * d.n_cb;
        d.col_off = col_off;   col_off += (long long)d.n_lc * s.C;
        d.k_off = k_off;       k_off += s.K;
        d.c_off = c_off;       c_off += s.C;
    }
    WsLayout &w = t->ws;
    size_t o = 0;
    w.linesum = o;   o = pt_align_up(o + (size_t)line_off * 4, 256);
    w.colpart = o;   o = pt_align_up(o + (size_t)col_off * 4, 256);
    w.inv_out = o;   o = pt_align_up(o + (size_t)k_off * 4, 256);
    w.inv_in = o;    o = pt_align_up(o + (size_t)c_off * 4, 256);
    w.layer_reg = o; o = pt_align_up(o + t->jobs.size() * 8, 256);
    w.maxbits = o;   o = pt_align_up(o + (size_t)(k_off + c_off) * 4, 256);
    w.total = o;
    return PT_OK;
}

// Uploads [LayerDev * n][Chunk * m] and returns device pointers.
pt_status upload(pt_ctx *c, const Tables &t, bool detect, cudaStream_t st, const LayerDev **dl, const Chunk **dc,
                 const FinishJob **dj)
{
    size_t lb = pt_align_up(t.layers.size() * sizeof(LayerDev), 256), cb = pt_align_up(t.chunks.size() * sizeof(Chunk), 256);
    size_t jb = t.jobs.size() * sizeof(FinishJob);
    std::vector<char> buf(lb + cb + jb, 0);
    memcpy(buf.data(), t.layers.data(), t.layers.size() * sizeof(LayerDev));
    memcpy(buf.data() + lb, t.chunks.data(), t.chunks.size() * sizeof(Chunk));
    memcpy(buf.data() + lb + cb, t.jobs.data(), jb);
    char *dev = nullptr;
    pt_status s = detect ? pt_upload_table_slots(c, c->detect_tab, 2, &c->detect_next, buf.data(), buf.size(), st, &dev)
                         : pt_upload_table_slots(c, c->lasso_tab, 3, &c->lasso_next, buf.data(), buf.size(), st, &dev);
    if (s != PT_OK) return s;
    *dl = (const LayerDev *)dev;
    *dc = (const Chunk *)(dev + lb);
    *dj = (const FinishJob *)(dev + lb + cb);
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

// phases: 1 = group norms (partial sums, finish, regulariser value), 2 = parameter update from the norms in the workspace
// The update may be restricted to layers [first, first + count) (count < 0: all): the chunk table is ordered by layer.
static pt_status lasso_phases(pt_ctx *c, const pt_layer *layers, int32_t n, const pt_sgd_hparams *hp, double *reg_sum_out, void *ws,
                              size_t ws_bytes, void *stream, int phases, int first = 0, int count = -1)
{
    if (!c || ((phases & 2) && !hp)) return PT_ERR_INVALID_ARG;
    if (count >= 0 && (first < 0 || first + count > n)) return PT_ERR_INVALID_ARG;
    Tables t;
    pt_status s = build_tables(layers, n, &t);
    if (s != PT_OK) return s;
    for (int i = 0; i < n; ++i)
        if (((phases & 2) && !layers[i].g) || !layers[i].sumsq_out || !layers[i].sumsq_in) return PT_ERR_INVALID_ARG;
    if (!ws || ws_bytes < t.ws.total || ((uintptr_t)ws & 255)) return PT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const LayerDev *dl; const Chunk *dc; const FinishJob *dj;
    s = upload(c, t, false, st, &dl, &dc, &dj);
    if (s != PT_OK) return s;
    char *b = (char *)ws;
    float *linesum = (float *)(b + t.ws.linesum), *colpart = (float *)(b + t.ws.colpart);
    float *inv_out = (float *)(b + t.ws.inv_out), *inv_in = (float *)(b + t.ws.inv_in);
    double *layer_reg = (double *)(b + t.ws.layer_reg);
    const unsigned nch = (unsigned)t.chunks.size();
    if (phases & 1) {
        norms_partial_kernel<<<nch, kThreads, 0, st>>>(dl, dc, linesum, colpart);
        const int nj = (int)t.jobs.size();
        norms_finish_kernel<<<nj, kThreads, 0, st>>>(dl, dj, linesum, colpart, inv_out, inv_in, layer_reg);
        c->launches += 2;
        if (reg_sum_out) { reg_total_kernel<<<1, 32, 0, st>>>(layer_reg, nj, reg_sum_out); c->launches += 1; }
    }
    if (phases & 2) {
        unsigned c0 = 0, c1 = nch;
        if (count >= 0) {
            c0 = nch; c1 = 0;
            for (unsigned i = 0; i < nch; ++i)
                if (t.chunks[i].layer >= first && t.chunks[i].layer < first + count) { c0 = i < c0 ? i : c0; c1 = i + 1; }
        }
        if (c1 > c0) {
            update_kernel<<<(c1 - c0) * kUpdateSplit, kThreads, 0, st>>>(dl, dc + c0, inv_out, inv_in, *hp);
            c->launches += 1;
        }
    }
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

extern "C" pt_status pt_group_lasso_sgd_step(pt_ctx *c, const pt_layer *layers, int32_t n, const pt_sgd_hparams *hp,
                                             double *reg_sum_out, void *ws, size_t ws_bytes, void *stream)
{
    return lasso_phases(c, layers, n, hp, reg_sum_out, ws, ws_bytes, stream, 3);
}

extern "C" pt_status pt_group_lasso_norms(pt_ctx *c, const pt_layer *layers, int32_t n, double *reg_sum_out, void *ws,
                                          size_t ws_bytes, void *stream)
{
    return lasso_phases(c, layers, n, nullptr, reg_sum_out, ws, ws_bytes, stream, 1);
}

extern "C" pt_status pt_group_lasso_sgd_apply(pt_ctx *c, const pt_layer *layers, int32_t n, const pt_sgd_hparams *hp, void *ws,
                                              size_t ws_bytes, void *stream)
{
    return lasso_phases(c, layers, n, hp, nullptr, ws, ws_bytes, stream, 2);
}

extern "C" pt_status pt_group_lasso_sgd_apply_layers(pt_ctx *c, const pt_layer *layers, int32_t n, int32_t first, int32_t count,
                                                     const pt_sgd_hparams *hp, void *ws, size_t ws_bytes, void *stream)
{
    if (count < 0) return PT_ERR_INVALID_ARG;
    return lasso_phases(c, layers, n, hp, nullptr, ws, ws_bytes, stream, 2, first, count);
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
    const LayerDev *dl; const Chunk *dc; const FinishJob *dj;
    s = upload(c, t, true, st, &dl, &dc, &dj);
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
