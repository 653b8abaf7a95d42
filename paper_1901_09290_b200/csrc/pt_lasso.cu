// Group-lasso regularised momentum SGD over all conv weights (Eq. 1-2, Algorithm 1) and
// zero-group detection (Sec. 4.1 threshold, Sec. 4.2 max-abs per channel).
//
// All layers are processed by one launch per phase through a chunk table. A weight tensor
// [K][RS][C] is seen as K*RS "lines" of C contiguous floats; a chunk is a run of lines of one
// layer restricted to a block of TX columns. Inside a block, thread (tx, ty) owns column
// col0 + tx and the lines ty, ty+TY, ... of its chunk (eight lines in flight per thread), so every
// access is a coalesced run of a line and per-column quantities stay in registers. TX is a power of
// two between 32 and 256 chosen per layer for the fewest idle lanes (C = 143: five blocks of 32 columns,
// 89 % of the lanes busy, where one block of 256 has 56 %).
//
// One kernel template walks the chunks:
//   sweep<UPD, SUM, MAX>  UPD: g~, v, w, bf16 shadow (reads w, g, v; writes w, v, shadow)
//                         SUM: per line and per (chunk, column) sums of squares of the weights (the new ones with UPD)
//                         MAX: the same for the maxima of |w| (bit patterns: ordered like the values, a NaN sorts above +inf)
//   <0,1,0> group norms of W_i;  <1,0,0> the update;  <1,1,1> the carried update, which leaves the sums and maxima of
//   W_{i+1} so that the next step needs no pass over the weights of its own;  <0,0,1> zero-group detection.
//   finish   fixed-order combination to s_out[k], s_in[c], the 1/norm factors, the Eq. 2 sum (last block, by ticket), the
//            group maxima and, for the detection, the zero masks.
// No floating-point atomics and fixed reduction trees: results are run-to-run identical.
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
    long long line_off;         // offset of this layer's per-line partials (lines * n_cb)
    long long col_off;          // offset of this layer's column partials (n_lc * C)
    long long k_off, c_off;     // offsets into the per-K / per-C arrays
};

// A chunk is a run of lines of one layer restricted to one block of TX columns.
struct Chunk { int layer, line0, nlines, col0, lc, cb, pad0, pad1; };

// kind 0: 256 output-channel groups from `start`; kind 1: 32 input-channel groups from `start` (x 8 slices of the chunk partials)
struct FinishJob { int layer, kind, start, pad; };

struct WsLayout { size_t linesum, colpart, linemax, colmax, inv_out, inv_in, gmax_out, gmax_in, job_reg, ticket, total; };

constexpr int kThreads = 256;
constexpr int kUnroll = 8;                // lines in flight per thread
constexpr int kSweeps = 8;                // unrolled sweeps per chunk of a large model (16384 thread slots; 4 measured 4 % slower, 16 slower again)
constexpr int kSweepsSmall = 4;           // ... of a model with fewer than kSmallModel parameters (more, smaller blocks: 8 measured 7-10 % slower there)
constexpr long long kSmallModel = 12ll << 20;
// The plain update has no per-chunk results to combine: sweeps / 2 blocks share a chunk (two sweeps each).

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

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

// ---- the sweep over the chunks
template <bool UPD, bool SUM, bool MAX>
__global__ void __launch_bounds__(kThreads) sweep_kernel(const LayerDev *__restrict__ layers, const Chunk *__restrict__ chunks,
                                                         const float *__restrict__ inv_out, const float *__restrict__ inv_in,
                                                         pt_sgd_hparams hp, float *__restrict__ linesum, float *__restrict__ colpart,
                                                         unsigned *__restrict__ linemax, unsigned *__restrict__ colmax,
                                                         unsigned *__restrict__ ticket, int split)
{
    constexpr bool RED = SUM || MAX;
    const int SPLIT = RED ? 1 : split;                 // the plain update has no per-chunk results: `split` blocks share a chunk
    __shared__ float s_col[RED ? kThreads : 1];
    __shared__ unsigned s_colm[MAX ? kThreads : 1];
    __shared__ float s_line[SUM ? 2 * kThreads : 1];       // [line in chunk][warp along the line]: at most 64 lines per TY x 8 warps
    __shared__ unsigned s_linem[MAX ? 2 * kThreads : 1];
    const Chunk ch = chunks[blockIdx.x / SPLIT];
    const int sub = blockIdx.x % SPLIT;
    const LayerDev L = layers[ch.layer];
    const int TX = 1 << L.tx_log2, TY = kThreads >> L.tx_log2;
    const int tx = threadIdx.x & (TX - 1), ty = threadIdx.x >> L.tx_log2;
    const int lane = threadIdx.x & 31;
    const int wx = tx >> 5, nwx = TX >> 5;
    const int c = ch.col0 + tx;
    const bool cv = c < L.C;
    pdl_wait();
    // A sweep that writes the weights lets its dependents start only when it has completed: the convolution kernels' weight
    // producers do not wait for their predecessor (weights are never written by a kernel that releases its dependents early),
    // and a convolution may well be the next launch of the stream.
    if (!UPD) pdl_trigger();
    if (RED && blockIdx.x == 0 && threadIdx.x == 0) *ticket = 0u;          // for the finish kernel that follows
    float ci = 0.f;
    if (UPD && cv) ci = inv_in[L.c_off + c];
    const float *io = inv_out + L.k_off;
    float cacc = 0.f;
    unsigned cm = 0u;
    for (int l = ty + sub * kUnroll * TY; l < ch.nlines; l += SPLIT * kUnroll * TY) {
        float w[kUnroll], g[kUnroll], v[kUnroll], ko[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int ll = l + u * TY, line = ch.line0 + ll;
            w[u] = 0.f;
            if (cv && ll < ch.nlines) {
                const size_t i = (size_t)line * L.C + c;
                w[u] = L.w[i];
                if (UPD) { g[u] = L.g[i]; v[u] = L.v[i]; ko[u] = io[line / L.RS]; }
            }
        }
        if (UPD) {
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int ll = l + u * TY, line = ch.line0 + ll;
                if (cv && ll < ch.nlines) {
                    const size_t i = (size_t)line * L.C + c;
                    const float gt = g[u] + hp.weight_decay * w[u] + hp.lambda * w[u] * (ko[u] + ci);
                    const float vn = hp.momentum * v[u] + gt;
                    const float wn = w[u] - hp.lr * vn;
                    L.v[i] = vn;
                    L.w[i] = wn;
                    if (L.wb) L.wb[(size_t)line * L.ldw + c] = __float2bfloat16_rn(wn);
                    w[u] = wn;
                }
            }
        }
        if (MAX) {
            unsigned b[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) { b[u] = __float_as_uint(w[u]) & 0x7fffffffu; cm = max(cm, b[u]); }
            const unsigned tot = warp_reduce8(b, lane, OpMax());
            if ((lane & 3) == 0) {
                const int ll = l + ((lane >> 2) & 7) * TY;      // the lane's 4-lane group holds this line's total
                if (ll < ch.nlines) s_linem[ll * nwx + wx] = tot;
            }
        }
        if (SUM) {
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) { w[u] *= w[u]; cacc += w[u]; }
            const float tot = warp_reduce8(w, lane, OpAdd());
            if ((lane & 3) == 0) {
                const int ll = l + ((lane >> 2) & 7) * TY;
                if (ll < ch.nlines) s_line[ll * nwx + wx] = tot;
            }
        }
    }
    if (!RED) return;
    if (SUM) s_col[threadIdx.x] = cacc;
    if (MAX) s_colm[threadIdx.x] = cm;
    __syncthreads();
    // one partial per (line, column block): the warps along a line are combined in ascending order
    for (int ln = threadIdx.x; ln < ch.nlines; ln += kThreads) {
        const size_t o = L.line_off + (size_t)(ch.line0 + ln) * L.n_cb + ch.cb;
        if (SUM) {
            float s = 0.f;
            for (int x = 0; x < nwx; ++x) s += s_line[ln * nwx + x];
            linesum[o] = s;
        }
        if (MAX) {
            unsigned m = 0u;
            for (int x = 0; x < nwx; ++x) m = max(m, s_linem[ln * nwx + x]);
            linemax[o] = m;
        }
    }
    // the TY line groups' column partials in fixed order
    if (ty == 0 && cv) {
        const size_t o = L.col_off + (size_t)ch.lc * L.C + c;
        if (SUM) {
            float s = 0.f;
            for (int y = 0; y < TY; ++y) s += s_col[y * TX + tx];
            colpart[o] = s;
        }
        if (MAX) {
            unsigned m = 0u;
            for (int y = 0; y < TY; ++y) m = max(m, s_colm[y * TX + tx]);
            colmax[o] = m;
        }
    }
}

// ---- finish. flags: 1 = sums (sumsq, 1/norm factors, Eq. 2 value), 2 = maxima (group maxima kept in the workspace),
//      4 = zero masks from the maxima (strict "<" on the fp32 value; a NaN compares false and keeps its group)
__global__ void __launch_bounds__(kThreads) finish_kernel(const LayerDev *__restrict__ layers, const FinishJob *__restrict__ jobs,
                                                          const float *__restrict__ linesum, const float *__restrict__ colpart,
                                                          const unsigned *__restrict__ linemax, const unsigned *__restrict__ colmax,
                                                          float *__restrict__ inv_out, float *__restrict__ inv_in,
                                                          unsigned *__restrict__ gmax_out, unsigned *__restrict__ gmax_in,
                                                          double *__restrict__ job_reg, unsigned *__restrict__ ticket,
                                                          double *__restrict__ reg_out, int flags, float thr)
{
    __shared__ double s_red[kThreads];
    __shared__ float s_ps[8][32];
    __shared__ unsigned s_pm[8][32];
    __shared__ unsigned s_last;
    const FinishJob J = jobs[blockIdx.x];
    const LayerDev L = layers[J.layer];
    pdl_wait();
    pdl_trigger();
    double reg = 0.0;
    if (J.kind == 0) {
        const int i = J.start + (int)threadIdx.x;
        if (i < L.K) {
            if (flags & 1) {
                const int np = L.RS * L.n_cb;                             // one partial per (line, column block)
                const float *p = linesum + L.line_off + (long long)i * np;
                float s = 0.f;
                // (a thread's partials are consecutive, the lanes' are np apart: every load is a round trip to L2, so many are
                // kept in flight; a 3x3 layer has 9 to 72 of them, the 7x7 stem 49)
#pragma unroll 16
                for (int e = 0; e < np; ++e) s += p[e];                   // fixed order
                L.sumsq_out[i] = s;
                inv_out[L.k_off + i] = (L.reg_out && s > 1e-24f) ? rsqrtf(s) : 0.f;
                if (L.reg_out) reg = (double)sqrtf(s);
            }
            if (flags & 6) {
                const int np = L.RS * L.n_cb;
                const unsigned *p = linemax + L.line_off + (long long)i * np;
                unsigned m = 0u;
#pragma unroll 16
                for (int e = 0; e < np; ++e) m = max(m, p[e]);
                if (flags & 2) gmax_out[L.k_off + i] = m;
                if (flags & 4) L.zero_out[i] = (__uint_as_float(m) < thr) ? 1 : 0;
            }
        }
    } else {
        const int cx = threadIdx.x & 31, sy = threadIdx.x >> 5;
        const int c = J.start + cx;
        float s = 0.f;
        unsigned m = 0u;
        if (c < L.C) {
            if (flags & 1) {
                const float *p = colpart + L.col_off + c;
#pragma unroll 4
                for (int e = sy; e < L.n_lc; e += 8) s += p[(long long)e * L.C];      // this slice in ascending order
            }
            if (flags & 6) {
                const unsigned *p = colmax + L.col_off + c;
#pragma unroll 4
                for (int e = sy; e < L.n_lc; e += 8) m = max(m, p[(long long)e * L.C]);
            }
        }
        s_ps[sy][cx] = s;
        s_pm[sy][cx] = m;
        __syncthreads();
        if (sy == 0 && c < L.C) {
            if (flags & 1) {
                float t = 0.f;
#pragma unroll
                for (int y = 0; y < 8; ++y) t += s_ps[y][cx];              // the eight slices in ascending order
                L.sumsq_in[c] = t;
                inv_in[L.c_off + c] = (L.reg_in && t > 1e-24f) ? rsqrtf(t) : 0.f;
                if (L.reg_in) reg = (double)sqrtf(t);
            }
            if (flags & 6) {
                unsigned t = 0u;
#pragma unroll
                for (int y = 0; y < 8; ++y) t = max(t, s_pm[y][cx]);
                if (flags & 2) gmax_in[L.c_off + c] = t;
                if (flags & 4) L.zero_in[c] = (__uint_as_float(t) < thr) ? 1 : 0;
            }
        }
    }
    if (!(flags & 1) || !reg_out) return;
    // Eq. 2 without lambda: per-block sum by a fixed tree (shuffles inside a warp, then the eight warps in order), then the
    // last block to finish adds the blocks' sums in order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) reg += __shfl_xor_sync(0xffffffffu, reg, o);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = reg;
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = 0.0;
#pragma unroll
        for (int wv = 0; wv < kThreads / 32; ++wv) tot += s_red[wv];
        job_reg[blockIdx.x] = tot;
        __threadfence();
        s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1u) ? 1u : 0u;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    double t = 0.0;
    for (int i = threadIdx.x; i < (int)gridDim.x; i += kThreads) t += __ldcg(job_reg + i);     // strided slices, ascending
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = 0.0;
#pragma unroll
        for (int wv = 0; wv < kThreads / 32; ++wv) tot += s_red[wv];
        *reg_out = tot;
        *ticket = 0u;
    }
}

// ---- zero masks from the group maxima a carried update left in the workspace
__global__ void masks_kernel(const LayerDev *__restrict__ layers, const unsigned *__restrict__ gmax_out,
                             const unsigned *__restrict__ gmax_in, float thr)
{
    const LayerDev L = layers[blockIdx.x];
    pdl_wait();
    for (int k = threadIdx.x; k < L.K; k += blockDim.x) L.zero_out[k] = (__uint_as_float(gmax_out[L.k_off + k]) < thr) ? 1 : 0;
    for (int c = threadIdx.x; c < L.C; c += blockDim.x) L.zero_in[c] = (__uint_as_float(gmax_in[L.c_off + c]) < thr) ? 1 : 0;
}

// ---- in-place zeroing of the detected groups (weights, momentum, shadow)
__global__ void __launch_bounds__(kThreads) zero_groups_kernel(const LayerDev *__restrict__ layers, const Chunk *__restrict__ chunks)
{
    const Chunk ch = chunks[blockIdx.x];
    const LayerDev L = layers[ch.layer];
    const int TX = 1 << L.tx_log2, TY = kThreads >> L.tx_log2;
    const int tx = threadIdx.x & (TX - 1), ty = threadIdx.x >> L.tx_log2;
    const int c = ch.col0 + tx;
    pdl_wait();
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
    std::vector<Chunk> chunks;             // grouped by layer, layers in the caller's order
    std::vector<int> first_chunk;          // per layer
    std::vector<FinishJob> jobs;
    WsLayout ws;
    int sweeps = kSweeps;                  // base sweeps per chunk of this model; the plain update runs sweeps / 2 blocks per chunk
};

pt_status build_tables(const pt_layer *layers, int n, Tables *t)
{
    if (!layers || n <= 0) return PT_ERR_INVALID_ARG;
    t->layers.resize(n);
    t->first_chunk.assign(n, 0);
    t->chunks.clear();
    t->jobs.clear();
    long long line_off = 0, col_off = 0, k_off = 0, c_off = 0;
    long long params = 0;
    for (int i = 0; i < n; ++i) params += (long long)layers[i].K * layers[i].RS * layers[i].C;
    t->sweeps = params >= kSmallModel ? kSweeps : kSweepsSmall;
    for (int i = 0; i < n; ++i) {
        const pt_layer &s = layers[i];
        if (!s.w || !s.v || s.K <= 0 || s.C <= 0 || s.RS <= 0) return PT_ERR_INVALID_ARG;
        if (s.w_bf16 && (s.ldw < s.C || s.ldw % 8)) return PT_ERR_INVALID_ARG;
        if ((long long)s.K * s.RS * (long long)(s.ldw > s.C ? s.ldw : s.C) >= (1ll << 31)) return PT_ERR_UNSUPPORTED;
        LayerDev &d = t->layers[i];
        memset(&d, 0, sizeof(d));
        d.w = s.w; d.g = s.g; d.v = s.v; d.wb = (__nv_bfloat16 *)s.w_bf16;
        d.sumsq_out = s.sumsq_out; d.sumsq_in = s.sumsq_in; d.zero_out = s.zero_out; d.zero_in = s.zero_in;
        d.K = s.K; d.C = s.C; d.RS = s.RS; d.ldw = s.ldw;
        d.reg_in = s.reg_in; d.reg_out = s.reg_out;
        // column block: the power of two in 32..256 that leaves the fewest lanes idle (ties: the wider one, fewer partials)
        int lg = 5;
        double best = -1.0;
        for (int t2 = 5; t2 <= 8; ++t2) {
            const int tx = 1 << t2;
            const double util = (double)s.C / (double)(tx * pt_ceil_div(s.C, tx));
            if (util >= best - 1e-9) { best = util > best ? util : best; lg = t2; }
        }
        d.tx_log2 = lg;
        const int TX = 1 << lg, TY = kThreads / TX;
        const int lines = s.K * s.RS;
        // a chunk is TY*kUnroll*sweeps lines x TX columns; sweeps = 8 or 4 by the model's size (at most 8: the line staging
        // holds 512 entries), more than the base for tall tensors so that no column has more than ~32 chunk partials to add up
        int sweeps = t->sweeps;
        while (sweeps < 8 && lines > 32 * TY * kUnroll * sweeps) sweeps *= 2;
        const int lines_per_chunk = TY * kUnroll * sweeps;
        d.n_cb = pt_ceil_div(s.C, TX);
        d.n_lc = pt_ceil_div(lines, lines_per_chunk);
        t->first_chunk[i] = (int)t->chunks.size();
        for (int lc = 0; lc < d.n_lc; ++lc)
            for (int cb = 0; cb < d.n_cb; ++cb) {
                Chunk ch;
                ch.layer = i; ch.line0 = lc * lines_per_chunk;
                ch.nlines = lines - ch.line0 < lines_per_chunk ? lines - ch.line0 : lines_per_chunk;
                ch.col0 = cb * TX; ch.lc = lc; ch.cb = cb; ch.pad0 = ch.pad1 = 0;
                t->chunks.push_back(ch);
            }
        for (int k0 = 0; k0 < s.K; k0 += kThreads) t->jobs.push_back(FinishJob{i, 0, k0, 0});
        for (int c0 = 0; c0 < s.C; c0 += 32) t->jobs.push_back(FinishJob{i, 1, c0, 0});
        d.line_off = line_off; line_off += (long long)lines * d.n_cb;
        d.col_off = col_off;   col_off += (long long)d.n_lc * s.C;
        d.k_off = k_off;       k_off += s.K;
        d.c_off = c_off;       c_off += s.C;
    }
    WsLayout &w = t->ws;
    size_t o = 0;
    w.linesum = o;  o = pt_align_up(o + (size_t)line_off * 4, 256);
    w.colpart = o;  o = pt_align_up(o + (size_t)col_off * 4, 256);
    w.linemax = o;  o = pt_align_up(o + (size_t)line_off * 4, 256);
    w.colmax = o;   o = pt_align_up(o + (size_t)col_off * 4, 256);
    w.inv_out = o;  o = pt_align_up(o + (size_t)k_off * 4, 256);
    w.inv_in = o;   o = pt_align_up(o + (size_t)c_off * 4, 256);
    w.gmax_out = o; o = pt_align_up(o + (size_t)k_off * 4, 256);
    w.gmax_in = o;  o = pt_align_up(o + (size_t)c_off * 4, 256);
    w.job_reg = o;  o = pt_align_up(o + t->jobs.size() * 8, 256);
    w.ticket = o;   o += 256;
    w.total = o;
    return PT_OK;
}

// Uploads [LayerDev * n][Chunk * m][FinishJob * j] and returns device pointers.
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

// Launch with programmatic stream serialization: the kernel may start while the previous kernel of the stream drains; every
// kernel of this file executes griddepcontrol.wait before it touches anything a predecessor wrote.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

struct Bound {
    const LayerDev *dl; const Chunk *dc; const FinishJob *dj;
    float *linesum, *colpart, *inv_out, *inv_in;
    unsigned *linemax, *colmax, *gmax_out, *gmax_in, *ticket;
    double *job_reg;
};

Bound bind(const Tables &t, void *ws, const LayerDev *dl, const Chunk *dc, const FinishJob *dj)
{
    char *b = (char *)ws;
    Bound r;
    r.dl = dl; r.dc = dc; r.dj = dj;
    r.linesum = (float *)(b + t.ws.linesum); r.colpart = (float *)(b + t.ws.colpart);
    r.linemax = (unsigned *)(b + t.ws.linemax); r.colmax = (unsigned *)(b + t.ws.colmax);
    r.inv_out = (float *)(b + t.ws.inv_out); r.inv_in = (float *)(b + t.ws.inv_in);
    r.gmax_out = (unsigned *)(b + t.ws.gmax_out); r.gmax_in = (unsigned *)(b + t.ws.gmax_in);
    r.job_reg = (double *)(b + t.ws.job_reg); r.ticket = (unsigned *)(b + t.ws.ticket);
    return r;
}

pt_status launch_finish(pt_ctx *c, const Bound &b, unsigned nj, double *reg_out, int flags, float thr, cudaStream_t st)
{
    PT_CUDA_OK(launch_pdl(finish_kernel, nj, kThreads, st, b.dl, b.dj, (const float *)b.linesum, (const float *)b.colpart,
                          (const unsigned *)b.linemax, (const unsigned *)b.colmax, b.inv_out, b.inv_in, b.gmax_out, b.gmax_in,
                          b.job_reg, b.ticket, reg_out, flags, thr));
    c->launches += 1;
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

// phases: 1 = group norms of the current weights (sweep + finish), 2 = parameter update from the factors in the workspace,
// 4 = the update also leaves the sums of squares of the new weights, and a finish follows it (carried form); 8 = and their
// maxima (for pt_find_zero_groups_carried).
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
    const Bound b = bind(t, ws, dl, dc, dj);
    const unsigned nch = (unsigned)t.chunks.size(), nj = (unsigned)t.jobs.size();
    pt_sgd_hparams none;
    memset(&none, 0, sizeof(none));
    if (phases & 1) {
        PT_CUDA_OK(launch_pdl(sweep_kernel<false, true, false>, nch, kThreads, st, b.dl, b.dc, (const float *)b.inv_out,
                              (const float *)b.inv_in, none, b.linesum, b.colpart, b.linemax, b.colmax, b.ticket, 1));
        c->launches += 1;
        s = launch_finish(c, b, nj, reg_sum_out, 1, 0.f, st);
        if (s != PT_OK) return s;
    }
    if (phases & 2) {
        unsigned c0 = 0, c1 = nch;
        if (count >= 0) {
            c0 = count > 0 ? (unsigned)t.first_chunk[first] : 0;
            c1 = count > 0 ? (first + count < n ? (unsigned)t.first_chunk[first + count] : nch) : 0;
        }
        if (c1 > c0) {
            if ((phases & 4) && (phases & 8))
                PT_CUDA_OK(launch_pdl(sweep_kernel<true, true, true>, c1 - c0, kThreads, st, b.dl, b.dc + c0, (const float *)b.inv_out,
                                      (const float *)b.inv_in, *hp, b.linesum, b.colpart, b.linemax, b.colmax, b.ticket, 1));
            else if (phases & 4)
                PT_CUDA_OK(launch_pdl(sweep_kernel<true, true, false>, c1 - c0, kThreads, st, b.dl, b.dc + c0, (const float *)b.inv_out,
                                      (const float *)b.inv_in, *hp, b.linesum, b.colpart, b.linemax, b.colmax, b.ticket, 1));
            else
                PT_CUDA_OK(launch_pdl(sweep_kernel<true, false, false>, (c1 - c0) * (unsigned)(t.sweeps / 2), kThreads, st, b.dl, b.dc + c0,
                                      (const float *)b.inv_out, (const float *)b.inv_in, *hp, b.linesum, b.colpart, b.linemax, b.colmax,
                                      b.ticket, t.sweeps / 2));
            c->launches += 1;
        }
        if (phases & 4) {
            s = launch_finish(c, b, nj, reg_sum_out, (phases & 8) ? (1 | 2) : 1, 0.f, st);
            if (s != PT_OK) return s;
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

extern "C" pt_status pt_group_lasso_sgd_step_carried(pt_ctx *c, const pt_layer *layers, int32_t n, const pt_sgd_hparams *hp,
                                                     int32_t with_maxima, double *reg_sum_next, void *ws, size_t ws_bytes, void *stream)
{
    return lasso_phases(c, layers, n, hp, reg_sum_next, ws, ws_bytes, stream, 2 | 4 | (with_maxima ? 8 : 0));
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
    const Bound b = bind(t, ws, dl, dc, dj);
    const unsigned nch = (unsigned)t.chunks.size(), nj = (unsigned)t.jobs.size();
    pt_sgd_hparams none;
    memset(&none, 0, sizeof(none));
    PT_CUDA_OK(launch_pdl(sweep_kernel<false, false, true>, nch, kThreads, st, b.dl, b.dc, (const float *)b.inv_out,
                          (const float *)b.inv_in, none, b.linesum, b.colpart, b.linemax, b.colmax, b.ticket, 1));
    c->launches += 1;
    s = launch_finish(c, b, nj, nullptr, 4, threshold, st);
    if (s != PT_OK) return s;
    if (zero_in_place) {
        PT_CUDA_OK(launch_pdl(zero_groups_kernel, nch, kThreads, st, b.dl, b.dc));
        c->launches += 1;
    }
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

extern "C" pt_status pt_find_zero_groups_carried(pt_ctx *c, const pt_layer *layers, int32_t n, float threshold, int32_t zero_in_place,
                                                 void *ws, size_t ws_bytes, void *stream)
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
    s = upload(c, t, false, st, &dl, &dc, &dj);          // the table of the step that left the maxima
    if (s != PT_OK) return s;
    const Bound b = bind(t, ws, dl, dc, dj);
    PT_CUDA_OK(launch_pdl(masks_kernel, (unsigned)n, 256u, st, b.dl, (const unsigned *)b.gmax_out, (const unsigned *)b.gmax_in, threshold));
    c->launches += 1;
    if (zero_in_place) {
        PT_CUDA_OK(launch_pdl(zero_groups_kernel, (unsigned)t.chunks.size(), kThreads, st, b.dl, b.dc));
        c->launches += 1;
    }
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}
