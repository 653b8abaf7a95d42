// Reconfiguration (Sec. 4.2): keep sets per channel space by the intersection / channel-union
// rule, ascending keep maps by a block-wide scan, and the gather of the surviving weights,
// momentum, bf16 shadow and BN vectors into the smaller dense model.
#include "pt_internal.h"
#include <atomic>
#include <chrono>

namespace {

struct SpaceDev {
    int size, fixed;
    int member0, n_members;     // range in the member table
    int map_off;                // start of this space's entries in new2old
    int pad_;
};
struct MemberDev { const uint8_t *mask; };   // a writer's zero_out or a reader's zero_in (length = space size)

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// One block per space. keep[j] = fixed | OR_writers !zero_out[j] | OR_readers !zero_in[j].
// The counts go straight to pinned host memory; the last block to finish (device ticket) then raises the host flag, so the
// host learns the new sizes from one posted write instead of a copy and a stream synchronisation.
__global__ void __launch_bounds__(1024) keep_scan_kernel(const SpaceDev *__restrict__ spaces,
                                                         const MemberDev *__restrict__ members,
                                                         int32_t *__restrict__ new2old, volatile int32_t *host_counts,
                                                         volatile unsigned int *host_flag, unsigned int seq, unsigned int *ticket)
{
    __shared__ int s_warp[32];
    __shared__ int s_base, s_tile;
    const SpaceDev sp = spaces[blockIdx.x];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    if (threadIdx.x == 0) s_base = 0;
    pdl_wait();                                  // the masks are the previous kernel's output
    __syncthreads();
    for (int j0 = 0; j0 < sp.size; j0 += blockDim.x) {
        const int j = j0 + threadIdx.x;
        int keep = 0;
        if (j < sp.size) {
            keep = sp.fixed;
            // all members' flags are fetched side by side (no early exit: the loads would form a dependent chain)
            int dead = 1;
#pragma unroll 4
            for (int m = 0; m < sp.n_members; ++m) dead &= (members[sp.member0 + m].mask[j] != 0);
            keep |= !dead;
        }
        const unsigned ball = __ballot_sync(0xffffffffu, keep);
        const int in_warp = __popc(ball & ((1u << lane) - 1u));
        if (lane == 0) s_warp[wid] = __popc(ball);
        __syncthreads();
        if (wid == 0) {
            const int v = (lane < nwarps) ? s_warp[lane] : 0;
            int incl = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            s_warp[lane] = incl - v;                 // exclusive prefix of the warp totals
            if (lane == 31) s_tile = incl;           // kept channels in this tile
        }
        __syncthreads();
        const int base = s_base;
        if (keep) new2old[sp.map_off + base + s_warp[wid] + in_warp] = j;   // ascending original index
        __syncthreads();
        if (threadIdx.x == 0) s_base = base + s_tile;
        __syncthreads();
    }
    const int total = s_base;
    for (int j = total + threadIdx.x; j < sp.size; j += blockDim.x) new2old[sp.map_off + j] = -1;
    __syncthreads();
    if (threadIdx.x == 0) {
        host_counts[blockIdx.x] = total;
        __threadfence_system();
        if (atomicAdd(ticket, 1u) == gridDim.x - 1u) {
            *ticket = 0u;
            __threadfence_system();
            *host_flag = seq;
        }
    }
}

// The gather walks the NEW tensor as one flat stream: a chunk is a run of whole lines (about 16K elements), thread t takes
// elements t, t + 256, ... of it, so consecutive lanes read and write consecutive elements whatever the channel count. The
// old line of every new line of the chunk and the old column of every new column sit in shared memory; a thread carries its
// (line, column) along incrementally. Blocks are persistent and take equal shares of the chunk list.
struct GatherJob {
    const float *ow, *ov; const __nv_bfloat16 *owb;
    float *nw, *nv; __nv_bfloat16 *nwb;
    const int32_t *mapK, *mapC;
    int Kn, Cn, RS, Co, ldwo, ldwn;
    int kind;                  // 0 = weight tensors, 1 = per-channel vector
    int Ko;                    // old number of output channels (range check of the map)
    int lines, pad_;           // new tensor: Kn*RS lines
};
struct GatherChunk { int job, line0, n_lines, pad; };

constexpr int kGThreads = 256;
constexpr int kGMaxC = 4096;
constexpr int kGMaxLines = 4096;
constexpr int kGUnroll = 8;

// A map entry outside the old tensor (a new graph larger than the plan's counts reads the -1 padding of the map) is skipped:
// nothing is read or written for it, and the status word reports it (PT_ERR_INVALID_ARG at the next poll).
__device__ __forceinline__ void bad_map_entry(unsigned int *status, unsigned int where)
{
    if (atomicCAS(&status[0], 0u, (unsigned)PT_DEV_BAD_INDEX) == 0u) status[1] = where;
}

__global__ void __launch_bounds__(kGThreads, 4) gather_kernel(const GatherJob *__restrict__ jobs, const GatherChunk *__restrict__ chunks,
                                                            const int *__restrict__ block_first, unsigned int *status)
{
    __shared__ int s_oline[kGMaxLines];          // old line of each new line of the chunk (-1: skipped)
    __shared__ int s_co[kGMaxC];                 // old column of each new column (-1: skipped)
    // block b takes chunks [block_first[b], block_first[b + 1]): consecutive chunks with about the same number of elements
    const int c_beg = block_first[blockIdx.x], c_end = block_first[blockIdx.x + 1];
    int cur_job = -1;
    for (int ci = c_beg; ci < c_end; ++ci) {
        const GatherChunk ch = chunks[ci];
        const GatherJob J = jobs[ch.job];
        if (J.kind == 1) {       // vector: nw[k'] = ow[mapK[k']]
            for (int k = threadIdx.x; k < J.Kn; k += kGThreads) {
                const int ko = J.mapK[k];
                if (ko < 0 || ko >= J.Ko) { bad_map_entry(status, 50u); continue; }
                J.nw[k] = J.ow[ko];
            }
            continue;
        }
        __syncthreads();                         // the previous chunk's tables are no longer read
        if (ch.job != cur_job) {
            cur_job = ch.job;
            for (int c = threadIdx.x; c < J.Cn; c += kGThreads) {
                int o = J.mapC[c];
                if (o < 0 || o >= J.Co) { bad_map_entry(status, 51u); o = -1; }
                s_co[c] = o;
            }
        }
        for (int l = threadIdx.x; l < ch.n_lines; l += kGThreads) {
            const int line = ch.line0 + l;
            const int kn = line / J.RS, rs = line - kn * J.RS;
            const int ko = J.mapK[kn];
            int ol = -1;
            if (ko < 0 || ko >= J.Ko) bad_map_entry(status, 52u);
            else ol = ko * J.RS + rs;
            s_oline[l] = ol;
        }
        __syncthreads();
        // 32-bit element offsets throughout (the host checks that both tensors have fewer than 2^31 elements at their pitches)
        const float *__restrict__ ow = J.ow;
        const float *__restrict__ ov = J.ov;
        const unsigned short *__restrict__ ob = reinterpret_cast<const unsigned short *>(J.owb);
        float *__restrict__ nw = J.nw + (size_t)ch.line0 * J.Cn;
        float *__restrict__ nv = J.nv ? J.nv + (size_t)ch.line0 * J.Cn : nullptr;
        unsigned short *__restrict__ nb = J.nwb ? reinterpret_cast<unsigned short *>(J.nwb) + (size_t)ch.line0 * J.ldwn : nullptr;
        const bool has_v = nv != nullptr, has_b = nb != nullptr;
        const unsigned Co = (unsigned)J.Co, ldwo = (unsigned)J.ldwo, ldwn = (unsigned)J.ldwn;
        const int Cn = J.Cn, total = ch.n_lines * Cn;
        const int dl = kGThreads / Cn, dc = kGThreads - dl * Cn;                 // one step of 256 elements in (line, column)
        int l = (int)threadIdx.x / Cn, c = (int)threadIdx.x - l * Cn;
        for (int i0 = threadIdx.x; i0 < total; i0 += kGUnroll * kGThreads) {
            float w[kGUnroll], v[kGUnroll];
            unsigned short hb[kGUnroll];
            int ll[kGUnroll], cc[kGUnroll];
            bool ok[kGUnroll];
#pragma unroll
            for (int u = 0; u < kGUnroll; ++u) {
                ll[u] = l; cc[u] = c;
                ok[u] = false;
                if (i0 + u * kGThreads < total) {
                    const int ol = s_oline[l], co = s_co[c];
                    if ((ol | co) >= 0) {
                        ok[u] = true;
                        const unsigned src = (unsigned)ol * Co + (unsigned)co;
                        w[u] = ow[src];
                        if (has_v) v[u] = ov[src];
                        if (has_b) hb[u] = ob[(unsigned)ol * ldwo + (unsigned)co];
                    }
                }
                l += dl; c += dc;
                if (c >= Cn) { c -= Cn; ++l; }
            }
#pragma unroll
            for (int u = 0; u < kGUnroll; ++u) {
                if (!ok[u]) continue;
                const unsigned idx = (unsigned)(i0 + u * kGThreads);
                nw[idx] = w[u];
                if (has_v) nv[idx] = v[u];
                if (has_b) nb[(unsigned)ll[u] * ldwn + (unsigned)cc[u]] = hb[u];
            }
        }
    }
}

pt_status check_graph(const pt_graph *g)
{
    if (!g || !g->spaces || !g->layers || !g->links || g->n_spaces <= 0 || g->n_layers <= 0) return PT_ERR_INVALID_ARG;
    for (int i = 0; i < g->n_layers; ++i) {
        const pt_layer_link &k = g->links[i];
        if (k.in_space < 0 || k.in_space >= g->n_spaces || k.out_space < 0 || k.out_space >= g->n_spaces) return PT_ERR_INVALID_ARG;
        if (g->layers[i].C != g->spaces[k.in_space].size || g->layers[i].K != g->spaces[k.out_space].size) return PT_ERR_INVALID_ARG;
    }
    return PT_OK;
}

}  // namespace

extern "C" pt_status pt_reconfigure_plan(pt_ctx *c, const pt_graph *g, int32_t *new2old, int32_t *new_sizes, void *stream)
{
    if (!c || !new2old || !new_sizes) return PT_ERR_INVALID_ARG;
    pt_status s = check_graph(g);
    if (s != PT_OK) return s;
    if (g->n_spaces > 65536) return PT_ERR_UNSUPPORTED;
    std::vector<SpaceDev> sp(g->n_spaces);
    std::vector<MemberDev> mem;
    long long off = 0;
    for (int i = 0; i < g->n_spaces; ++i) {
        if (g->spaces[i].size < 0) return PT_ERR_INVALID_ARG;
        sp[i].size = g->spaces[i].size;
        sp[i].fixed = g->spaces[i].fixed ? 1 : 0;
        sp[i].member0 = (int)mem.size();
        for (int l = 0; l < g->n_layers; ++l) {
            if (g->links[l].out_space == i) {
                if (!g->layers[l].zero_out) return PT_ERR_INVALID_ARG;
                mem.push_back(MemberDev{g->layers[l].zero_out});
            }
            if (g->links[l].in_space == i) {
                if (!g->layers[l].zero_in) return PT_ERR_INVALID_ARG;
                mem.push_back(MemberDev{g->layers[l].zero_in});
            }
        }
        sp[i].n_members = (int)mem.size() - sp[i].member0;
        sp[i].map_off = (int)off;
        sp[i].pad_ = 0;
        off += sp[i].size;
        if (off >= (1ll << 31)) return PT_ERR_UNSUPPORTED;
    }
    size_t sb = pt_align_up(sp.size() * sizeof(SpaceDev), 256), mb = pt_align_up(mem.size() * sizeof(MemberDev) + 8, 256);
    std::vector<char> buf(sb + mb + (size_t)g->n_spaces * 4, 0);
    memcpy(buf.data(), sp.data(), sp.size() * sizeof(SpaceDev));
    if (!mem.empty()) memcpy(buf.data() + sb, mem.data(), mem.size() * sizeof(MemberDev));
    cudaStream_t st = (cudaStream_t)stream;
    char *dev = nullptr;
    s = pt_upload_table(c, &c->graph_tab, buf.data(), buf.size(), st, &dev);
    if (s != PT_OK) return s;
    // counts and flag live in pinned host memory the kernel writes directly: [0] = flag (sequence number), [16..] = counts
    volatile unsigned int *flag = (volatile unsigned int *)c->h_counts;
    volatile int32_t *counts = (volatile int32_t *)c->h_counts + 16;
    const unsigned int seq = ++c->plan_seq;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)g->n_spaces); cfg.blockDim = dim3(1024); cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    PT_CUDA_OK(cudaLaunchKernelEx(&cfg, keep_scan_kernel, (const SpaceDev *)dev, (const MemberDev *)(dev + sb), new2old,
                                  (volatile int32_t *)counts, (volatile unsigned int *)flag, seq, c->d_status + 2));
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    // The documented synchronisation: the host needs the new sizes. It waits for the kernel's flag (bounded), looking at the
    // stream now and then so that an error upstream ends the wait.
    {
        const auto t0 = std::chrono::steady_clock::now();
        unsigned spins = 0;
        bool seen = false;
        while (!(seen = (*flag == seq))) {
            if ((++spins & 0x3fffu) == 0u) {
                const cudaError_t q = cudaStreamQuery(st);
                if (q == cudaSuccess) { seen = (*flag == seq); break; }
                if (q != cudaErrorNotReady) { (void)cudaGetLastError(); return PT_ERR_CUDA; }
                if (std::chrono::steady_clock::now() - t0 > std::chrono::seconds(30)) break;
            }
        }
        if (!seen) {
            PT_CUDA_OK(cudaStreamSynchronize(st));
            if (*flag != seq) return PT_ERR_CUDA;
        }
    }
    std::atomic_thread_fence(std::memory_order_acquire);
    for (int i = 0; i < g->n_spaces; ++i) new_sizes[i] = counts[i];
    return PT_OK;
}

extern "C" pt_status pt_reconfigure(pt_ctx *c, const pt_graph *og, const int32_t *new2old, const pt_graph *ng, void *stream)
{
    if (!c || !new2old || !og || !ng) return PT_ERR_INVALID_ARG;
    if (!og->spaces || !og->layers || !og->links || !ng->spaces || !ng->layers || !ng->links) return PT_ERR_INVALID_ARG;
    if (og->n_spaces <= 0 || og->n_layers <= 0 || og->n_spaces != ng->n_spaces || og->n_layers != ng->n_layers) return PT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    // The table below depends on the arguments only (shapes, pointers, the map's address), not on what the buffers hold:
    // this call sits right behind the host synchronisation of the plan, so a repeated reconfiguration skips the rebuild.
    std::vector<char> args;
    {
        const size_t ns = (size_t)og->n_spaces * sizeof(pt_space), nl = (size_t)og->n_layers * sizeof(pt_layer);
        const size_t nk = (size_t)og->n_layers * sizeof(pt_layer_link);
        args.resize(2 * (ns + nl + nk) + sizeof(new2old));
        char *a = args.data();
        memcpy(a, og->spaces, ns); a += ns; memcpy(a, ng->spaces, ns); a += ns;
        memcpy(a, og->layers, nl); a += nl; memcpy(a, ng->layers, nl); a += nl;
        memcpy(a, og->links, nk); a += nk; memcpy(a, ng->links, nk); a += nk;
        memcpy(a, &new2old, sizeof(new2old));
    }
    for (int i = 0; i < 4; ++i) {
        pt_ctx::GatherSlot &gs = c->gather_slot[i];
        if (!(gs.reg.valid && gs.chunks && args == gs.args)) continue;
        const char *dev = c->d_arena + gs.reg.off;
        gather_kernel<<<gs.grid, kGThreads, 0, st>>>((const GatherJob *)dev, (const GatherChunk *)(dev + gs.jobs_bytes),
                                                     (const int *)(dev + gs.first_off), c->d_status);
        c->launches += 1;
        PT_CUDA_OK(cudaGetLastError());
        return PT_OK;
    }
    pt_status s = check_graph(og);
    if (s != PT_OK) return s;
    s = check_graph(ng);
    if (s != PT_OK) return s;
    std::vector<int> map_off(og->n_spaces);
    long long off = 0;
    for (int i = 0; i < og->n_spaces; ++i) {
        map_off[i] = (int)off;
        off += og->spaces[i].size;
        if (ng->spaces[i].size > og->spaces[i].size) return PT_ERR_INVALID_ARG;
    }
    std::vector<GatherJob> jobs;
    std::vector<GatherChunk> chunks;
    for (int l = 0; l < og->n_layers; ++l) {
        const pt_layer &o = og->layers[l], &n = ng->layers[l];
        const pt_layer_link &ol = og->links[l], &nl = ng->links[l];
        if (ol.in_space != nl.in_space || ol.out_space != nl.out_space || o.RS != n.RS) return PT_ERR_INVALID_ARG;
        if (n.K == 0 || n.C == 0) continue;                 // a dead layer: nothing to carry over
        if (!o.w || !n.w || (n.v && !o.v) || (n.w_bf16 && !o.w_bf16)) return PT_ERR_INVALID_ARG;
        if (n.w_bf16 && (n.ldw < n.C || n.ldw % 8)) return PT_ERR_INVALID_ARG;
        if (n.C > kGMaxC) return PT_ERR_UNSUPPORTED;
        if ((long long)o.K * o.RS * (o.ldw > o.C ? o.ldw : o.C) >= (1ll << 31)) return PT_ERR_UNSUPPORTED;
        GatherJob J;
        memset(&J, 0, sizeof(J));
        J.ow = o.w; J.ov = o.v; J.owb = (const __nv_bfloat16 *)o.w_bf16;
        J.nw = n.w; J.nv = n.v; J.nwb = (__nv_bfloat16 *)n.w_bf16;
        J.mapK = new2old + map_off[ol.out_space];
        J.mapC = new2old + map_off[ol.in_space];
        J.Kn = n.K; J.Cn = n.C; J.RS = n.RS; J.Co = o.C; J.Ko = o.K; J.ldwo = o.ldw; J.ldwn = n.ldw;
        J.kind = 0;
        J.lines = n.K * n.RS;
        const int job = (int)jobs.size();
        jobs.push_back(J);
        {
            int per = 8192 / n.C;                        // whole lines, about 8K elements per chunk
            if (per < 1) per = 1;
            if (per > kGMaxLines) per = kGMaxLines;
            for (int l0 = 0; l0 < J.lines; l0 += per) chunks.push_back(GatherChunk{job, l0, J.lines - l0 < per ? J.lines - l0 : per, 0});
        }
        for (int b = 0; b < 4; ++b) {
            if (!nl.bn[b]) continue;
            if (!ol.bn[b]) return PT_ERR_INVALID_ARG;
            GatherJob V;
            memset(&V, 0, sizeof(V));
            V.ow = ol.bn[b]; V.nw = nl.bn[b]; V.mapK = J.mapK; V.Kn = n.K; V.Ko = o.K; V.kind = 1;
            chunks.push_back(GatherChunk{(int)jobs.size(), 0, 0, 0});
            jobs.push_back(V);
        }
    }
    if (chunks.empty()) return PT_OK;
    // Blocks are persistent (at most four per SM) and take consecutive chunks; the list is cut where the running element
    // count passes the next multiple of total / grid, so that every block moves about the same number of elements (a
    // per-channel vector counts as one block-wide step).
    const unsigned nchk = (unsigned)chunks.size();
    const unsigned grid = nchk < (unsigned)(4 * c->sm_count) ? nchk : (unsigned)(4 * c->sm_count);
    std::vector<int> first(grid + 1, 0);
    {
        std::vector<long long> cost(nchk);
        long long total = 0;
        for (unsigned i = 0; i < nchk; ++i) {
            const GatherJob &J = jobs[chunks[i].job];
            cost[i] = J.kind == 1 ? kGThreads : (long long)chunks[i].n_lines * J.Cn;
            total += cost[i];
        }
        long long run = 0;
        unsigned b = 1;
        for (unsigned i = 0; i < nchk && b < grid; ++i) {
            run += cost[i];
            // chunk i ends block b - 1 once the running count reaches that block's share (and enough chunks remain for the rest)
            while (b < grid && (run * grid >= total * b || nchk - (i + 1) <= grid - b)) first[b++] = (int)(i + 1);
        }
        while (b <= grid) first[b++] = (int)nchk;
        first[grid] = (int)nchk;
    }
    size_t jb = pt_align_up(jobs.size() * sizeof(GatherJob), 256), cb = pt_align_up(chunks.size() * sizeof(GatherChunk), 256);
    const size_t fb = first.size() * sizeof(int);
    std::vector<char> buf(jb + cb + fb, 0);
    memcpy(buf.data(), jobs.data(), jobs.size() * sizeof(GatherJob));
    memcpy(buf.data() + jb, chunks.data(), chunks.size() * sizeof(GatherChunk));
    memcpy(buf.data() + jb + cb, first.data(), fb);
    char *dev = nullptr;
    pt_ctx::GatherSlot &gs = c->gather_slot[c->gather_next];
    c->gather_next = (c->gather_next + 1) & 3;
    gs.chunks = 0;
    s = pt_upload_table(c, &gs.reg, buf.data(), buf.size(), st, &dev);
    if (s != PT_OK) return s;
    gather_kernel<<<grid, kGThreads, 0, st>>>((const GatherJob *)dev, (const GatherChunk *)(dev + jb), (const int *)(dev + jb + cb),
                                              c->d_status);
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    gs.args.swap(args);
    gs.chunks = nchk;
    gs.jobs_bytes = jb;
    gs.first_off = jb + cb;
    gs.grid = grid;
    return PT_OK;
}
