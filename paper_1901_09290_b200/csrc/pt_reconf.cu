// Reconfiguration (Sec. 4.2): keep sets per channel space by the intersection / channel-union
// rule, ascending keep maps by a block-wide scan, and the gather of the surviving weights,
// momentum, bf16 shadow and BN vectors into the smaller dense model.
#include "pt_internal.h"

namespace {

struct SpaceDev {
    int size, fixed;
    int member0, n_members;     // range in the member table
    int map_off;                // start of this space's entries in new2old
    int pad_;
};
struct MemberDev { const uint8_t *mask; };   // a writer's zero_out or a reader's zero_in (length = space size)

// One block per space. keep[j] = fixed | OR_writers !zero_out[j] | OR_readers !zero_in[j].
__global__ void __launch_bounds__(1024) keep_scan_kernel(const SpaceDev *__restrict__ spaces,
                                                         const MemberDev *__restrict__ members,
                                                         int32_t *__restrict__ new2old, int32_t *__restrict__ counts)
{
    __shared__ int s_warp[32];
    __shared__ int s_base, s_tile;
    const SpaceDev sp = spaces[blockIdx.x];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    if (threadIdx.x == 0) s_base = 0;
    __syncthreads();
    for (int j0 = 0; j0 < sp.size; j0 += blockDim.x) {
        const int j = j0 + threadIdx.x;
        int keep = 0;
        if (j < sp.size) {
            keep = sp.fixed;
            for (int m = 0; m < sp.n_members && !keep; ++m) keep |= (members[sp.member0 + m].mask[j] == 0);
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
    if (threadIdx.x == 0) counts[blockIdx.x] = total;
}

struct GatherJob {
    const float *ow, *ov; const __nv_bfloat16 *owb;
    float *nw, *nv; __nv_bfloat16 *nwb;
    const int32_t *mapK, *mapC;
    int Kn, Cn, RS, Co, ldwo, ldwn;
    int kind;                  // 0 = weight tensors, 1 = per-channel vector
    int Ko;                    // old number of output channels (range check of the map)
};
struct GatherChunk { int job, line0, nlines, col0; };

constexpr int kGatherUnroll = 8;

// A map entry outside the old tensor (a new graph larger than the plan's counts reads the -1 padding of the map) is skipped:
// nothing is read or written for it, and the status word reports it (PT_ERR_INVALID_ARG at the next poll).
__device__ __forceinline__ void bad_map_entry(unsigned int *status, unsigned int where)
{
    if (atomicCAS(&status[0], 0u, (unsigned)PT_DEV_BAD_INDEX) == 0u) status[1] = where;
}

__global__ void __launch_bounds__(256) gather_kernel(const GatherJob *__restrict__ jobs, const GatherChunk *__restrict__ chunks,
                                                     unsigned int *status)
{
    const GatherChunk ch = chunks[blockIdx.x];
    const GatherJob J = jobs[ch.job];
    if (J.kind == 1) {       // vector: nw[k'] = ow[mapK[k']]
        for (int k = ch.line0 + threadIdx.x; k < ch.line0 + ch.nlines; k += blockDim.x) {
            const int ko = J.mapK[k];
            if (ko < 0 || ko >= J.Ko) { bad_map_entry(status, 50u); continue; }
            J.nw[k] = J.ow[ko];
        }
        return;
    }
    // Lines of the NEW tensor are (k', rs); a block covers a run of lines x up to 256 columns. Each thread owns one new
    // column c' (its old column looked up once) and keeps four lines in flight; writes are coalesced, reads gathered.
    int TX = 32;
    while (TX < J.Cn && TX < 256) TX <<= 1;
    const int TY = 256 / TX, tx = threadIdx.x % TX, ty = threadIdx.x / TX;
    const int c = ch.col0 + tx;
    if (c >= J.Cn) return;
    const int co = J.mapC[c];
    if (co < 0 || co >= J.Co) { bad_map_entry(status, 51u); return; }
    for (int l = ty; l < ch.nlines; l += kGatherUnroll * TY) {
        float w[kGatherUnroll], v[kGatherUnroll];
        __nv_bfloat16 h[kGatherUnroll];
        bool okk[kGatherUnroll];
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u) {
            const int line = ch.line0 + l + u * TY;
            okk[u] = false;
            if (l + u * TY < ch.nlines) {
                const int kn = line / J.RS, rs = line - kn * J.RS;
                const int ko = J.mapK[kn];
                if (ko < 0 || ko >= J.Ko) { bad_map_entry(status, 52u); continue; }
                okk[u] = true;
                const size_t oline = (size_t)ko * J.RS + rs;
                w[u] = J.ow[oline * J.Co + co];
                if (J.nv) v[u] = J.ov[oline * J.Co + co];
                if (J.nwb) h[u] = J.owb[oline * J.ldwo + co];
            }
        }
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u) {
            const int line = ch.line0 + l + u * TY;
            if (okk[u]) {
                const size_t dst = (size_t)line * J.Cn + c;
                J.nw[dst] = w[u];
                if (J.nv) J.nv[dst] = v[u];
                if (J.nwb) J.nwb[(size_t)line * J.ldwn + c] = h[u];
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
    int32_t *d_counts = (int32_t *)(dev + sb + mb);
    keep_scan_kernel<<<g->n_spaces, 1024, 0, st>>>((const SpaceDev *)dev, (const MemberDev *)(dev + sb), new2old, d_counts);
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    PT_CUDA_OK(cudaMemcpyAsync(c->h_counts, d_counts, (size_t)g->n_spaces * 4, cudaMemcpyDeviceToHost, st));
    PT_CUDA_OK(cudaStreamSynchronize(st));     // the documented synchronisation: the host needs the new sizes
    memcpy(new_sizes, c->h_counts, (size_t)g->n_spaces * 4);
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
    if (c->gather_tab.valid && c->gather_chunks && args == c->gather_args) {
        const char *dev = c->d_arena + c->gather_tab.off;
        gather_kernel<<<c->gather_chunks, 256, 0, st>>>((const GatherJob *)dev, (const GatherChunk *)(dev + c->gather_jobs_bytes), c->d_status);
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
        GatherJob J;
        memset(&J, 0, sizeof(J));
        J.ow = o.w; J.ov = o.v; J.owb = (const __nv_bfloat16 *)o.w_bf16;
        J.nw = n.w; J.nv = n.v; J.nwb = (__nv_bfloat16 *)n.w_bf16;
        J.mapK = new2old + map_off[ol.out_space];
        J.mapC = new2old + map_off[ol.in_space];
        J.Kn = n.K; J.Cn = n.C; J.RS = n.RS; J.Co = o.C; J.Ko = o.K; J.ldwo = o.ldw; J.ldwn = n.ldw;
        J.kind = 0;
        const int job = (int)jobs.size();
        jobs.push_back(J);
        const int lines = n.K * n.RS;
        int TX = 32;
        while (TX < n.C && TX < 256) TX <<= 1;
        const int per = (256 / TX) * kGatherUnroll * 3;      // equal trip counts for every block
        for (int l0 = 0; l0 < lines; l0 += per)
            for (int c0 = 0; c0 < n.C; c0 += TX) chunks.push_back(GatherChunk{job, l0, lines - l0 < per ? lines - l0 : per, c0});
        for (int b = 0; b < 4; ++b) {
            if (!nl.bn[b]) continue;
            if (!ol.bn[b]) return PT_ERR_INVALID_ARG;
            GatherJob V;
            memset(&V, 0, sizeof(V));
            V.ow = ol.bn[b]; V.nw = nl.bn[b]; V.mapK = J.mapK; V.Kn = n.K; V.Ko = o.K; V.kind = 1;
            chunks.push_back(GatherChunk{(int)jobs.size(), 0, n.K, 0});
            jobs.push_back(V);
        }
    }
    if (chunks.empty()) return PT_OK;
    size_t jb = pt_align_up(jobs.size() * sizeof(GatherJob), 256), cb = chunks.size() * sizeof(GatherChunk);
    std::vector<char> buf(jb + cb, 0);
    memcpy(buf.data(), jobs.data(), jobs.size() * sizeof(GatherJob));
    memcpy(buf.data() + jb, chunks.data(), cb);
    char *dev = nullptr;
    c->gather_chunks = 0;
    s = pt_upload_table(c, &c->gather_tab, buf.data(), buf.size(), st, &dev);
    if (s != PT_OK) return s;
    gather_kernel<<<(unsigned)chunks.size(), 256, 0, st>>>((const GatherJob *)dev, (const GatherChunk *)(dev + jb), c->d_status);
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    c->gather_args.swap(args);
    c->gather_chunks = (unsigned)chunks.size();
    c->gather_jobs_bytes = jb;
    return PT_OK;
}
