// tcgen05 / TMEM / TMA implicit-GEMM convolutions for sm_100a.
//
//   conv_gemm_kernel   fwd and dgrad of 1x1 / strided layers: persistent CTAs, im2col-mode (or plain 2-D) TMA loads of
//                      128 pixels x 64 channels, K-major (fwd) or MN-major (dgrad) weight tiles from the same bf16 shadow,
//                      double/triple-buffered fp32 accumulators in TMEM, TMA-store epilogue.
//   conv_halo_kernel   stride-1 RxS fwd/dgrad and the parities of a stride-2 dgrad: one halo tile per 64-channel chunk,
//                      filter taps as row-shifted UMMA descriptors of that tile; a 32-byte-pixel mode (16 lanes per
//                      position, 32-byte swizzle, one MMA per tap) runs the space-to-depth stem.
//   conv_wgrad_kernel  weight gradient: both operands MN-major, reduction over pixels split across CTAs, partial tiles
//                      summed in-kernel in a fixed order.
//   conv_wgrad_rows_kernel  weight gradient of stride-1 layers with at most 64 input channels: row blocks of x staged
//                      once, taps as row-shifted descriptors, two taps per MMA on the M side; same finish phase.
//   stem_* kernels     space-to-depth layout kernels of the few-channel stride-2 stem.
// Ragged channel counts are handled by the TMA unit (true extents in the tensor maps: zero-fill on load, clipping on
// store) and by skipping the 16-wide k-steps past the last valid channel.
// Issue is spread over warps in all three kernels: one thread spends ~200 cycles per TMA instruction and 50-100 per
// tcgen05.mma, more than a narrow MMA takes to run, so operands are loaded by several producer warps and, where
// independent accumulators exist, MMAs are issued by up to four warps, each with its own ring and TMEM buffers.
// The kernels are launched with programmatic stream serialization (griddepcontrol.wait after the prologue).
// Every wait is bounded; on expiry the CTA records PT_DEV_TIMEOUT in the status word, drains its copies and exits.
#include "pt_internal.h"
#include "pt_sm100_ptx.cuh"
#include <cudaTypedefs.h>

using namespace sm100;

namespace {
// Launch with programmatic stream serialization: the kernel may be scheduled while the previous kernel of the stream is
// still draining, so its prologue (barrier setup, TMEM allocation, descriptor prefetch) and the launch latency overlap that
// kernel's tail. Every kernel launched this way executes griddepcontrol.wait before its first global-memory access.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// A tensor-map encode that the driver refused is kept, with its line, for pt_last_cuda_error.
bool map_ok(CUresult r, int line)
{
    if (r != CUDA_SUCCESS) pt_note_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncode* (refused by the driver)", __FILE__, line);
    return r == CUDA_SUCCESS;
}


constexpr int kBM = 128;            // output pixels per CTA tile
constexpr int kKC = 64;             // reduction channels per stage (one 128-byte swizzle row)
constexpr int kMaxStages = 8;
constexpr int kThreads = 288;           // wgrad kernel: dy producer, MMA issuer, 4 epilogue warps (x producers in the main loop), 3 more MMA issuers
constexpr int kGemmThreads = 512;       // fwd/dgrad kernel: A producer, MMA issuer, up to 12 epilogue warps, B producer, second MMA issuer
constexpr int kMaxTaps = 64;

struct GemmP {
    int M_total;        // output pixels of this launch's raster
    int n_cols;         // true number of output channels
    int BN;             // tile width (multiple of 16)
    int n_tiles;        // tiles along the channel dimension
    int c_red;          // true number of reduction channels
    int k_chunks;       // ceil(c_red / 64)
    int taps;           // filter taps visited by this launch (<= kMaxTaps)
    int Pd, Qd;         // raster of output pixels (rows, columns) per image
    int stride;         // traversal stride of the raster in the source tensor
    int lo_h, lo_w;     // source coordinate of raster position (0,0) for tap (0,0)
    int stages;
    int tmem_cols;
    // output pixel mapping: pixel (n, i, j) of the raster -> out[((n*oH + i*o_step + o_h0)*oW + j*o_step + o_w0)*ld_out]
    int oH, oW, o_step, o_h0, o_w0;
    int ld_out, out_f32;
    int zero_mask;      // stride-2 dgrad: bit (a*2+b) set => also write zeros to the pixel at parity (a,b) of each 2x2 cell
    int tma_store;      // 1: bf16 output rows are consecutive pixels -> staged in shared memory and written by TMA stores
    int m_tiles;        // ceil(M_total / 128)
    int epi_groups;     // 1..3 groups of four epilogue warps
    int a_tiled;        // 1: 1x1 stride-1 problem, the A operand is a plain 2-D (channels, pixels) tiled map
    int resident;       // 1: every weight tile of the launch stays in shared memory (loaded once); the ring carries A only
    int n_issuers;      // 2 (resident weights only): two MMA issuer warps take alternate tiles, each with half of the ring's stages
    int acc_per;        // two issuers: accumulator buffers per issuer (1 or 2)
    int alias_staging;  // 1: the CTA has a single tile; the epilogue's staging slabs lie in the (then idle) ring
    int test_skip;      // test hook (pt_test_skip_next_arrive): the A producer leaves out the first stage of its first tile
    int stats_off;      // byte offset in shared memory of the epilogue warps' statistics accumulators (stats != nullptr)
    int stats_warp;     // bytes of one warp's accumulators: 512 per 64-channel chunk of the tile
    float *stats;       // optional: per (pixel tile, warp quarter) and output channel, sum and sum of squares of the bf16 values
                        // stored, as [part][2][ld_out] floats (the batch-normalisation statistics of the layer that follows)
    void *out;
    unsigned int *status;
    unsigned char tap_oh[kMaxTaps], tap_ow[kMaxTaps];   // im2col offsets of each visited tap
    unsigned short tap_wt[kMaxTaps];                    // index r*S+s of the weights the tap multiplies
};

struct __align__(8) Ctl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t accum;
    uint32_t tmem_base;
    int abort_flag;
};

// Control block of the persistent fwd/dgrad kernel.
struct __align__(8) PCtl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t acc_full[4];       // MMA issuer -> epilogue: accumulator buffer b holds a finished tile
    uint64_t acc_empty[4];      // epilogue -> MMA issuer: buffer b has been read out (4 arrivals, one per warp of its group)
    uint64_t w_full;            // resident weights have landed
    uint32_t tmem_base;
    int abort_flag;
#ifdef PT_DEVICE_TRACE
    unsigned int chain_seq;
#endif
};

constexpr uint32_t kSlabs = 2;                          // staging slabs per epilogue warp (TMA stores in flight)

// Batch-normalisation statistics of a staged output chunk: `rows` is a bit mask of the warp's 32 staged rows (128 bytes each,
// 128-byte swizzle, first row `row0` of the slab) that are real output pixels. Lane l owns channels 2l and 2l + 1 of the
// 64-channel chunk and adds the bf16 values exactly as they were stored, rows in ascending order: sum and sum of squares,
// accumulated in the warp's own shared-memory slots (acc: 128 floats per chunk of the tile, four per lane) and written to the
// warp's row of partial sums by stats_flush. Feature normalisation (Sec. 2.1) reads its input twice; taking the sums here,
// from the tile that is still in shared memory, removes the first of the two passes.
constexpr uint32_t kStatsChunkBytes = 128u * 4u;              // per 64-channel chunk: 32 lanes x (sum, sum of squares) x two channels

__device__ __forceinline__ void chunk_stats(uint32_t slab, int row0, uint32_t rows, int lane, uint32_t acc)
{
    float s0a = 0.f, s1a = 0.f, s0b = 0.f, s1b = 0.f;
    const uint32_t jj = (uint32_t)lane >> 2, wi = ((uint32_t)lane & 3u) << 2;
    // Eight loads are issued before the first is used (one at a time, each waits out the shared-memory latency: 1500 cycles
    // per chunk in the first version, more than the rest of the epilogue). Rows that are not output pixels (the halo tiles'
    // raster has some) are loaded too and count as zeros.
#pragma unroll
    for (int r0 = 0; r0 < 32; r0 += 8) {
        uint32_t word[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t m = (uint32_t)(row0 + r0 + j);
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(word[j]) : "r"(slab + m * 128u + ((jj ^ (m & 7u)) << 4) + wi));
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const bool on = (rows >> (r0 + j)) & 1u;
            const float a = on ? __uint_as_float(word[j] << 16) : 0.f, b = on ? __uint_as_float(word[j] & 0xffff0000u) : 0.f;
            s0a += a; s1a = fmaf(a, a, s1a);
            s0b += b; s1b = fmaf(b, b, s1b);
        }
    }
    float4 t;
    const uint32_t slot = acc + (uint32_t)lane * 16u;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(t.x), "=f"(t.y), "=f"(t.z), "=f"(t.w) : "r"(slot) : "memory");
    t.x += s0a; t.y += s1a; t.z += s0b; t.w += s1b;
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(slot), "f"(t.x), "f"(t.y), "f"(t.z), "f"(t.w) : "memory");
}

__device__ __forceinline__ void stats_clear(uint32_t acc0, int lane, int n_chunks)
{
#pragma unroll
    for (int ch = 0; ch < 4; ++ch)
        if (ch < n_chunks)
            asm volatile("st.shared.v4.f32 [%0], {%1, %1, %1, %1};" ::"r"(acc0 + (uint32_t)ch * 512u + (uint32_t)lane * 16u), "f"(0.f) : "memory");
}

// Adds the warp's shared-memory sums of the channels n0 .. n0 + 64 * n_chunks into its row of partial sums (zeroed by the warp
// at kernel start; a column is always this lane's: read, add, write) and clears them.
__device__ __forceinline__ void stats_flush(uint32_t acc0, int lane, float *dst, int ld, int n0, int n_chunks, int n_cols, bool add)
{
    float4 t[4];
    float o[4][4];
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
        if (ch >= n_chunks) break;
        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(t[ch].x), "=f"(t[ch].y), "=f"(t[ch].z), "=f"(t[ch].w)
                     : "r"(acc0 + (uint32_t)ch * 512u + (uint32_t)lane * 16u) : "memory");
        const int c = n0 + ch * 64 + 2 * lane;
        // (a warp that visits its columns once, at the very end, has nothing to add to: the row still holds its zeros)
        o[ch][0] = (add && c < n_cols) ? dst[c] : 0.f;
        o[ch][1] = (add && c < n_cols) ? dst[ld + c] : 0.f;
        o[ch][2] = (add && c + 1 < n_cols) ? dst[c + 1] : 0.f;
        o[ch][3] = (add && c + 1 < n_cols) ? dst[ld + c + 1] : 0.f;
    }
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
        if (ch >= n_chunks) break;
        const int c = n0 + ch * 64 + 2 * lane;
        if (c < n_cols) { dst[c] = o[ch][0] + t[ch].x; dst[ld + c] = o[ch][1] + t[ch].y; }
        if (c + 1 < n_cols) { dst[c + 1] = o[ch][2] + t[ch].z; dst[ld + c + 1] = o[ch][3] + t[ch].w; }
    }
    stats_clear(acc0, lane, n_chunks);
}

// Device-side timeline of CTA 0 (a build with -DPT_DEVICE_TRACE; read back with pt_debug_gemm_trace): per pipeline stage in
// issue order, when the A producer found it free / issued it, when the MMA issuer found it full / committed it; per tile, when
// the epilogue got the accumulator and when it had issued its stores.
#ifdef PT_DEVICE_TRACE
__device__ unsigned long long g_gemm_trace[8][64];
#define GTRACE(role, idx) do { if (blockIdx.x == 0 && (idx) < 64 && (threadIdx.x & 31) == 0) g_gemm_trace[role][idx] = globaltimer_ns(); } while (0)
// Timeline of a chain of launches: launch number seq (a device counter, taken by CTA 0 at entry) stamps its entry, the end of
// its prologue, the return of its dependency wait, its first activation load, its first full stage, its last commit, the end
// of its last epilogue and its exit.
__device__ unsigned long long g_chain_trace[256][12];
__device__ unsigned int g_chain_seq;
#define CTRACE(ev) do { if (blockIdx.x == 0 && (threadIdx.x & 31) == 0 && ctl->chain_seq < 256) g_chain_trace[ctl->chain_seq][ev] = globaltimer_ns(); } while (0)
#else
#define GTRACE(role, idx) do { } while (0)
#define CTRACE(ev) do { } while (0)
#endif

// Persistent: each CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ... The TMA ring runs continuously across
// tiles. The accumulator has G = 2 or 3 buffers in TMEM and buffer b has its own group of four epilogue warps, so the
// loads and MMAs of the next tiles overlap the epilogues of the previous ones.
// STATS: the epilogue also takes the batch-normalisation statistics (a variant of its own: the plain kernels keep their registers).
template <bool B_MN, bool STATS>
__global__ void __launch_bounds__(kGemmThreads, 1) conv_gemm_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                 const __grid_constant__ CUtensorMap tmB,
                                                                 const __grid_constant__ CUtensorMap tmC, const GemmP p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    PCtl *ctl = reinterpret_cast<PCtl *>(smem_raw);
    const uint32_t smem_base = smem_u32(smem_raw);
    const uint32_t staging_base = (smem_base + (uint32_t)sizeof(PCtl) + 1023u) & ~1023u;
    const uint32_t a_bytes = kBM * kKC * 2;
    const uint32_t b_bytes = B_MN ? (uint32_t)((p.BN + 63) / 64) * 8192u : (uint32_t)p.BN * 128u;
    const uint32_t b_slot = (b_bytes + 1023u) & ~1023u;
    // resident weights: all taps x chunks sit in front of the ring, whose stages then hold an A tile only
    // a CTA with a single tile stages its output in the ring, which is idle by then: no separate staging area
    const uint32_t w_base = staging_base + (p.alias_staging ? 0u : (uint32_t)p.epi_groups * 4u * kSlabs * 4096u);
    const uint32_t stage_bytes = p.resident ? a_bytes : a_bytes + b_slot;
    const uint32_t data_base = w_base + (p.resident ? (uint32_t)(p.taps * p.k_chunks) * b_slot : 0u);
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int iters = p.taps * p.k_chunks;
    const int total_tiles = p.m_tiles * p.n_tiles;
    // streamed MN-major weight tiles are one 8 KB box per 64 columns: with several boxes per stage a second producer warp
    // (warp 15, otherwise idle without resident weights) issues every other one
    const int nb_b = (p.BN + 63) / 64;
    const bool two_b = B_MN && !p.resident && nb_b > 1;

#ifdef PT_DEVICE_TRACE
    if (threadIdx.x == 0) {
        ctl->chain_seq = blockIdx.x == 0 ? atomicAdd(&g_chain_seq, 1u) : 0xffffffffu;
        CTRACE(0);
    }
#endif
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), p.resident ? 1 : (two_b ? 3 : 2));   // the A producer and, with streamed weights, the B producer(s)
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        mbar_init(smem_u32(&ctl->w_full), 1);
        for (int b = 0; b < 4; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), 1);
            mbar_init(smem_u32(&ctl->acc_empty[b]), 4);
        }
        ctl->abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        if (p.tma_store) prefetch_tmap(&tmC);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    // The weights are not written by the kernels that precede a convolution in a stream (those that trigger their dependents
    // early are convolutions themselves), so the weight producers start loading at once; everybody else waits for the
    // previous kernel's results here.
    // The activation producer (warp 0) waits just before its first load instead: its set-up (tile coordinates, tap tables: a
    // few hundred cycles of divisions and first-touch parameter reads) then runs while the previous kernel drains.
    if (!(warp == 0 || warp == 14 || (warp == 15 && two_b))) grid_dependency_wait();
    grid_launch_dependents();

    if (warp == 0 || warp == 14 || (warp == 15 && two_b)) {
        if (lane == 0) {
            // ---------------- TMA producers: warp 0 brings the A tile of every stage, warp 14 the B tile (issuing a TMA
            // instruction costs its thread about 200 cycles, so the two operands are issued side by side)
            const bool is_a = warp == 0;
            if (is_a) CTRACE(8);
            const int bsel = warp == 15 ? 1 : 0, nbp = two_b ? 2 : 1;         // this B producer's boxes: bsel, bsel + nbp, ...
            const uint32_t my_bytes = is_a ? a_bytes : (two_b ? (uint32_t)((nb_b + 1 - bsel) / 2) * 8192u : b_bytes);
            int s = 0, ph = 0, issued = 0;   // stage-ring position, continuous across tiles
            int s1 = 0, ph1 = 0;             // position in the second issuer's ring
            bool dep_waited = false;         // the activation producer has waited for the previous kernel's results
            const int SR = p.stages / p.n_issuers;
            if (!is_a && p.resident) {
                // n_tiles == 1 here: every weight tile of the launch, once
                const uint32_t bar = smem_u32(&ctl->w_full);
                mbar_arrive_expect_tx(bar, (uint32_t)iters * b_bytes);
                for (int tap = 0; tap < p.taps; ++tap)
                    for (int kc = 0; kc < p.k_chunks; ++kc) {
                        const uint32_t dst = w_base + (uint32_t)(tap * p.k_chunks + kc) * b_slot;
                        const int wtap = p.tap_wt[tap];
                        if (!B_MN) tma_load_3d(dst, &tmB, bar, kc * kKC, wtap, 0);
                        else for (int nb = 0; nb < (p.BN + 63) / 64; ++nb) tma_load_3d(dst + (uint32_t)nb * 8192u, &tmB, bar, nb * 64, wtap, kc * kKC);
                    }
            }
            int ring = 0;
            for (int tile = blockIdx.x; tile < total_tiles && !*abort_flag && (is_a || !p.resident); tile += gridDim.x,
                     ring = p.n_issuers == 2 ? ring ^ 1 : 0) {
                const int n_tile = tile % p.n_tiles, m_tile = tile / p.n_tiles;
                const int m0 = m_tile * kBM, n0 = n_tile * p.BN;
                if (ring) { int t = s; s = s1; s1 = t; t = ph; ph = ph1; ph1 = t; }     // work on the second ring's position
                const int sbase = ring * SR;
                int w0 = 0, h0 = 0, n = 0;
                if (is_a && !p.a_tiled) {
                    const int q = m0 % p.Qd, t = m0 / p.Qd, pp = t % p.Pd;
                    n = t / p.Pd;
                    w0 = q * p.stride + p.lo_w; h0 = pp * p.stride + p.lo_h;
                }
                bool ok = true;
                for (int tap = 0; tap < p.taps && ok; ++tap) {
                    const int wtap = p.tap_wt[tap];
                    const uint16_t ow = (uint16_t)p.tap_ow[tap], oh = (uint16_t)p.tap_oh[tap];
                    for (int kc = 0; kc < p.k_chunks; ++kc) {
                        if (is_a && issued == 0) CTRACE(9);
                        ok = mbar_wait(smem_u32(&ctl->empty[sbase + s]), ph ^ 1, abort_flag, p.status, 1);
                        if (!ok) break;
                        if (is_a && issued == 0) CTRACE(10);
                        if (is_a) GTRACE(0, issued); else if (warp == 14) GTRACE(2, issued);
                        const uint32_t bar = smem_u32(&ctl->full[sbase + s]);
                        const uint32_t a_dst = data_base + (uint32_t)(sbase + s) * stage_bytes, b_dst = a_dst + a_bytes;
                        if (is_a && p.test_skip && issued == 0) {         // test hook: this stage never becomes full
                            ++issued;
                            if (++s == SR) { s = 0; ph ^= 1; }
                            continue;
                        }
                        mbar_arrive_expect_tx(bar, my_bytes);
                        if (is_a && !dep_waited) { CTRACE(1); grid_dependency_wait(); CTRACE(2); dep_waited = true; }
                        if (is_a) {
                            if (p.a_tiled) tma_load_2d(a_dst, &tmA, bar, kc * kKC, m0);
                            else tma_load_im2col_4d(a_dst, &tmA, bar, kc * kKC, w0, h0, n, ow, oh);
                        } else if (!B_MN) {
                            tma_load_3d(b_dst, &tmB, bar, kc * kKC, wtap, n0);
                        } else {
                            for (int nb = bsel; nb < nb_b; nb += nbp)
                                tma_load_3d(b_dst + (uint32_t)nb * 8192u, &tmB, bar, n0 + nb * 64, wtap, kc * kKC);
                        }
                        if (is_a) GTRACE(1, issued); else if (warp == 14) GTRACE(3, issued);
                        if (is_a && issued == 0) CTRACE(3);
                        ++issued;
                        if (++s == SR) { s = 0; ph ^= 1; }
                    }
                }
                if (ring) { int t = s; s = s1; s1 = t; t = ph; ph = ph1; ph1 = t; }
                if (!ok) break;
            }
            if (*abort_flag && is_a) {
                // drain: give the copies already issued a bounded time to land before the CTA's smem is released
                const uint64_t t0 = globaltimer_ns();
                for (int s2 = 0; s2 < p.stages && issued > 0; ++s2)
                    while (!mbar_try_wait(smem_u32(&ctl->full[s2]), 0) && !mbar_try_wait(smem_u32(&ctl->full[s2]), 1) &&
                           globaltimer_ns() - t0 < 20000000ull) {}
            }
        }
    } else if (warp == 1 || (warp == 15 && p.n_issuers == 2)) {
        // ---------------- MMA issuer(s): the warp walks the loops in lockstep, lane 0 issues. With two issuers, issuer i
        // takes the CTA's tiles i, i + 2, ..., reads ring i and owns the accumulator buffers i*acc_per .. + acc_per - 1.
        const uint32_t leader = lane == 0 ? 1u : 0u;
        const uint32_t idesc = make_idesc_bf16(kBM, p.BN, 0, B_MN ? 1 : 0);
        const uint64_t bstep = B_MN ? 128ull : 2ull;
        const uint32_t b_lbo = B_MN ? 8192u : 16u;
        const int last_steps = (p.c_red - (p.k_chunks - 1) * kKC + 15) / 16;      // k-steps of a tap's last chunk
        const int NI = p.n_issuers, issuer = warp == 1 ? 0 : 1;
        const int SR = p.stages / NI, sbase = issuer * SR;
        int s = 0, ph = 0, b = 0, aph = 0, nt = 0;
        int consumed = 0;
        (void)consumed;
        bool ok = true;
        if (p.resident) ok = mbar_wait(smem_u32(&ctl->w_full), 0, abort_flag, p.status, 8);
        for (int tile = blockIdx.x + issuer * (int)gridDim.x; tile < total_tiles && ok; tile += NI * (int)gridDim.x, ++nt) {
            if (NI == 2) { b = p.acc_per == 2 ? issuer * 2 + (nt & 1) : issuer; aph = p.acc_per == 2 ? (nt >> 1) & 1 : nt & 1; }
            ok = mbar_wait(smem_u32(&ctl->acc_empty[b]), aph ^ 1, abort_flag, p.status, 7);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(b * p.BN);
            uint32_t acc = 0u;
            for (int tap = 0; tap < p.taps && ok; ++tap) {
                for (int kc = 0; kc < p.k_chunks; ++kc) {
                    ok = mbar_wait(smem_u32(&ctl->full[sbase + s]), ph, abort_flag, p.status, 2);
                    if (!ok) break;
                    if (warp == 1) GTRACE(4, consumed);
                    if (warp == 1 && consumed == 0) CTRACE(4);
                    tc_fence_after();
                    const uint32_t a_src = data_base + (uint32_t)(sbase + s) * stage_bytes;
                    const uint32_t b_src = p.resident ? w_base + (uint32_t)(tap * p.k_chunks + kc) * b_slot : a_src + a_bytes;
                    // one descriptor per operand and stage; a k-step only moves the 14-bit start-address field
                    // (units of 16 bytes): +32 B inside a K-major row, +2048 B (16 rows) in an MN-major tile
                    const uint64_t ad0 = make_desc(a_src, 16u, 1024u);
                    const uint64_t bd0 = make_desc(b_src, b_lbo, 1024u);
                    if (kc + 1 < p.k_chunks || last_steps == 4) {
                        umma_bf16_lead(d_tmem, ad0, bd0, idesc, acc, leader);
#pragma unroll
                        for (int k = 1; k < 4; ++k) umma_bf16_lead(d_tmem, ad0 + 2ull * k, bd0 + bstep * k, idesc, 1u, leader);
                    } else {
                        for (int k = 0; k < last_steps; ++k) umma_bf16_lead(d_tmem, ad0 + 2ull * k, bd0 + bstep * k, idesc, k ? 1u : acc, leader);
                    }
                    acc = 1u;
                    umma_commit_lead(smem_u32(&ctl->empty[sbase + s]), leader);   // frees the stage when these MMAs have read it
                    if (warp == 1) GTRACE(5, consumed);
                    ++consumed;
                    if (++s == SR) { s = 0; ph ^= 1; }
                }
            }
            if (ok) umma_commit_lead(smem_u32(&ctl->acc_full[b]), leader);   // this tile's accumulator is complete
            if (NI == 1 && ++b == p.epi_groups) { b = 0; aph ^= 1; }
            if (warp == 1) CTRACE(5);
        }
    } else if (warp - 2 < 4 * p.epi_groups) {
        // ---------------- epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31; group g drains accumulator buffer g,
        // i.e. the tiles tc = g, g + G, g + 2G, ... of this CTA
        const int quarter = warp & 3, group = (warp - 2) >> 2, G = p.epi_groups;
        const uint32_t slab0 = (p.alias_staging ? data_base : staging_base) + (uint32_t)(warp - 2) * (kSlabs * 4096u);
        // statistics: one row of partial sums per epilogue warp of the grid, [2][ld_out] floats, accumulated over the warp's tiles
        float *my_stats = (STATS && p.stats) ? p.stats + ((size_t)blockIdx.x * (4 * G) + (warp - 2)) * 2 * p.ld_out : nullptr;
        const uint32_t st_acc = smem_base + (uint32_t)p.stats_off + (uint32_t)(warp - 2) * (uint32_t)p.stats_warp;
        if (my_stats) {
            for (int e = lane; e < 2 * p.ld_out; e += 32) my_stats[e] = 0.f;
            stats_clear(st_acc, lane, (p.BN + 63) / 64);
            __syncwarp();
        }
        int tc = group, sl = 0;
        bool ok = true;
        for (int tile = blockIdx.x + group * gridDim.x; tile < total_tiles && ok; tile += G * gridDim.x, tc += G) {
            int b = group, aph = (tc / G) & 1;
            if (p.n_issuers == 2) {                     // G == 2: group g serves issuer g, whose nt-th tile this is
                const int nt = tc >> 1;
                b = p.acc_per == 2 ? group * 2 + (nt & 1) : group;
                aph = p.acc_per == 2 ? (nt >> 1) & 1 : nt & 1;
            }
            const int n_tile = tile % p.n_tiles, m_tile = tile / p.n_tiles;
            const int m0 = m_tile * kBM, n0 = n_tile * p.BN;
            // direct stores: this thread's raster pixel and where it lands in the output view
            const int m = m0 + quarter * 32 + lane;
            const bool row_ok = !p.tma_store && m < p.M_total;
            size_t row_off = 0;
            int cell_h = 0, cell_w = 0, img = 0;
            if (row_ok) {
                const int j = m % p.Qd, t = m / p.Qd, i = t % p.Pd;
                img = t / p.Pd;
                cell_h = i * p.o_step;
                cell_w = j * p.o_step;
                row_off = ((size_t)(img * p.oH + cell_h + p.o_h0) * p.oW + cell_w + p.o_w0) * (size_t)p.ld_out;
            }
            if (!p.tma_store && p.zero_mask && n_tile == 0) {
                // stride-2 data gradient: the pixels of each 2x2 cell that no tap reaches are zeros. They do not depend on the
                // accumulator, so the warp writes them (a row at a time, lanes on consecutive 16-byte pieces) while the
                // main loop is still running
                for (int r = 0; r < 32; ++r) {
                    if (!__shfl_sync(0xffffffffu, row_ok ? 1 : 0, r)) continue;
                    const int ch_ = __shfl_sync(0xffffffffu, cell_h, r), cw_ = __shfl_sync(0xffffffffu, cell_w, r);
                    const int im_ = __shfl_sync(0xffffffffu, img, r);
                    for (int ab = 0; ab < 4; ++ab) {
                        if (!((p.zero_mask >> ab) & 1)) continue;
                        const int hh = ch_ + (ab >> 1), ww = cw_ + (ab & 1);
                        if (hh >= p.oH || ww >= p.oW) continue;
                        const size_t off = ((size_t)(im_ * p.oH + hh) * p.oW + ww) * (size_t)p.ld_out;
                        if (p.out_f32) {
                            float *o = (float *)p.out + off;
                            for (int e = lane; e < p.n_cols; e += 32) o[e] = 0.f;
                        } else {
                            __nv_bfloat16 *o = (__nv_bfloat16 *)p.out + off;
                            const int whole = p.n_cols & ~7;
                            for (int e = lane * 8; e < whole; e += 256) *reinterpret_cast<uint4 *>(o + e) = make_uint4(0, 0, 0, 0);
                            if (lane < p.n_cols - whole) o[whole + lane] = __float2bfloat16_rn(0.f);
                        }
                    }
                }
            }
            ok = mbar_wait(smem_u32(&ctl->acc_full[b]), aph, abort_flag, p.status, 3);
            if (!ok) break;
            if (quarter == 0) GTRACE(6, tc);
            tc_fence_after();
            const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * p.BN);
            if (p.tma_store) {
                // Each warp stages its 32 rows x 64 channels (4 KB, 128-byte swizzle) and stores it with one TMA store,
                // which drops the channels past the true count and the rows past the last pixel. Two slabs alternate.
                const int n_chunks = (p.BN + 63) / 64;
                for (int ch = 0; ch < n_chunks; ++ch, sl ^= 1) {
                    const uint32_t slab = slab0 + (uint32_t)sl * 4096u;
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the slab's previous store has read it
                    __syncwarp();
                    const int groups = min(4, (p.BN - ch * 64) / 16);
                    uint32_t v[4][16];
                    // all of the chunk's TMEM loads are issued before the single wait
#pragma unroll
                    for (int g = 0; g < 4; ++g)
                        if (g < groups) tmem_ld16(lane_addr + (uint32_t)(ch * 64 + g * 16), v[g]);
                    tmem_ld_wait();
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        if (g >= groups) break;
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            __nv_bfloat162 b0 = __floats2bfloat162_rn(__uint_as_float(v[g][8 * h + 0]), __uint_as_float(v[g][8 * h + 1]));
                            __nv_bfloat162 b1 = __floats2bfloat162_rn(__uint_as_float(v[g][8 * h + 2]), __uint_as_float(v[g][8 * h + 3]));
                            __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(v[g][8 * h + 4]), __uint_as_float(v[g][8 * h + 5]));
                            __nv_bfloat162 b3 = __floats2bfloat162_rn(__uint_as_float(v[g][8 * h + 6]), __uint_as_float(v[g][8 * h + 7]));
                            const uint32_t j = (uint32_t)(g * 2 + h);
                            const uint32_t addr = slab + (uint32_t)lane * 128u + ((j ^ ((uint32_t)lane & 7u)) << 4);
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(*reinterpret_cast<uint32_t *>(&b0)),
                                         "r"(*reinterpret_cast<uint32_t *>(&b1)), "r"(*reinterpret_cast<uint32_t *>(&b2)),
                                         "r"(*reinterpret_cast<uint32_t *>(&b3))
                                         : "memory");
                        }
                    }
                    if (ch + 1 >= n_chunks) {
                        // every TMEM read of this tile by this warp is done: hand the buffer back to the MMA issuer
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[b]));
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        if (m0 + quarter * 32 < p.M_total) tma_store_2d(&tmC, slab, n0 + ch * 64, m0 + quarter * 32);
                        tma_store_commit();
                    }
                    if (STATS && p.stats) {
                        const int left = p.M_total - (m0 + quarter * 32);
                        const uint32_t rows = left >= 32 ? 0xffffffffu : (left > 0 ? (1u << left) - 1u : 0u);
                        chunk_stats(slab, 0, rows, lane, st_acc + (uint32_t)ch * 512u);
                    }
                }
                // several channel tiles: the sums of this tile's columns leave shared memory now; one tile: after the last tile
                if (my_stats && p.n_tiles > 1) stats_flush(st_acc, lane, my_stats, p.ld_out, n0, n_chunks, p.n_cols, true);
                if (quarter == 0) GTRACE(7, tc);
                continue;
            }
            // ---- direct stores (fp32 outputs, strided stride-2 data-gradient outputs)
            for (int c0 = 0; c0 < p.BN; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(lane_addr + (uint32_t)c0, v);
                tmem_ld_wait();
                if (c0 + 16 >= p.BN) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[b]));
                }
                const int col = n0 + c0;
                if (!row_ok || col >= p.n_cols) continue;
                const int nvalid = min(16, p.n_cols - col);
                if (p.out_f32) {
                    float *o = (float *)p.out + row_off + col;
                    if (nvalid == 16) {
#pragma unroll
                        for (int g = 0; g < 4; ++g)
                            reinterpret_cast<float4 *>(o)[g] = make_float4(__uint_as_float(v[4 * g]), __uint_as_float(v[4 * g + 1]),
                                                                          __uint_as_float(v[4 * g + 2]), __uint_as_float(v[4 * g + 3]));
                    } else {
                        for (int e = 0; e < nvalid; ++e) o[e] = __uint_as_float(v[e]);
                    }
                } else {
                    __nv_bfloat16 *o = (__nv_bfloat16 *)p.out + row_off + col;
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        if (nvalid >= 8 * (g + 1)) {
                            uint4 pk;
                            __nv_bfloat162 b0 = __floats2bfloat162_rn(__uint_as_float(v[8 * g + 0]), __uint_as_float(v[8 * g + 1]));
                            __nv_bfloat162 b1 = __floats2bfloat162_rn(__uint_as_float(v[8 * g + 2]), __uint_as_float(v[8 * g + 3]));
                            __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(v[8 * g + 4]), __uint_as_float(v[8 * g + 5]));
                            __nv_bfloat162 b3 = __floats2bfloat162_rn(__uint_as_float(v[8 * g + 6]), __uint_as_float(v[8 * g + 7]));
                            pk.x = *reinterpret_cast<uint32_t *>(&b0);
                            pk.y = *reinterpret_cast<uint32_t *>(&b1);
                            pk.z = *reinterpret_cast<uint32_t *>(&b2);
                            pk.w = *reinterpret_cast<uint32_t *>(&b3);
                            *reinterpret_cast<uint4 *>(o + 8 * g) = pk;
                        } else {
                            for (int e = 8 * g; e < nvalid; ++e) o[e] = __float2bfloat16_rn(__uint_as_float(v[e]));
                        }
                    }
                }
            }
        }
        if (my_stats && p.n_tiles == 1) stats_flush(st_acc, lane, my_stats, p.ld_out, 0, (p.BN + 63) / 64, p.n_cols, false);
        if (p.tma_store && lane == 0) tma_store_wait_read();     // the staging slabs must outlive the stores' reads
        if (warp == 2) CTRACE(6);
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 0) CTRACE(7);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ------------------------------------------------------------------------------------------ halo kernel (RxS, stride 1)
// For a stride-1 RxS filter the per-tap im2col loads fetch every input pixel R*S times. Here each input pixel row is
// fetched ONCE per 64-channel chunk: a tile is `nr` output rows of one image, laid out as a raster of pitch
// Wp = Q + S - 1 (the S - 1 extra columns per row are garbage outputs that are never stored). One tiled 4-D TMA load
// brings the (nr + R - 1) x Wp input positions of the tile, halo included, zero-filled outside the image. In that
// raster the input position of output position m for tap (r, s) is m + r*Wp + s, a constant row shift, and the
// 128-byte swizzle is a function of the absolute shared-memory address, so tap (r, s) is simply the same A tile read
// through a descriptor whose start address is (r*Wp + s) rows further on. Weights: if all taps x chunks of the CTA's
// channel tile fit in shared memory they are loaded once and stay resident; otherwise they stream through a ring.
struct HaloP {
    int N, P, Q, Wp, nr, row_tiles;      // images, output rows/cols, raster pitch, output rows per tile, tiles per image
    int n_cols, BN, n_tiles;
    int c_red, k_chunks, taps;
    int lo_h, lo_w;                      // source coordinate of raster position (0, 0) for tap offset (0, 0)
    int a_box_bytes, a_alloc;            // bytes one A load brings / bytes reserved per A stage
    int stages_a, stages_b, resident;    // ring depths; resident: weights loaded once
    int n_issuers, acc_per;              // MMA issuer warps (each with its own A ring of stages_a / n_issuers stages); accumulators per issuer (1 or 2)
    int shared_b;                        // two pipelines fed by ONE weight stream: a stage is read by both issuers (their tiles of a round)
    int row32;                           // 1: 16 channel lanes per pixel, 32-byte rows and swizzle (the space-to-depth stem): one MMA per tap
    int b_slot, b_rows, staging;         // bytes reserved per weight tile, rows a K-major weight box brings, bytes of an epilogue group's staging slab
    int tmem_cols, tma_store, out_f32, ld_out;
    int oH, oW, o_step, o_h0, o_w0;      // direct stores: raster (n, i, j) -> out[((n*oH + i*o_step + o_h0)*oW + j*o_step + o_w0)*ld_out]
    int stats_off;                       // byte offset in shared memory of the epilogue warps' statistics accumulators
    int stats_warp;                      // bytes of one warp's accumulators: 512 per 64-channel chunk of the tile
    float *stats;                        // optional: per epilogue warp and channel, sum and sum of squares of the stored bf16
    void *out;
    unsigned int *status;
    unsigned char tap_oh[kMaxTaps], tap_ow[kMaxTaps];
    unsigned short tap_wt[kMaxTaps];
};

constexpr int kHaloMaxIssuers = 4;

// Coordinates of the tiles t0, t0 + D, t0 + 2D, ... of a halo launch, advanced without integer divisions (a division costs
// a single issuing thread ~150 cycles, and the smallest tiles are only a few hundred cycles of work).
struct TileWalk {
    int n_tile, rt, img;          // channel tile, row tile within the image, image
    int dn, d_rt, d_img, n_tiles, row_tiles;
    __device__ __forceinline__ void init(int tile, int D, int n_tiles_, int row_tiles_)
    {
        n_tiles = n_tiles_; row_tiles = row_tiles_;
        n_tile = tile % n_tiles;
        const int m_tile = tile / n_tiles;
        img = m_tile / row_tiles; rt = m_tile - img * row_tiles;
        dn = D % n_tiles;
        const int dm = D / n_tiles;
        d_img = dm / row_tiles; d_rt = dm - d_img * row_tiles;
    }
    __device__ __forceinline__ void next()
    {
        n_tile += dn;
        rt += d_rt; img += d_img;
        if (n_tile >= n_tiles) { n_tile -= n_tiles; ++rt; }
        while (rt >= row_tiles) { rt -= row_tiles; ++img; }
    }
};
// Device-side timeline for tuning: a build with -DPT_DEVICE_TRACE makes CTA 0 stamp %globaltimer at the hand-over points of
// each role (producer issue, accumulator free, operands landed, MMAs committed, epilogue start, store issued) and exports
// pt_debug_halo_trace / pt_debug_wgrad_trace / pt_debug_gemm_trace to read the stamps back. The normal build compiles the macros away.
#ifdef PT_DEVICE_TRACE
__device__ unsigned long long g_halo_trace[8][64];
#define HTRACE(role, idx) do { if (blockIdx.x == 0 && (idx) < 64 && (threadIdx.x & 31) == 0) g_halo_trace[role][idx] = globaltimer_ns(); } while (0)
#else
#define HTRACE(role, idx) do { } while (0)
#endif

struct __align__(8) HCtl {
    uint64_t full_a[4], empty_a[4];
    uint64_t full_b[kMaxStages], empty_b[kMaxStages];
    uint64_t w_full;
    uint64_t acc_full[2 * kHaloMaxIssuers], acc_empty[2 * kHaloMaxIssuers];
    uint32_t tap_aoff[kMaxTaps];         // row shift of each tap in descriptor units (16 bytes)
    uint32_t tmem_base;
    int abort_flag;
};

// warp 0 (and 13): TMA producers (weights; with resident weights warp 0 also brings the activations); warps 14, 15: activation
// producers of the streamed-weight pipelines; warp 1 and warps 10..12: MMA issuers; warps 2..9: two groups of four epilogue warps
constexpr int kHaloThreads = 512;

// Issuing one tcgen05.mma costs the issuing warp 50 to 100 cycles of instruction time, more than a narrow MMA (N <= 64)
// takes to execute, so with a single issuer the tensor pipe of a small-channel layer idles most of the time. The
// kernel therefore runs up to four issuer warps, each on its own scheduler: issuer i owns accumulator buffer i and
// an A ring of its own (a waiter may lag an mbarrier by at most one phase, so issuers cannot share a ring), and takes
// the tiles i, i + I, i + 2I, ... of the CTA. Weights that stream through a ring keep a single issuer.
template <bool B_MN, bool STATS>
__global__ void __launch_bounds__(kHaloThreads, 1) conv_halo_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                     const __grid_constant__ CUtensorMap tmB,
                                                                     const __grid_constant__ CUtensorMap tmC, const HaloP p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    HCtl *ctl = reinterpret_cast<HCtl *>(smem_raw);
    const uint32_t smem_base = smem_u32(smem_raw);
    const uint32_t staging_base = (smem_base + (uint32_t)sizeof(HCtl) + 1023u) & ~1023u;
    const uint32_t b_base = staging_base + 2u * (uint32_t)p.staging;
    // bytes one weight tile brings: a K-major tile only holds the rows (output channels) that exist
    const uint32_t b_bytes = B_MN ? (uint32_t)((p.BN + 63) / 64) * 8192u : (uint32_t)p.b_rows * (p.row32 ? 32u : 128u);
    const uint32_t b_slot = (uint32_t)p.b_slot;
    const uint32_t n_bslots = p.resident ? (uint32_t)(p.taps * p.k_chunks) : (uint32_t)p.stages_b;
    const uint32_t a_base = b_base + n_bslots * b_slot;
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m_tiles = p.N * p.row_tiles;
    const int total_tiles = m_tiles * p.n_tiles;
    const int NI = p.n_issuers, SR = p.stages_a / NI;        // issuers, A stages per issuer ring

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages_a; ++s) { mbar_init(smem_u32(&ctl->full_a[s]), 1); mbar_init(smem_u32(&ctl->empty_a[s]), 1); }
        for (int s = 0; s < p.stages_b; ++s) { mbar_init(smem_u32(&ctl->full_b[s]), 1); mbar_init(smem_u32(&ctl->empty_b[s]), p.shared_b ? 2 : 1); }
        mbar_init(smem_u32(&ctl->w_full), 1);
        for (int b = 0; b < 2 * kHaloMaxIssuers; ++b) { mbar_init(smem_u32(&ctl->acc_full[b]), 1); mbar_init(smem_u32(&ctl->acc_empty[b]), 4); }
        ctl->abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        if (p.tma_store) prefetch_tmap(&tmC);
    }
    if (threadIdx.x < p.taps) ctl->tap_aoff[threadIdx.x] = (uint32_t)(p.tap_oh[threadIdx.x] * p.Wp + p.tap_ow[threadIdx.x]) * (p.row32 ? 2u : 8u);
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int issuer = warp == 1 ? 0 : warp - 9;             // warps 10, 11, 12 -> issuers 1, 2, 3
    // the weight producers do not read the previous kernel's output: resident weights are issued first and the wait follows
    // them (below); the producers of streamed weights never need it
    // Warps that load activations wait just before their first activation load, after their set-up (tile walk, ring positions).
    if (!(warp == 0 || ((warp == 13 || warp == 14 || warp == 15) && !p.resident))) grid_dependency_wait();
    grid_launch_dependents();

    // Streamed weights with two issuers: two complete pipelines (producer warp, A ring, B ring, issuer warp, accumulators),
    // one per tile parity. Resident weights: one producer feeds every issuer's A ring.
    // With `shared_b` the two pipelines read the same weight stages: the tiles of a round (blockIdx.x + 2r*grid and + (2r+1)*grid)
    // use the same weights, so one stream through the whole ring feeds both issuers, half the bytes and twice the depth.
    const int n_prod = p.resident ? 1 : NI;
    const int SB = p.shared_b ? p.stages_b : p.stages_b / n_prod;     // weight stages per weight stream
    // Streamed weights: the activation boxes have a producer warp of their own per pipeline (14, 15), so that the next tile's
    // boxes go out as soon as their stage is free instead of behind the weight loads of the current tile, which wait for the
    // MMAs (the next tile's activations used to be issued only when the current tile was nearly done: ~4 us per tile exposed).
    const bool a_warp = !p.resident && (warp == 14 || (warp == 15 && n_prod == 2));
    if (warp == 0 || (warp == 13 && n_prod == 2 && !p.shared_b) || a_warp) {
        if (lane == 0) {
            // ---------------- TMA producer(s)
            const int pid = (warp == 0 || warp == 14) ? 0 : 1;
            const bool a_role = a_warp || p.resident, b_role = !a_warp && !p.resident;
            if (p.resident) {
                // n_tiles == 1 here: the whole weight tensor of the layer, tap by tap and chunk by chunk, once
                const uint32_t bar = smem_u32(&ctl->w_full);
                mbar_arrive_expect_tx(bar, (uint32_t)(p.taps * p.k_chunks) * b_bytes);
                for (int tap = 0; tap < p.taps; ++tap)
                    for (int kc = 0; kc < p.k_chunks; ++kc) {
                        const uint32_t dst = b_base + (uint32_t)(tap * p.k_chunks + kc) * b_slot;
                        const int wtap = p.tap_wt[tap];
                        if (!B_MN) tma_load_3d(dst, &tmB, bar, kc * kKC, wtap, 0);
                        else for (int nb = 0; nb < (p.BN + 63) / 64; ++nb) tma_load_3d(dst + (uint32_t)nb * 8192u, &tmB, bar, nb * 64, wtap, kc * kKC);
                    }
            }
            bool dep_waited = false;             // the activations are the previous kernel's output
            int tc = pid;
            TileWalk tw;
            tw.init((int)blockIdx.x + pid * (int)gridDim.x, n_prod * (int)gridDim.x, p.n_tiles, p.row_tiles);
            // ring = tc % NI; every ring has carried (tc / NI) * k_chunks chunks before its tile of this round: position and
            // phase of that count in a ring of SR stages, advanced per round
            int ring = pid % NI, base_pos = 0, base_ph = 0;
            const int kdiv = p.k_chunks / SR, kmod = p.k_chunks - kdiv * SR;
            int sb_pos = 0, sb_ph = 0;                         // position in this pipeline's weight ring
            for (int tile = blockIdx.x + pid * (int)gridDim.x; tile < total_tiles && !*abort_flag; tile += n_prod * (int)gridDim.x, tc += n_prod) {
                const int img = tw.img, p0 = tw.rt * p.nr;
                const int n0 = tw.n_tile * p.BN;
                bool ok = true;
                int pos = base_pos, pha = base_ph;
                for (int kc = 0; kc < p.k_chunks && ok; ++kc) {
                    const int sa = ring * SR + pos, ph_use = pha;
                    if (++pos == SR) { pos = 0; pha ^= 1; }
                    if (a_role) {
                        ok = mbar_wait(smem_u32(&ctl->empty_a[sa]), ph_use ^ 1, abort_flag, p.status, 11);
                        if (!ok) break;
                        const uint32_t bar = smem_u32(&ctl->full_a[sa]);
                        HTRACE(0, tc);
                        mbar_arrive_expect_tx(bar, (uint32_t)p.a_box_bytes);
                        if (!dep_waited) { grid_dependency_wait(); dep_waited = true; }
                        tma_load_4d(a_base + (uint32_t)sa * (uint32_t)p.a_alloc, &tmA, bar, kc * kKC, p.lo_w, p0 + p.lo_h, img);
                    }
                    if (!b_role) continue;
                    for (int tap = 0; tap < p.taps; ++tap) {
                        const int sb = (p.shared_b ? 0 : pid * SB) + sb_pos, phb = sb_ph;
                        if (++sb_pos == SB) { sb_pos = 0; sb_ph ^= 1; }
                        ok = mbar_wait(smem_u32(&ctl->empty_b[sb]), phb ^ 1, abort_flag, p.status, 12);
                        if (!ok) break;
                        const uint32_t bbar = smem_u32(&ctl->full_b[sb]);
                        const uint32_t dst = b_base + (uint32_t)sb * b_slot;
                        const int wtap = p.tap_wt[tap];
                        mbar_arrive_expect_tx(bbar, b_bytes);
                        if (!B_MN) tma_load_3d(dst, &tmB, bbar, kc * kKC, wtap, n0);
                        else for (int nb = 0; nb < (p.BN + 63) / 64; ++nb) tma_load_3d(dst + (uint32_t)nb * 8192u, &tmB, bbar, n0 + nb * 64, wtap, kc * kKC);
                    }
                }
                if (!ok) break;
                tw.next();
                ring += n_prod;
                while (ring >= NI) {                           // next round: every ring has carried k_chunks more
                    ring -= NI;
                    base_pos += kmod;
                    int wraps = kdiv;
                    if (base_pos >= SR) { base_pos -= SR; ++wraps; }
                    base_ph ^= wraps & 1;
                }
            }
            if (*abort_flag && pid == 0 && a_role) {   // bounded drain of the copies in flight before the shared memory is released
                const uint64_t t0 = globaltimer_ns();
                for (int s = 0; s < p.stages_a; ++s)
                    while (!mbar_try_wait(smem_u32(&ctl->full_a[s]), 0) && !mbar_try_wait(smem_u32(&ctl->full_a[s]), 1) &&
                           globaltimer_ns() - t0 < 20000000ull) {}
            }
        }
    } else if (warp == 1 || (warp >= 10 && issuer < NI)) {
        // ---------------- MMA issuer `issuer`: the whole warp walks the loops in lockstep, lane 0 issues
        const uint32_t leader = lane == 0 ? 1u : 0u;
        const uint32_t idesc = make_idesc_bf16(kBM, p.BN, 0, B_MN ? 1 : 0);
        const uint64_t bstep = B_MN ? 128ull : 2ull;
        const uint32_t b_lbo = B_MN ? 8192u : 16u;
        int sb_pos = 0, sb_ph = 0;                            // position in this issuer's weight ring
        int s_loc = 0, pha = 0;                               // position in this issuer's A ring
        bool ok = true;
        if (p.resident) ok = mbar_wait(smem_u32(&ctl->w_full), 0, abort_flag, p.status, 13);
        int nt = 0;                                           // tiles this issuer has started
        for (int tc = issuer; ok; tc += NI, ++nt) {
            const int tile = blockIdx.x + tc * (int)gridDim.x;
            if (tile >= total_tiles) {
                // shared weight stream: the other issuer may still have a tile in this round; its stages need this issuer's
                // release too, given in step with the stream
                if (p.shared_b && issuer == 1 && tile - (int)gridDim.x < total_tiles) {
                    for (int i = 0; i < p.k_chunks * p.taps && ok; ++i) {
                        const int sb = sb_pos, phb = sb_ph;
                        if (++sb_pos == SB) { sb_pos = 0; sb_ph ^= 1; }
                        ok = mbar_wait(smem_u32(&ctl->full_b[sb]), phb, abort_flag, p.status, 16);
                        if (ok && lane == 0) mbar_arrive(smem_u32(&ctl->empty_b[sb]));
                    }
                }
                break;
            }
            // accumulator buffers issuer*acc_per .. +acc_per-1, used in turn
            const int b = p.acc_per == 2 ? issuer * 2 + (nt & 1) : issuer, aph = p.acc_per == 2 ? (nt >> 1) & 1 : nt & 1;
            ok = mbar_wait(smem_u32(&ctl->acc_empty[b]), aph ^ 1, abort_flag, p.status, 14);
            if (!ok) break;
            HTRACE(1, tc);
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(b * p.BN);
            uint32_t accumulate = 0u;
            for (int kc = 0; kc < p.k_chunks && ok; ++kc) {
                const int sa = issuer * SR + s_loc;
                ok = mbar_wait(smem_u32(&ctl->full_a[sa]), pha, abort_flag, p.status, 15);
                if (!ok) break;
                HTRACE(2, tc);
                tc_fence_after();
                const int rem = p.c_red - kc * kKC;
                const int ksteps = rem >= kKC ? 4 : (rem + 15) / 16;
                const uint64_t abase = make_desc(a_base + (uint32_t)sa * (uint32_t)p.a_alloc, 16u, 1024u);
                if (p.row32) {
                    // 32-byte rows: a pixel's 16 lanes are one K step, so a tap is a single MMA on the row-shifted tile
                    const uint64_t a32 = make_desc_sw32(a_base + (uint32_t)sa * (uint32_t)p.a_alloc, 256u);
                    uint64_t b32 = make_desc_sw32(b_base, 256u);
                    const uint64_t b_tap_step = (uint64_t)(b_slot >> 4);
                    for (int tap = 0; tap < p.taps; ++tap, b32 += b_tap_step) {
                        umma_bf16_lead(d_tmem, a32 + ctl->tap_aoff[tap], b32, idesc, accumulate, leader);
                        accumulate = 1u;
                    }
                } else if (p.resident) {
                    // every tap is the same A tile read through a descriptor that starts (r*Wp + s) rows further on
                    uint64_t bd0 = make_desc(b_base + (uint32_t)kc * b_slot, b_lbo, 1024u);
                    const uint64_t b_tap_step = (uint64_t)(((uint32_t)p.k_chunks * b_slot) >> 4);
                    if (ksteps == 4) {
                        for (int tap = 0; tap < p.taps; ++tap, bd0 += b_tap_step) {
                            const uint64_t ad0 = abase + ctl->tap_aoff[tap];
#pragma unroll
                            for (int k = 0; k < 4; ++k) { umma_bf16_lead(d_tmem, ad0 + 2ull * k, bd0 + bstep * k, idesc, accumulate, leader); accumulate = 1u; }
                        }
                    } else {
                        for (int tap = 0; tap < p.taps; ++tap, bd0 += b_tap_step) {
                            const uint64_t ad0 = abase + ctl->tap_aoff[tap];
                            for (int k = 0; k < ksteps; ++k) { umma_bf16_lead(d_tmem, ad0 + 2ull * k, bd0 + bstep * k, idesc, accumulate, leader); accumulate = 1u; }
                        }
                    }
                } else {
                    for (int tap = 0; tap < p.taps; ++tap) {
                        const int sb = (p.shared_b ? 0 : issuer * SB) + sb_pos, phb = sb_ph;
                        if (++sb_pos == SB) { sb_pos = 0; sb_ph ^= 1; }
                        ok = mbar_wait(smem_u32(&ctl->full_b[sb]), phb, abort_flag, p.status, 16);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t ad0 = abase + ctl->tap_aoff[tap];
                        const uint64_t bd0 = make_desc(b_base + (uint32_t)sb * b_slot, b_lbo, 1024u);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            if (k < ksteps) { umma_bf16_lead(d_tmem, ad0 + 2ull * k, bd0 + bstep * k, idesc, accumulate, leader); accumulate = 1u; }
                        umma_commit_lead(smem_u32(&ctl->empty_b[sb]), leader);
                    }
                }
                if (ok) umma_commit_lead(smem_u32(&ctl->empty_a[sa]), leader);
                if (++s_loc == SR) { s_loc = 0; pha ^= 1; }
            }
            if (ok) umma_commit_lead(smem_u32(&ctl->acc_full[b]), leader);
            HTRACE(3, tc);
        }
    } else if (warp >= 2 && warp < 10) {
        // ---------------- epilogue: group g (four warps) drains the accumulator buffers of its parity
        const int quarter = warp & 3, group = (warp - 2) >> 2;
        const int gtid = (warp - 2 - group * 4) * 32 + lane;         // 0..127 within the group
        const uint32_t slab = staging_base + (uint32_t)group * (uint32_t)p.staging;
        // statistics: one row of partial sums per epilogue warp of the grid, [2][ld_out] floats, accumulated over the warp's tiles
        float *my_stats = (STATS && p.stats) ? p.stats + ((size_t)blockIdx.x * 8 + (warp - 2)) * 2 * p.ld_out : nullptr;
        const uint32_t st_acc = smem_base + (uint32_t)p.stats_off + (uint32_t)(warp - 2) * (uint32_t)p.stats_warp;
        if (my_stats) {
            for (int e = lane; e < 2 * p.ld_out; e += 32) my_stats[e] = 0.f;
            stats_clear(st_acc, lane, (p.BN + 63) / 64);
            __syncwarp();
        }
        bool ok = true;
        const int ni_shift = NI == 4 ? 2 : NI == 2 ? 1 : 0;   // NI is 1, 2 or 4
        TileWalk tw;
        tw.init((int)blockIdx.x + group * (int)gridDim.x, 2 * (int)gridDim.x, p.n_tiles, p.row_tiles);
        for (int tc = group; ok; tc += 2, tw.next()) {
            const int tile = blockIdx.x + tc * (int)gridDim.x;
            if (tile >= total_tiles) break;
            // tile tc is the nt-th tile of issuer tc % NI (NI is 1 or even, so a group always serves the same issuers)
            const int iss = tc & (NI - 1), nt = tc >> ni_shift;
            const int b = p.acc_per == 2 ? iss * 2 + (nt & 1) : iss, aph = p.acc_per == 2 ? (nt >> 1) & 1 : nt & 1;
            const int img = tw.img, p0 = tw.rt * p.nr;
            const int n0 = tw.n_tile * p.BN;
            ok = mbar_wait(smem_u32(&ctl->acc_full[b]), aph, abort_flag, p.status, 17);
            if (!ok) break;
            if (gtid == 0) HTRACE(4, tc);
            tc_fence_after();
            const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * p.BN);
            const int m = quarter * 32 + lane;                       // raster position of this thread's accumulator row
            if (p.tma_store) {
                const int n_chunks = (p.BN + 63) / 64;
                for (int ch = 0; ch < n_chunks; ++ch) {
                    if (gtid == 0) tma_store_wait_read();            // the slab's previous store has read it
                    if (gtid == 0) HTRACE(5, tc);
                    named_barrier(1 + group, 128);
                    const int groups = min(4, (p.BN - ch * 64) / 16);
                    uint32_t v[4][16];
#pragma unroll
                    for (int g = 0; g < 4; ++g)
                        if (g < groups) tmem_ld16(lane_addr + (uint32_t)(ch * 64 + g * 16), v[g]);
                    tmem_ld_wait();
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        if (g >= groups || m >= p.nr * p.Wp) break;   // the slab only holds the tile's raster rows
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            __nv_bfloat162 b0 = __floats2bfloat162_rn(__uint_as_float(v[g][8 * h + 0]), __uint_as_float(v[g][8 * h + 1]));
                            __nv_bfloat162 b1 = __floats2bfloat162_rn(__uint_as_float(v[g][8 * h + 2]), __uint_as_float(v[g][8 * h + 3]));
                            __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(v[g][8 * h + 4]), __uint_as_float(v[g][8 * h + 5]));
                            __nv_bfloat162 b3 = __floats2bfloat162_rn(__uint_as_float(v[g][8 * h + 6]), __uint_as_float(v[g][8 * h + 7]));
                            const uint32_t j = (uint32_t)(g * 2 + h);
                            const uint32_t addr = slab + (uint32_t)m * 128u + ((j ^ ((uint32_t)m & 7u)) << 4);
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(*reinterpret_cast<uint32_t *>(&b0)),
                                         "r"(*reinterpret_cast<uint32_t *>(&b1)), "r"(*reinterpret_cast<uint32_t *>(&b2)),
                                         "r"(*reinterpret_cast<uint32_t *>(&b3))
                                         : "memory");
                        }
                    }
                    if (ch + 1 >= n_chunks) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[b]));
                    }
                    fence_proxy_async();
                    named_barrier(1 + group, 128);
                    // one store per tile and chunk: box = nr rows x Wp columns x 64 channels; the columns past Q, the rows
                    // past P and the channels past the true count fall outside the tensor and are dropped
                    if (gtid == 0) {
                        HTRACE(6, tc);
                        tma_store_4d(&tmC, slab, n0 + ch * 64, 0, p0, img);
                        tma_store_commit();
                        HTRACE(7, tc);
                    }
                    if (STATS && p.stats) {
                        // this thread's raster position is a real output pixel iff it lies inside the row and the image
                        const int ri = m / p.Wp, rj = m - ri * p.Wp;
                        const uint32_t rows = __ballot_sync(0xffffffffu, m < p.nr * p.Wp && rj < p.Q && p0 + ri < p.P);
                        chunk_stats(slab, quarter * 32, rows, lane, st_acc + (uint32_t)ch * 512u);
                    }
                }
                if (my_stats && p.n_tiles > 1) stats_flush(st_acc, lane, my_stats, p.ld_out, n0, n_chunks, p.n_cols, true);
                continue;
            }
            // ---- direct stores (fp32 outputs)
            const int i = m / p.Wp, j = m - i * p.Wp;
            const bool row_ok = m < p.nr * p.Wp && j < p.Q && p0 + i < p.P;
            const size_t row_off = ((size_t)(img * p.oH + (p0 + i) * p.o_step + p.o_h0) * p.oW + j * p.o_step + p.o_w0) * (size_t)p.ld_out;
            for (int c0 = 0; c0 < p.BN; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(lane_addr + (uint32_t)c0, v);
                tmem_ld_wait();
                if (c0 + 16 >= p.BN) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[b]));
                }
                const int col = n0 + c0;
                if (!row_ok || col >= p.n_cols) continue;
                const int nvalid = min(16, p.n_cols - col);
                if (p.out_f32) {
                    float *o = (float *)p.out + row_off + col;
                    for (int e = 0; e < nvalid; ++e) o[e] = __uint_as_float(v[e]);
                } else {
                    __nv_bfloat16 *o = (__nv_bfloat16 *)p.out + row_off + col;
                    for (int e = 0; e < nvalid; ++e) o[e] = __float2bfloat16_rn(__uint_as_float(v[e]));
                }
            }
        }
        if (my_stats && p.n_tiles == 1) stats_flush(st_acc, lane, my_stats, p.ld_out, 0, (p.BN + 63) / 64, p.n_cols, false);
        if (p.tma_store && gtid == 0) tma_store_wait_read();
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ------------------------------------------------------------------------------------------ wgrad
// dw[k][tap][c] = sum over output pixels of dy[pixel][k] * x[pixel shifted by the tap][c]   (Eq. 4)
//   GEMM per tap: M = 128 output channels k, N = BN input channels c, reduction = output pixels, 64 per stage.
//   A operand: dy[pixel][k], k contiguous -> MN-major tiles (two 64-channel boxes of a 2-D tiled map).
//   B operand: x through the im2col map (same pixel raster as the forward pass, tap offset added by the TMA unit),
//              c contiguous -> MN-major tiles (one 64-channel box per 64 columns).
//   The pixel range is split across CTAs (blockIdx.y), at most one CTA per SM in total so that all of them are resident.
//   With more than one split every CTA TMA-stores its fp32 partial tile to the workspace, announces it on a counter,
//   waits (bounded) until all splits of its tile have arrived, and then sums its share of the tile's rows over the
//   splits in ascending order: deterministic, and no second kernel.
struct WgradP {
    int K, C, taps;         // true channel counts, number of taps (R*S)
    int BN, n_tiles;        // input-channel tile
    int m_tiles;            // ceil(K / 128)
    int tpc, tap_groups;    // taps per CTA (they share the dy tile; one accumulator of BN columns each) and groups of taps
    int npix;               // N*P*Q
    int pix_per_split;      // multiple of 64
    int splits;
    int Pd, Qd, stride, lo_h, lo_w, S;
    int x_tiled;            // 1: 1x1 stride-1 filter without padding: x is a plain 2-D (channels, pixels) tiled map
    int stages, tmem_cols;
    // row-block form (stride-1 filters with several taps): a stage is `nr` output rows of one image
    int nr, Wp, RB;         // rows per unit, row pitch of both staged tiles in pixels (Q + S - 1), units per image
    int units, units_per_split;
    int ksteps;             // 16-pixel MMA steps per unit: ceil(nr * Wp / 16)
    int nb_a;               // 64-channel dy boxes per stage (1 when K <= 64)
    int lo_span;            // R - 1: extra rows of the x halo box
    int pair;               // row-block form, C <= 64: the M side of an MMA is TWO taps x 64 input channels of the x tile
                            // (the second tap is the first one shifted: the operand's 64-element block stride is that shift)
                            // and the N side is the output channels; accumulator lanes = (tap, c), columns = k
    int apc;                // accumulators per CTA (= tpc, or tpc / 2 in the paired form)
    int acc_cols;           // columns of one accumulator (= BN, or the padded K in the paired form)
    unsigned a_box, b_box;  // bytes reserved per dy box and per x box (multiples of 1024)
    float *out;             // dw
    int test_skip;          // test hook (pt_test_skip_next_arrive): split 0 does not announce its partial tile
    float *partial;         // splits > 1: workspace [blockIdx.x][tap in group][split][128][BN] fp32
    unsigned int *sync;     // splits > 1: two zeroed counters per blockIdx.x (arrived, reduced); left zero again at exit
    unsigned int *status;
};

#ifdef PT_DEVICE_TRACE
__device__ unsigned long long g_wg_trace[8][64];
#define WTRACE(i) do { if (blockIdx.x == 0 && blockIdx.y < 64 && (threadIdx.x & 31) == 0) g_wg_trace[i][blockIdx.y] = globaltimer_ns(); } while (0)
#else
#define WTRACE(i) do { } while (0)
#endif
// n / d for 0 <= n < 2^22 and a divisor known per kernel: float reciprocal plus one correction step (an integer division
// costs ~40 instructions, and the reduction below does two per 16-byte item).
__device__ __forceinline__ int fast_div(int n, int d, float inv_d)
{
    int q = __float2int_rz(__int2float_rn(n) * inv_d);
    if ((q + 1) * d <= n) ++q;
    if (q * d > n) --q;
    return q;
}

// Everything after the main loop of a weight-gradient kernel: the accumulators leave TMEM (directly to dw, or as this
// split's partial tile), the splits of a tile meet, and every CTA sums its share of the tile over the splits.
// `ring_bytes` of shared memory at `data_base` are free by then and serve as staging.
__device__ __forceinline__ void wgrad_finish(const WgradP &p, const CUtensorMap &tmP, Ctl *ctl, uint32_t data_base, uint32_t tmem_base,
                                             int ntap, int tap0, int k0, int c0, int split, int iters, uint32_t ring_bytes, int n_acc, int acc_cols)
{
    volatile int *abort_flag = &ctl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp >= 1) {
        // ---------------- epilogue: the four epilogue warps and, once they are done issuing, the four issuer warps; a warp
        // may read the TMEM lanes of quarter warp % 4, so each quarter has two warps, which take alternate 32-column chunks
        const int quarter = warp & 3, wset = (warp >= 2 && warp < 6) ? 0 : 1;
        bool ok = true;
        if (iters > 0) ok = mbar_wait(smem_u32(&ctl->accum), 0, abort_flag, p.status, 6);
        if (warp == 2) WTRACE(3);
        tc_fence_after();
        if (ok) {
            const int k = k0 + quarter * 32 + lane;
            const bool row_ok = k < p.K;
            (void)row_ok;
            const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
            if (p.splits > 1) {
                // ---- (1) this CTA's fp32 partial tile goes to the workspace through swizzled staging + TMA stores
                const int gtid = (warp - 1) * 32 + lane;
                int sl = 0, ci = 0;
                for (int tt = 0; tt < n_acc; ++tt)
                for (int cc = 0; cc < acc_cols; cc += 32, ++ci) {
                    if ((ci & 1) != wset) continue;
                    sl ^= 1;
                    const uint32_t slab = data_base + (uint32_t)((wset * 4 + quarter) * 2 + sl) * 4096u;
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
                    uint32_t lo[16], hi[16];
                    if (iters > 0) {
                        tmem_ld16(lane_addr + (uint32_t)(tt * acc_cols + cc), lo);
                        if (cc + 16 < acc_cols) tmem_ld16(lane_addr + (uint32_t)(tt * acc_cols + cc) + 16u, hi);
                        tmem_ld_wait();
                    }
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        if (iters <= 0) lo[e] = 0u;
                        if (iters <= 0 || cc + 16 >= acc_cols) hi[e] = 0u;
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t *src = j < 4 ? &lo[4 * j] : &hi[4 * (j - 4)];
                        const uint32_t addr = slab + (uint32_t)lane * 128u + (((uint32_t)j ^ ((uint32_t)lane & 7u)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(src[0]), "r"(src[1]), "r"(src[2]), "r"(src[3])
                                     : "memory");
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tmP, slab, cc, (((int)blockIdx.x * p.apc + tt) * p.splits + split) * 128 + quarter * 32);
                        tma_store_commit();
                    }
                }
                if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");      // the writes have completed
                __threadfence();
                if (warp == 2) WTRACE(4);
                named_barrier(1, 256);
                // ---- (2) every split CTA of this tile is resident (the grid is at most one CTA per SM): wait for all of them
                unsigned int *arrived = p.sync + 2 * blockIdx.x;
                if (gtid == 0) {
                    // (test hook: split 0 stays silent, so that every split of the tile runs into the bounded wait below)
                    if (!(p.test_skip && split == 0)) atomicAdd(arrived, 1u);
                    const uint64_t t0 = globaltimer_ns();
                    while (atomicAdd(arrived, 0u) < (unsigned)p.splits) {
                        if (*abort_flag) break;
                        if (globaltimer_ns() - t0 > *(volatile unsigned long long *)&g_wait_limit_ns) { record_timeout(p.status, 8); *abort_flag = 1; break; }
                        __nanosleep(64);
                    }
                }
                named_barrier(1, 256);
                if (warp == 2) WTRACE(5);
            } else if (p.pair) {
                // lanes are (tap of the pair, input channel), columns are output channels: for one column a warp's lanes
                // write consecutive floats of dw
                const int l = quarter * 32 + lane, c = l & 63;
                int ci = 0;
                for (int tt = 0; tt < n_acc; ++tt)
                for (int cc = 0; cc < acc_cols; cc += 16, ++ci) {
                    if ((ci & 1) != wset) continue;
                    const int tap = tap0 + 2 * tt + (l >> 6);
                    uint32_t v[16];
                    if (iters > 0) {
                        tmem_ld16(lane_addr + (uint32_t)(tt * acc_cols + cc), v);
                        tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int e = 0; e < 16; ++e) v[e] = 0u;
                    }
                    if (c >= p.C || tap >= tap0 + ntap) continue;
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        if (cc + e < p.K) p.out[((size_t)(cc + e) * p.taps + tap) * p.C + c] = __uint_as_float(v[e]);
                }
            } else {
            float *obase = p.out;
            // The stages are free once the accumulator is complete: each warp transposes its 32 x 32 blocks through
            // a padded shared-memory square so that a warp writes 32 consecutive floats of one dw row at a time.
            const uint32_t sq = data_base + (uint32_t)(wset * 4 + quarter) * (32u * 33u * 4u);
            int ci = 0;
            for (int tt = 0; tt < n_acc; ++tt)
            for (int cc = 0; cc < acc_cols; cc += 32, ++ci) {
                if ((ci & 1) != wset) continue;
                const int tap = tap0 + tt;
                uint32_t v[32];
                if (iters > 0) {
                    uint32_t lo[16], hi[16];
                    tmem_ld16(lane_addr + (uint32_t)(tt * acc_cols + cc), lo);
                    if (cc + 16 < acc_cols) tmem_ld16(lane_addr + (uint32_t)(tt * acc_cols + cc) + 16u, hi);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 16; ++e) { v[e] = lo[e]; v[16 + e] = (cc + 16 < acc_cols) ? hi[e] : 0u; }
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = 0u;
                }
                __syncwarp();
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(sq + (uint32_t)(lane * 33 + e) * 4u), "r"(v[e]) : "memory");
                __syncwarp();
                const int col = c0 + cc + lane;
                for (int rr = 0; rr < 32; ++rr) {
                    const int kk = k0 + quarter * 32 + rr;
                    if (kk >= p.K) break;
                    uint32_t t;
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(t) : "r"(sq + (uint32_t)(rr * 33 + lane) * 4u) : "memory");
                    if (col < p.C && cc + lane < p.BN) obase[((size_t)kk * p.taps + tap) * p.C + col] = __uint_as_float(t);
                }
            }
            }
        }
        tc_fence_before();
    }
    __syncthreads();
    if (p.splits > 1 && !*abort_flag) {
        // ---- (3) all threads: this CTA sums its share of the tile's elements over the splits
        __threadfence();
        // Work items are (tap, row, 4-column group) of the real rows of the CTA's tiles, dealt out evenly to the split CTAs.
        // The partial tiles sit in L2; what costs time is a chain of dependent loads, so every thread first issues the
        // asynchronous 16-byte copies of its items for ALL splits into the (now idle) stage memory, and only then are the
        // copies summed from shared memory in ascending split order: deterministic, whichever CTA does the work.
        const int rows_real = p.pair ? 128 : min(128, p.K - k0);
        const int ngrp = acc_cols / 4;                               // float4 groups per row (a multiple of 16 columns)
        const int items = rows_real * ngrp;
        const int total = n_acc * items;
        const int per_cta = (total + p.splits - 1) / p.splits;
        const int it_beg = split * per_cta, it_end = min(total, it_beg + per_cta);
        const size_t zstride = (size_t)128 * acc_cols;
        const float *pbase = p.partial + (size_t)blockIdx.x * p.apc * p.splits * zstride;
        const int cap = (int)(((size_t)ring_bytes) / ((size_t)p.splits * 16));   // items the stage memory holds
        const float inv_items = 1.0f / (float)items, inv_ngrp = 1.0f / (float)ngrp;
        for (int c_beg = it_beg; c_beg < it_end; c_beg += cap) {
            const int n_chunk = min(cap, it_end - c_beg);
            for (int i = threadIdx.x; i < n_chunk; i += kThreads) {
                const int idx = c_beg + i, tt = fast_div(idx, items, inv_items), item = idx - tt * items;
                const float *src = pbase + (size_t)tt * p.splits * zstride + (size_t)item * 4;
                uint32_t dst = data_base + (uint32_t)i * 16u;
                for (int z = 0; z < p.splits; ++z, src += zstride, dst += (uint32_t)n_chunk * 16u)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
            }
            asm volatile("cp.async.wait_all;" ::: "memory");
            __syncthreads();
            for (int i = threadIdx.x; i < n_chunk; i += kThreads) {
                const int idx = c_beg + i, tt = fast_div(idx, items, inv_items), item = idx - tt * items;
                const int r = fast_div(item, ngrp, inv_ngrp), col = (item - r * ngrp) * 4;
                if (!p.pair && c0 + col >= p.C) continue;
                float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
                uint32_t a = data_base + (uint32_t)i * 16u;
                for (int z = 0; z < p.splits; ++z, a += (uint32_t)n_chunk * 16u) {
                    float4 t;
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(t.x), "=f"(t.y), "=f"(t.z), "=f"(t.w) : "r"(a) : "memory");
                    sum.x += t.x; sum.y += t.y; sum.z += t.z; sum.w += t.w;
                }
                if (p.pair) {
                    // row = (tap of the pair, input channel), columns = output channels
                    const int tap = tap0 + 2 * tt + (r >> 6), c = r & 63;
                    if (c < p.C && tap < tap0 + ntap) {
                        const float v4[4] = {sum.x, sum.y, sum.z, sum.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (col + e < p.K) p.out[((size_t)(col + e) * p.taps + tap) * p.C + c] = v4[e];
                    }
                    continue;
                }
                float *dst = p.out + ((size_t)(k0 + r) * p.taps + tap0 + tt) * p.C + c0 + col;
                const int nv = min(4, p.C - (c0 + col));
                if (nv == 4 && ((uintptr_t)dst & 15) == 0) {
                    *reinterpret_cast<float4 *>(dst) = sum;           // a dw row starts on a 16-byte boundary only if C allows it
                    continue;
                }
                if (nv == 4 && ((uintptr_t)dst & 7) == 0) {
                    reinterpret_cast<float2 *>(dst)[0] = make_float2(sum.x, sum.y);
                    reinterpret_cast<float2 *>(dst)[1] = make_float2(sum.z, sum.w);
                    continue;
                }
                dst[0] = sum.x;
                if (nv > 1) dst[1] = sum.y;
                if (nv > 2) dst[2] = sum.z;
                if (nv > 3) dst[3] = sum.w;
            }
            __syncthreads();
        }
        __syncthreads();
        if (threadIdx.x == 0) WTRACE(6);
        if (threadIdx.x == 0) {
            unsigned int *arrived = p.sync + 2 * blockIdx.x, *reduced = arrived + 1;
            __threadfence();
            if (atomicAdd(reduced, 1u) == (unsigned)p.splits - 1u) {          // last one out clears the counters
                *arrived = 0u;
                *reduced = 0u;
                __threadfence();
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads) conv_wgrad_kernel(const __grid_constant__ CUtensorMap tmDy,
                                                              const __grid_constant__ CUtensorMap tmX,
                                                              const __grid_constant__ CUtensorMap tmP, const WgradP p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Ctl *ctl = reinterpret_cast<Ctl *>(smem_raw);
    const uint32_t smem_base = smem_u32(smem_raw);
    const uint32_t data_base = (smem_base + (uint32_t)sizeof(Ctl) + 1023u) & ~1023u;
    const uint32_t a_bytes = 2u * 8192u;
    const uint32_t nb_b = (uint32_t)((p.BN + 63) / 64);
    const uint32_t b_bytes = nb_b * 8192u;                            // one tap's x tile
    const uint32_t stage_bytes = a_bytes + (uint32_t)p.tpc * b_bytes;
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int bx = blockIdx.x;
    const int n_tile = bx % p.n_tiles; bx /= p.n_tiles;
    const int m_tile = bx % p.m_tiles; bx /= p.m_tiles;
    const int tap0 = bx * p.tpc;                                      // this CTA's taps: tap0 .. tap0 + ntap - 1
    const int ntap = min(p.tpc, p.taps - tap0);
    const int split = blockIdx.y;
    const int k0 = m_tile * 128, c0 = n_tile * p.BN;
    const int pix_beg = split * p.pix_per_split;
    const int pix_end = min(p.npix, pix_beg + p.pix_per_split);
    const int iters = pix_end > pix_beg ? (pix_end - pix_beg + 63) / 64 : 0;

    // Issuing is what a single thread does slowly (about 200 cycles per TMA instruction, 50 to 100 per MMA), so both
    // sides of the pipeline are spread over warps: warp 0 loads the dy tile, the four epilogue warps (idle until the
    // accumulators are complete) load the x tiles, and up to four issuer warps each own the accumulators of the taps
    // tt = i, i + NI, ... Every participant arrives on a stage's barriers itself.
    const int n_x = ntap * (int)nb_b;                                 // x boxes per stage
    const int NXP = n_x < 4 ? n_x : 4;                                // x producer warps in use
    const int NI = ntap < 4 ? ntap : 4;                               // MMA issuer warps in use
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 1u + (uint32_t)NXP);
            mbar_init(smem_u32(&ctl->empty[s]), (uint32_t)NI);
        }
        mbar_init(smem_u32(&ctl->accum), (uint32_t)NI);
        ctl->abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmDy);
        prefetch_tmap(&tmX);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int issuer = warp == 1 ? 0 : warp - 5;                      // warps 6, 7, 8 -> issuers 1, 2, 3
    // Nothing above touches global memory. The producer threads wait for the previous kernel after their set-up (pixel
    // coordinates of the first stage: several divisions) instead of before it.
    if (!((warp == 0 || (warp >= 2 && warp < 2 + NXP)) && lane == 0)) grid_dependency_wait();
    grid_launch_dependents();
    if (threadIdx.x == 0) WTRACE(0);

    if (warp == 0 || (warp >= 2 && warp < 2 + NXP)) {
        if (lane == 0) {
            // ---------------- producers: warp 0 brings dy, warp 2 + j the x boxes j, j + 4, ... of every stage
            const bool is_dy = warp == 0;
            const int xp = warp - 2;
            // output channels k0+64.. of this tile do not exist when K - k0 <= 64: their accumulator rows are never
            // stored, so that half of the A tile is not loaded at all (the MMA reads stale shared memory there)
            const bool second = p.K - k0 > 64;
            uint32_t my_bytes;
            if (is_dy) my_bytes = second ? a_bytes : 8192u;
            else my_bytes = (uint32_t)((n_x - xp + 3) / 4) * 8192u;
            int q = pix_beg % p.Qd, t = pix_beg / p.Qd, pp = t % p.Pd, n = t / p.Pd;   // first pixel of the stage
            // a stage advances 64 pixels = dn images + dp rows + dq columns: carried without divisions in the loop
            const int dn = 64 / (p.Pd * p.Qd), rem64 = 64 - dn * p.Pd * p.Qd, dp = rem64 / p.Qd, dq = rem64 - dp * p.Qd;
            // this warp's x boxes (at most two per stage: tpc * BN/64 <= 8 boxes over four warps): tap and channel block of each
            int n_mine = 0, box_dst[2] = {0, 0}, box_c[2] = {0, 0};
            uint16_t box_sw[2] = {0, 0}, box_sh[2] = {0, 0};
            if (!is_dy)
                for (int j = xp; j < n_x && n_mine < 2; j += 4, ++n_mine) {
                    const int tt = j / (int)nb_b, nb = j - tt * (int)nb_b;
                    const int r = (tap0 + tt) / p.S;
                    box_dst[n_mine] = j * 8192; box_c[n_mine] = c0 + nb * 64;
                    box_sh[n_mine] = (uint16_t)r; box_sw[n_mine] = (uint16_t)((tap0 + tt) - r * p.S);
                }
            int s = 0, ph = 0, issued = 0;
            grid_dependency_wait();
            for (int it = 0; it < iters; ++it) {
                if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1, abort_flag, p.status, 4)) break;
                const uint32_t bar = smem_u32(&ctl->full[s]);
                const uint32_t a_dst = data_base + (uint32_t)s * stage_bytes, b_dst = a_dst + a_bytes;
                mbar_arrive_expect_tx(bar, my_bytes);
                if (is_dy) {
                    const int pix = pix_beg + it * 64;
                    tma_load_2d(a_dst, &tmDy, bar, k0, pix);
                    if (second) tma_load_2d(a_dst + 8192u, &tmDy, bar, k0 + 64, pix);
                } else {
                    const int w = q * p.stride + p.lo_w, h = pp * p.stride + p.lo_h;
                    if (p.x_tiled) {
                        const int pix = pix_beg + it * 64;
                        tma_load_2d(b_dst + (uint32_t)box_dst[0], &tmX, bar, box_c[0], pix);
                        if (n_mine > 1) tma_load_2d(b_dst + (uint32_t)box_dst[1], &tmX, bar, box_c[1], pix);
                    } else {
                        tma_load_im2col_4d(b_dst + (uint32_t)box_dst[0], &tmX, bar, box_c[0], w, h, n, box_sw[0], box_sh[0]);
                        if (n_mine > 1) tma_load_im2col_4d(b_dst + (uint32_t)box_dst[1], &tmX, bar, box_c[1], w, h, n, box_sw[1], box_sh[1]);
                    }
                    q += dq; pp += dp; n += dn;                       // the next stage starts 64 pixels further on
                    if (q >= p.Qd) { q -= p.Qd; ++pp; }
                    if (pp >= p.Pd) { pp -= p.Pd; ++n; }
                }
                issued = it + 1;
                if (++s == p.stages) { s = 0; ph ^= 1; }
            }
            if (*abort_flag && is_dy) {
                for (int it = max(0, issued - p.stages); it < issued; ++it) {
                    const int s2 = it % p.stages, ph2 = (it / p.stages) & 1;
                    const uint64_t t0 = globaltimer_ns();
                    while (!mbar_try_wait(smem_u32(&ctl->full[s2]), ph2) && globaltimer_ns() - t0 < 20000000ull) {}
                }
            }
        }
        __syncwarp();
    }
    if (warp == 1 || (warp >= 6 && issuer < NI)) {
        // ---------------- MMA issuer `issuer`: the warp walks the loop in lockstep, lane 0 issues
        const uint32_t leader = lane == 0 ? 1u : 0u;
        const uint32_t idesc = make_idesc_bf16(128, p.BN, 1, 1);
        bool ok = true;
        int s = 0, ph = 0;
        for (int it = 0; it < iters && ok; ++it) {
            ok = mbar_wait(smem_u32(&ctl->full[s]), ph, abort_flag, p.status, 5);
            if (!ok) break;
            if (it == 0 && warp == 1) WTRACE(1);
            tc_fence_after();
            const int rem = pix_end - (pix_beg + it * 64);
            const int ksteps = rem >= 64 ? 4 : (rem + 15) / 16;
            const uint32_t a_src = data_base + (uint32_t)s * stage_bytes, b_src = a_src + a_bytes;
            const uint64_t ad0 = make_desc(a_src, 8192u, 1024u);
            const uint32_t acc = it != 0 ? 1u : 0u;
            for (int tt = issuer; tt < ntap; tt += NI) {
                const uint64_t bd0 = make_desc(b_src + (uint32_t)tt * b_bytes, 8192u, 1024u);
                const uint32_t d_tmem = tmem_base + (uint32_t)(tt * p.BN);
                if (ksteps == 4) {
                    umma_bf16_lead(d_tmem, ad0, bd0, idesc, acc, leader);
#pragma unroll
                    for (int k = 1; k < 4; ++k) umma_bf16_lead(d_tmem, ad0 + 128ull * k, bd0 + 128ull * k, idesc, 1u, leader);
                } else {
                    for (int k = 0; k < ksteps; ++k) umma_bf16_lead(d_tmem, ad0 + 128ull * k, bd0 + 128ull * k, idesc, k ? 1u : acc, leader);
                }
            }
            umma_commit_lead(smem_u32(&ctl->empty[s]), leader);
            if (++s == p.stages) { s = 0; ph ^= 1; }
        }
        if (ok) umma_commit_lead(smem_u32(&ctl->accum), leader);
        if (warp == 1) WTRACE(2);
    }
    wgrad_finish(p, tmP, ctl, data_base, tmem_base, ntap, tap0, k0, c0, split, iters, (uint32_t)p.stages * stage_bytes, ntap, p.BN);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// Row-block form of the weight gradient for stride-1 filters with several taps and at most 64 input channels. A stage is
// one unit = `nr` output rows of one image: dy as a box of nr rows x Wp columns (the columns past Q and the rows past P
// are zero-filled by the TMA unit) and x as the halo box of nr + R - 1 rows x Wp columns starting at (-pad, -pad) of the
// unit, both with one 128-byte swizzle row per pixel. Pixel m = i * Wp + j of the dy box pairs with pixel
// m + r * Wp + s of the x box for tap (r, s), so every tap reads the SAME staged x tile through an operand descriptor
// whose start is shifted by r * Wp + s rows: x crosses the memory system once per unit instead of once per tap. Where
// j + s runs past the row the dy factor is a zero column. Rows past the boxes (up to the 16-pixel step) are zeroed once
// and never written again.
//   The x tile is the M side of the MMA and carries TWO taps: M rows 0..63 are the 64 channel lanes at the first tap's
// shift, rows 64..127 the same lanes at the second tap's shift (the descriptor's 64-element block stride is the
// difference of the shifts). The N side is dy's output channels. An accumulator therefore holds dw^T of a pair of taps:
// lanes = (tap, c), columns = k -- half the MMAs of the one-tap-per-accumulator form, and none of the 128 rows wasted
// when K is small.
__global__ void __launch_bounds__(kThreads) conv_wgrad_rows_kernel(const __grid_constant__ CUtensorMap tmDy,
                                                                   const __grid_constant__ CUtensorMap tmX,
                                                                   const __grid_constant__ CUtensorMap tmP, const WgradP p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Ctl *ctl = reinterpret_cast<Ctl *>(smem_raw);
    const uint32_t smem_base = smem_u32(smem_raw);
    const uint32_t data_base = (smem_base + (uint32_t)sizeof(Ctl) + 1023u) & ~1023u;
    const uint32_t nb_b = (uint32_t)((p.BN + 63) / 64);
    const uint32_t a_bytes = (uint32_t)p.nb_a * p.a_box;
    const uint32_t stage_bytes = a_bytes + nb_b * p.b_box;
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int bx = blockIdx.x;
    const int n_tile = bx % p.n_tiles; bx /= p.n_tiles;
    const int m_tile = bx % p.m_tiles; bx /= p.m_tiles;
    const int tap0 = bx * p.tpc;
    const int ntap = min(p.tpc, p.taps - tap0);
    const int split = blockIdx.y;
    const int k0 = m_tile * 128, c0 = n_tile * p.BN;
    const int u_beg = split * p.units_per_split;
    const int u_end = min(p.units, u_beg + p.units_per_split);
    const int iters = u_end > u_beg ? u_end - u_beg : 0;
    const int n_acc = (ntap + 1) / 2;                                 // accumulators: one per pair of taps
    const int NI = n_acc < 4 ? n_acc : 4;                             // MMA issuer warps in use: pairs i, i + NI, ...

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 2u);                   // the dy producer and the x producer
            mbar_init(smem_u32(&ctl->empty[s]), (uint32_t)NI);
        }
        mbar_init(smem_u32(&ctl->accum), (uint32_t)NI);
        ctl->abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmDy);
        prefetch_tmap(&tmX);
    }
    // the ring starts as zeros: the rows between the end of a box and the end of the last 16-pixel step are read by the
    // MMAs (times zero) and must be finite
    for (uint32_t off = threadIdx.x * 16u; off < (uint32_t)p.stages * stage_bytes; off += kThreads * 16u)
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(data_base + off), "r"(0u) : "memory");
    fence_proxy_async();
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int issuer = warp == 1 ? 0 : warp - 5;                      // warps 6, 7, 8 -> issuers 1, 2, 3
    // nothing above touches global memory; the producer threads wait after their set-up
    if (!((warp == 0 || warp == 2) && lane == 0)) grid_dependency_wait();
    grid_launch_dependents();
    if (threadIdx.x == 0) WTRACE(0);

    if (warp == 0 || warp == 2) {
        if (lane == 0) {
            // ---------------- producers: warp 0 brings the dy boxes of every unit, warp 2 the x halo boxes
            const bool is_dy = warp == 0;
            const int n_dy = p.nb_a;
            const uint32_t my_bytes = is_dy ? (uint32_t)(n_dy * p.nr * p.Wp) * 128u
                                            : nb_b * (uint32_t)((p.nr + p.lo_span) * p.Wp) * 128u;
            int n = u_beg / p.RB, rb = u_beg - n * p.RB;
            int s = 0, ph = 0, issued = 0;
            grid_dependency_wait();
            for (int it = 0; it < iters; ++it) {
                if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1, abort_flag, p.status, 4)) break;
                const uint32_t bar = smem_u32(&ctl->full[s]);
                const uint32_t a_dst = data_base + (uint32_t)s * stage_bytes, b_dst = a_dst + a_bytes;
                mbar_arrive_expect_tx(bar, my_bytes);
                const int p0 = rb * p.nr;
                if (is_dy) {
                    for (int b = 0; b < n_dy; ++b) tma_load_4d(a_dst + (uint32_t)b * p.a_box, &tmDy, bar, b * 64, 0, p0, n);
                } else {
                    for (uint32_t b = 0; b < nb_b; ++b)
                        tma_load_4d(b_dst + b * p.b_box, &tmX, bar, c0 + (int)b * 64, p.lo_w, p0 + p.lo_h, n);
                }
                if (++rb == p.RB) { rb = 0; ++n; }
                issued = it + 1;
                if (++s == p.stages) { s = 0; ph ^= 1; }
            }
            if (*abort_flag) {
                for (int it = max(0, issued - p.stages); it < issued; ++it) {
                    const int s2 = it % p.stages, ph2 = (it / p.stages) & 1;
                    const uint64_t t0 = globaltimer_ns();
                    while (!mbar_try_wait(smem_u32(&ctl->full[s2]), ph2) && globaltimer_ns() - t0 < 20000000ull) {}
                }
            }
        }
        __syncwarp();
    }
    if (warp == 1 || (warp >= 6 && issuer < NI)) {
        // ---------------- MMA issuer `issuer`: the warp walks the loop in lockstep, lane 0 issues
        const uint32_t leader = lane == 0 ? 1u : 0u;
        const uint32_t idesc = make_idesc_bf16(128, p.acc_cols, 1, 1);
        // this issuer's pairs (at most four: 16 accumulators of 32 columns fill the tensor memory): byte offset of the
        // first tap's rows in the x tile and the distance to the second tap's rows
        uint32_t tap_shift[4] = {0u, 0u, 0u, 0u}, tap_lbo[4] = {128u, 128u, 128u, 128u};
        int n_mine = 0;
        for (int a = issuer; a < n_acc && n_mine < 4; a += NI, ++n_mine) {
            const int t0 = tap0 + 2 * a, r0 = t0 / p.S, sh0 = r0 * p.Wp + (t0 - r0 * p.S);
            int sh1 = sh0 + 1;                                        // an odd last tap: the upper 64 lanes are not stored
            if (2 * a + 1 < ntap) {
                const int r1 = (t0 + 1) / p.S;
                sh1 = r1 * p.Wp + (t0 + 1 - r1 * p.S);
            }
            tap_shift[n_mine] = (uint32_t)sh0 * 128u;
            tap_lbo[n_mine] = (uint32_t)(sh1 - sh0) * 128u;
        }
        bool ok = true;
        int s = 0, ph = 0;
        for (int it = 0; it < iters && ok; ++it) {
            ok = mbar_wait(smem_u32(&ctl->full[s]), ph, abort_flag, p.status, 5);
            if (!ok) break;
            if (it == 0 && warp == 1) WTRACE(1);
            tc_fence_after();
            const uint32_t a_src = data_base + (uint32_t)s * stage_bytes, b_src = a_src + a_bytes;
            const uint64_t dyd = make_desc(a_src, p.a_box, 1024u);
            const uint32_t acc = it != 0 ? 1u : 0u;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (j >= n_mine) break;
                const uint64_t xd = make_desc(b_src + tap_shift[j], tap_lbo[j], 1024u);
                const uint32_t d_tmem = tmem_base + (uint32_t)((issuer + j * NI) * p.acc_cols);
                umma_bf16_lead(d_tmem, xd, dyd, idesc, acc, leader);
                for (int k = 1; k < p.ksteps; ++k) umma_bf16_lead(d_tmem, xd + 128ull * k, dyd + 128ull * k, idesc, 1u, leader);
            }
            umma_commit_lead(smem_u32(&ctl->empty[s]), leader);
            if (++s == p.stages) { s = 0; ph ^= 1; }
        }
        if (ok) umma_commit_lead(smem_u32(&ctl->accum), leader);
        if (warp == 1) WTRACE(2);
    }
    wgrad_finish(p, tmP, ctl, data_base, tmem_base, ntap, tap0, k0, c0, split, iters, (uint32_t)p.stages * stage_bytes, n_acc, p.acc_cols);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ------------------------------------------------------------------------------------------ few-channel stride-2 stem
// A stride-2 convolution over very few input channels (the 7x7 / 3-channel network stem) is rewritten as a stride-1
// convolution over a space-to-depth copy of the input: xs[n][i][j + pl][(a,b,c)] = x[n][2i+a][2j+b][c], 16 bf16 per pixel,
// with pl zero columns on the left and V-1-pl on the right. Consecutive pixels of a row are contiguous, so the V
// horizontal taps x 16 lanes of one output position are ONE run of 64 elements: the tensor map below gives every output
// column its own 128-byte row (overlapping windows, 32-byte stride), and the conv becomes U vertical taps of 64
// "channels" each -- full swizzle rows for TMA and UMMA instead of 49 taps of 3 channels.
//   h = 2p - pad + r = 2(p - pl) + t,  t = r + off,  off = 2*pl - pad,  u = t / 2, a = t % 2   (same for columns)
struct StemPlan {
    int ok;
    int pl, off, U, V, Hs, Ws, Wp, P, Q;
    size_t xs_bytes, w2_elems;     // padded space-to-depth input; weights / weight gradient as [K][U][64]
};

StemPlan stem_plan(const pt_conv_desc *d)
{
    StemPlan s;
    memset(&s, 0, sizeof(s));
    if (d->stride != 2 || d->C > 4 || (d->H & 1) || (d->W & 1) || d->R != d->S || d->ldx != 8) return s;
    s.pl = (d->pad + 1) / 2;
    s.off = 2 * s.pl - d->pad;
    s.U = (d->R - 1 + s.off) / 2 + 1;
    s.V = s.U;
    if (s.V > 4) return s;
    s.Hs = d->H / 2; s.Ws = d->W / 2;
    s.Wp = s.Ws + 3;                        // every window is 4 pixels wide whatever V is: pl zero columns left, 3 - pl right
    s.P = pt_out_dim(d->H, d->R, 2, d->pad);
    s.Q = pt_out_dim(d->W, d->S, 2, d->pad);
    if (s.Q > s.Ws || s.P > s.Hs + s.pl) return s;
    s.xs_bytes = pt_align_up((size_t)d->N * s.Hs * s.Wp * 32, 1024);
    s.w2_elems = (size_t)d->K * s.U * 64;
    s.ok = 1;
    return s;
}

// CT = channel count as a compile-time constant (1..4): the 16 output lanes are then plain registers
template <int CT>
__global__ void __launch_bounds__(256) stem_s2d_x_kernel_t(const __nv_bfloat16 *__restrict__ x, __nv_bfloat16 *__restrict__ xs, int N, int H,
                                                           int W, int Hs, int Ws, int Wp, int pl)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t total = (size_t)N * Hs * Wp;
    if (idx >= total) return;
    const int jp = (int)(idx % Wp);
    const size_t t = idx / Wp;
    const int i = (int)(t % Hs), n = (int)(t / Hs);
    __align__(16) unsigned short o[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) o[e] = 0;
    const int j = jp - pl;
    if (j >= 0 && j < Ws) {
        uint4 px[4];
#pragma unroll
        for (int ab = 0; ab < 4; ++ab)          // the four loads go out together
            px[ab] = __ldg(reinterpret_cast<const uint4 *>(x + ((size_t)(n * H + 2 * i + (ab >> 1)) * W + 2 * j + (ab & 1)) * 8));
#pragma unroll
        for (int ab = 0; ab < 4; ++ab) {
            const unsigned short *pe = reinterpret_cast<const unsigned short *>(&px[ab]);
#pragma unroll
            for (int c = 0; c < CT; ++c) o[ab * CT + c] = pe[c];
        }
    }
    uint4 *dst = reinterpret_cast<uint4 *>(xs + idx * 16);
    dst[0] = *reinterpret_cast<uint4 *>(&o[0]);
    dst[1] = *reinterpret_cast<uint4 *>(&o[8]);
}

void stem_s2d_x_kernel_launch(unsigned blocks, cudaStream_t st, const __nv_bfloat16 *x, __nv_bfloat16 *xs, int N, int H, int W, int C,
                              int Hs, int Ws, int Wp, int pl)
{
    switch (C) {
    case 1: stem_s2d_x_kernel_t<1><<<blocks, 256, 0, st>>>(x, xs, N, H, W, Hs, Ws, Wp, pl); break;
    case 2: stem_s2d_x_kernel_t<2><<<blocks, 256, 0, st>>>(x, xs, N, H, W, Hs, Ws, Wp, pl); break;
    case 3: stem_s2d_x_kernel_t<3><<<blocks, 256, 0, st>>>(x, xs, N, H, W, Hs, Ws, Wp, pl); break;
    default: stem_s2d_x_kernel_t<4><<<blocks, 256, 0, st>>>(x, xs, N, H, W, Hs, Ws, Wp, pl); break;
    }
}

// w2[k][u][v*16 + (a*2+b)*C + c] = w[k][2u+a-off][2v+b-off][c]  (0 where the tap falls outside the filter)
__global__ void stem_s2d_w_kernel(const __nv_bfloat16 *__restrict__ w, __nv_bfloat16 *__restrict__ w2, int K, int R, int S, int C,
                                  int ldw, int U, int V, int off)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= K * U * 64) return;
    const int l = idx & 63, u = (idx >> 6) % U, k = (idx >> 6) / U;
    const int v = l >> 4, e = l & 15;
    float val = 0.f;
    if (v < V && e < 4 * C) {
        const int ab = e / C, c = e - ab * C, a = ab >> 1, b = ab & 1;
        const int r = 2 * u + a - off, s = 2 * v + b - off;
        if (r >= 0 && r < R && s >= 0 && s < S) val = __bfloat162float(w[((size_t)(k * R + r) * S + s) * ldw + c]);
    }
    w2[idx] = __float2bfloat16_rn(val);
}

// dw[k][r][s][c] = dw2[k][u][v*16 + (a*2+b)*C + c] with (u,a) from r + off and (v,b) from s + off
__global__ void stem_dw_back_kernel(const float *__restrict__ dw2, float *__restrict__ dw, int K, int R, int S, int C, int U, int off)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= K * R * S * C) return;
    const int c = idx % C;
    int t = idx / C;
    const int s = t % S; t /= S;
    const int r = t % R, k = t / R;
    const int tr = r + off, ts = s + off;
    dw[idx] = dw2[((size_t)k * U + (tr >> 1)) * 64 + (ts >> 1) * 16 + ((tr & 1) * 2 + (ts & 1)) * C + c];
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                   const int *, const int *, cuuint32_t, cuuint32_t, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 tensor (C, W, H, N) with channel pitch ld: im2col map loading `pixels` x 64 channels.
bool make_im2col_map(const pt_ctx *c, CUtensorMap *tm, const void *base, int C, int W, int H, int N, int ld, int lo_w, int lo_h,
                     int up_w, int up_h, int stride, int pixels, int row_pixels = 0)
{
    if (!c->encode_im2col) return false;
    if (lo_w < -128 || lo_h < -128 || up_w < -128 || up_h < -128 || lo_w > 127 || lo_h > 127 || up_w > 127 || up_h > 127) return false;
    const int rowp = row_pixels ? row_pixels : W;        // pixels between two image rows in memory (>= W)
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
    cuuint64_t strides[3] = {(cuuint64_t)ld * 2, (cuuint64_t)rowp * ld * 2, (cuuint64_t)H * rowp * ld * 2};
    int lo[2] = {lo_w, lo_h}, up[2] = {up_w, up_h};
    cuuint32_t estr[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
    CUresult r = ((EncodeIm2colFn)c->encode_im2col)(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, lo,
                                                    up, (cuuint32_t)kKC, (cuuint32_t)pixels, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return map_ok(r, __LINE__);
}

// bf16 activations as a plain 2-D tensor (channels, pixels) with row pitch ld: box 64 channels x `pixels`.
bool make_act2d_map(const pt_ctx *c, CUtensorMap *tm, const void *base, int C, long long npix, int ld, int pixels)
{
    if (!c->encode_tiled) return false;
    cuuint64_t dims[2] = {(cuuint64_t)C, (cuuint64_t)npix};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)kKC, (cuuint32_t)pixels}, estr[2] = {1, 1};
    CUresult r = ((CUresult(*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                               const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill))c->encode_tiled)(
        tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return map_ok(r, __LINE__);
}

// bf16 weight shadow as (C, R*S, K) with row pitch ldw: box (64, 1, box_k).
bool make_weight_map(const pt_ctx *c, CUtensorMap *tm, const void *base, int C, int RS, int K, int ldw, int box_k)
{
    if (!c->encode_tiled) return false;
    cuuint64_t dims[3] = {(cuuint64_t)C, (cuuint64_t)RS, (cuuint64_t)K};
    cuuint64_t strides[2] = {(cuuint64_t)ldw * 2, (cuuint64_t)RS * ldw * 2};
    cuuint32_t box[3] = {(cuuint32_t)kKC, 1, (cuuint32_t)box_k};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ((EncodeTiledFn)c->encode_tiled)(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box,
                                                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return map_ok(r, __LINE__);
}

// Tile width along the output channels. One tile: the ragged count rounded up to 16. Several tiles: a multiple of
// 64 (the TMA-store chunk) chosen to waste the fewest padded columns.
int tile_n(int cols, int *n_tiles, int m_tiles = 1 << 30, int sms = 0)
{
    int best = 256;
    if (cols <= 256) {
        *n_tiles = 1;
        best = pt_ceil_div(cols, 16) * 16;
    } else {
        int best_pad = 1 << 30;
        for (int bn = 256; bn >= 128; bn -= 64) {
            int pad = pt_ceil_div(cols, bn) * bn;
            if (pad < best_pad) { best_pad = pad; best = bn; }
        }
        *n_tiles = pt_ceil_div(cols, best);
    }
    if (sms <= 0 || m_tiles >= sms) return best;
    // Few pixel tiles (the 7x7 maps): a CTA's time is what it streams per reduction stage -- the 16 KB activation tile plus
    // bn x 128 bytes of weights -- times the waves of tiles. Narrower channel tiles put more SMs to work and cut the weight
    // bytes per CTA; the activation tile is then read by more CTAs, from L2. Taken when the estimate drops by 10 % or more.
    long long cost0 = (long long)pt_ceil_div(m_tiles * *n_tiles, sms) * (16 * 1024 + (long long)pt_ceil_div(best, 64) * 8192);
    for (int bn = 192; bn >= 64; bn -= 64) {
        if (bn >= best) continue;
        const int nt = pt_ceil_div(cols, bn);
        const long long cost = (long long)pt_ceil_div(m_tiles * nt, sms) * (16 * 1024 + (long long)bn * 128);
        if (cost * 10 <= cost0 * 9) { cost0 = cost; best = bn; *n_tiles = nt; }
    }
    return best;
}

int pow2_cols(int bn)
{
    int c = 32;
    while (c < bn) c <<= 1;
    return c;
}

// Pipeline depth for a kernel that owns the SM: as many stages as fit beside `reserved` bytes, at most kMaxStages.
// The GEMM-form kernel may take all but 1 KB of the 227 KB a CTA can have (one more stage for the wide 1x1 layers).
constexpr size_t kGemmSmemCap = (size_t)226 * 1024;
int pick_stages(size_t stage_bytes, int iters, size_t reserved, size_t *smem, size_t cap = (size_t)220 * 1024)
{
    int st = (int)((cap - 2048 - reserved) / stage_bytes);
    if (st > kMaxStages) st = kMaxStages;
    if (st > iters && iters >= 2) st = iters;
    if (st < 2) st = 2;
    *smem = 2048 + reserved + (size_t)st * stage_bytes;
    return st;
}

// bf16 output viewed as (channels, pixels) with row pitch ld: box 64 channels x 32 pixels, 128-byte swizzle.
// Channel extent of an output tensor map: the channel count rounded up to a whole 32-byte sector where the pitch has room
// for it (the pad lanes there receive zeros). A row whose last sector is only partly written costs a read-modify-write in
// the memory system: measured 35 us against 20 us for 56x56x209..216 channels at pitch 224.
int store_cols(int cols, int ld)
{
    const int up = pt_ceil_div(cols, 16) * 16;
    return up <= ld ? up : cols;
}

bool make_out_map(const pt_ctx *c, CUtensorMap *tm, void *base, int cols, int rows, int ld)
{
    cuuint64_t dims[2] = {(cuuint64_t)store_cols(cols, ld), (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64, 32}, estr[2] = {1, 1};
    CUresult r = ((EncodeTiledFn)c->encode_tiled)(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
                                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return map_ok(r, __LINE__);
}

template <bool B_MN>
pt_status launch_gemm(pt_ctx *c, const CUtensorMap &tmA, const CUtensorMap &tmB, GemmP &p, cudaStream_t st)
{
    CUtensorMap tmC;
    memset(&tmC, 0, sizeof(tmC));
    p.tma_store = (!p.out_f32 && p.o_step == 1 && p.zero_mask == 0) ? 1 : 0;
    if (p.tma_store && !make_out_map(c, &tmC, p.out, p.n_cols, p.M_total, p.ld_out)) return PT_ERR_CUDA;
    const size_t a_bytes = kBM * kKC * 2;
    const size_t b_bytes = B_MN ? (size_t)pt_ceil_div(p.BN, 64) * 8192 : pt_align_up((size_t)p.BN * 128, 1024);
    size_t smem = 0;
    p.m_tiles = pt_ceil_div(p.M_total, kBM);
    const int total_tiles = p.m_tiles * p.n_tiles;
    const int per_cta = pt_ceil_div(total_tiles, c->sm_count);
    // accumulator buffers = epilogue groups: three when 3 * BN fits the 512 TMEM columns, else two; narrow layers whose
    // CTAs get a single tile need no more than that
    p.epi_groups = 3 * p.BN <= 512 ? 3 : 2;
    if (per_cta < p.epi_groups) p.epi_groups = per_cta;           // a single tile per CTA: one group, and its staging goes to the ring
    // Small weights (one channel tile, all taps x chunks within 64 KB) stay resident: the ring then carries A tiles only and
    // holds more of them, which is what an activation-bound layer needs to cover the memory latency.
    const size_t w_all = (size_t)p.taps * p.k_chunks * b_bytes;
    p.resident = (p.n_tiles == 1 && w_all <= 64 * 1024 && per_cta >= 2) ? 1 : 0;
    p.n_issuers = 1; p.acc_per = 1;
    if (p.resident && per_cta >= 4 && 2 * p.BN <= 512) {
        // narrow tiles are bound by what one thread can issue: two issuer warps, two epilogue groups
        p.n_issuers = 2;
        p.epi_groups = 2;
        p.acc_per = 4 * p.BN <= 512 ? 2 : 1;
    }
    // one tile per CTA and streamed weights: the output is staged in the ring (all of its stages have been consumed when the
    // accumulator is complete), which leaves room for one more stage
    p.alias_staging = (per_cta == 1 && !p.resident) ? 1 : 0;
    // statistics mode: the epilogue warps' accumulators sit at the end of the shared memory (taken from the ring's room)
    p.stats_warp = pt_ceil_div(p.BN, 64) * (int)kStatsChunkBytes;
    const size_t st_smem = c->stats_mode ? (size_t)4 * p.epi_groups * p.stats_warp : 0;     // (the group count can only shrink below)
    size_t staging2 = p.alias_staging ? 0 : (size_t)p.epi_groups * 4 * kSlabs * 4096;
    if (p.resident) p.stages = pick_stages(a_bytes, p.taps * p.k_chunks * per_cta, staging2 + w_all + st_smem, &smem, kGemmSmemCap);
    else {
        p.stages = pick_stages(a_bytes + b_bytes, p.taps * p.k_chunks * per_cta, staging2 + st_smem, &smem, kGemmSmemCap);
        if (p.stages < 4 && p.epi_groups == 3 && p.taps * p.k_chunks * per_cta >= 4) {
            // a third epilogue group costs 32 KB of staging: with wide weight tiles that is the fourth pipeline stage
            p.epi_groups = 2;
            staging2 = (size_t)p.epi_groups * 4 * kSlabs * 4096;
            p.stages = pick_stages(a_bytes + b_bytes, p.taps * p.k_chunks * per_cta, staging2 + st_smem, &smem, kGemmSmemCap);
        }
    }
    p.stats_off = (int)(smem - st_smem);
    if (p.n_issuers == 2) {
        p.stages = p.stages / 2 * 2;
        if (p.stages < 2) { p.n_issuers = 1; p.acc_per = 1; p.stages = 2; }
    }
    p.tmem_cols = pow2_cols((p.n_issuers == 2 ? 2 * p.acc_per : p.epi_groups) * p.BN);
    // the statistics variant exists for the forward kernel only
    void (*kernel)(CUtensorMap, CUtensorMap, CUtensorMap, GemmP) =
        (!B_MN && c->stats_mode) ? conv_gemm_kernel<false, true> : conv_gemm_kernel<B_MN, false>;
    const int kid = (!B_MN && c->stats_mode) ? 2 : (B_MN ? 1 : 0);
    static bool attr_set[3] = {false, false, false};
    if (!attr_set[kid]) {
        PT_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        attr_set[kid] = true;
    }
    const int grid = total_tiles < c->sm_count ? total_tiles : c->sm_count;
    if (c->stats_mode) {
        if (!p.tma_store) return PT_ERR_UNSUPPORTED;
        c->stats_parts = grid * 4 * p.epi_groups;
        if ((size_t)c->stats_parts * 2 * p.ld_out * sizeof(float) > c->stats_cap) return PT_ERR_WORKSPACE;
        p.stats = c->stats_out;
    }
    if (c->test_skip == 2) { p.test_skip = 1; c->test_skip = 0; }
    PT_CUDA_OK(launch_pdl(kernel, dim3((unsigned)grid), dim3(kGemmThreads), smem, st, tmA, tmB, tmC, p));
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

// Source activations as a tiled 4-D tensor (C, W, H, N): box 64 channels x box_w x box_h x 1 (the halo tile).
// `lanes` = 64 (128-byte rows and swizzle) or 16 (32-byte rows and swizzle).
// `row_pixels` > 0: pixels between the starts of consecutive rows when that is not W (a padded row).
bool make_halo_in_map(const pt_ctx *c, CUtensorMap *tm, const void *base, int C, int W, int H, int N, int ld, int box_w, int box_h,
                      int lanes = kKC, int row_pixels = 0)
{
    if (!c->encode_tiled || box_w > 256 || box_h > 256) return false;
    const cuuint64_t rp = row_pixels > 0 ? (cuuint64_t)row_pixels : (cuuint64_t)W;
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
    cuuint64_t strides[3] = {(cuuint64_t)ld * 2, rp * ld * 2, (cuuint64_t)H * rp * ld * 2};
    cuuint32_t box[4] = {(cuuint32_t)lanes, (cuuint32_t)box_w, (cuuint32_t)box_h, 1}, estr[4] = {1, 1, 1, 1};
    CUresult r = ((EncodeTiledFn)c->encode_tiled)(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box,
                                                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, lanes == 16 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                                                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return map_ok(r, __LINE__);
}

// One launch of the halo kernel: a stride-1 correlation of `src` with a list of taps, written to a (possibly strided)
// view of the output.
struct HaloSpec {
    const void *src; int Cs, Ws, Hs, lds;            // activations read: channels, width, height, pitch
    int P, Q;                                        // output raster per image (rows, columns)
    int n_taps, span_h, span_w;                      // taps and the extent of their offsets (max offset + 1)
    int lo_h, lo_w;                                  // source coordinate of raster (0,0) at tap offset (0,0)
    int tap_oh[kMaxTaps], tap_ow[kMaxTaps], tap_wt[kMaxTaps];
    int n_cols, ld_out;                              // output channels and pitch
    int oH, oW, o_step, o_h0, o_w0;                  // output view: raster (i, j) -> pixel (i*o_step + o_h0, j*o_step + o_w0) of oH x oW
    int row32, w_taps;                               // 16-lane pixels (32-byte rows); taps per output channel in the weight tensor
    int max_ctas;                                    // > 0: grid limit (launches meant to run side by side share the SMs)
};

template <bool B_MN>
pt_status launch_halo(pt_ctx *c, const pt_conv_desc *d, const HaloSpec &h, const void *w, void *out, cudaStream_t st)
{
    const int Wp = h.Q + h.span_w - 1;
    if (h.n_taps < 1 || h.n_taps > kMaxTaps || Wp > 128 || h.Ws > 250) return PT_ERR_UNSUPPORTED;
    HaloP p;
    memset(&p, 0, sizeof(p));
    p.N = d->N; p.P = h.P; p.Q = h.Q; p.Wp = Wp;
    p.nr = 128 / Wp < h.P ? 128 / Wp : h.P;
    p.row_tiles = pt_ceil_div(h.P, p.nr);
    p.n_cols = h.n_cols;
    p.BN = tile_n(h.n_cols, &p.n_tiles);
    p.c_red = h.Cs; p.k_chunks = pt_ceil_div(h.Cs, kKC); p.taps = h.n_taps;
    p.row32 = h.row32 ? 1 : 0;
    const int row_bytes = h.row32 ? 32 : 128;
    if (h.row32 && (B_MN || h.Cs != 16)) return PT_ERR_UNSUPPORTED;
    p.lo_h = h.lo_h; p.lo_w = h.lo_w;
    for (int t = 0; t < h.n_taps; ++t) {
        p.tap_oh[t] = (unsigned char)h.tap_oh[t]; p.tap_ow[t] = (unsigned char)h.tap_ow[t];
        p.tap_wt[t] = (unsigned short)h.tap_wt[t];
    }
    const int box_h = p.nr + h.span_h - 1;
    if (box_h > 256) return PT_ERR_UNSUPPORTED;
    p.a_box_bytes = box_h * Wp * row_bytes;
    // The M = 128 MMAs of the last tap read up to this many rows; the rows past the box only feed raster positions that
    // are never stored, so consecutive A stages may overlap there (and a tail pad follows the last stage).
    const int need_rows = 128 + (h.span_h - 1) * Wp + h.span_w - 1;
    p.a_alloc = (int)pt_align_up((size_t)p.a_box_bytes, 1024);
    const size_t a_tail = need_rows * row_bytes > p.a_alloc ? pt_align_up((size_t)need_rows * row_bytes - p.a_alloc, 1024) : 0;
    // a K-major weight box brings the output channels that exist rounded up to 16 (the rows past the count are zero-filled
    // by the TMA unit): exactly the columns the output map covers, so the pad lanes it writes are zeros; the MMA may still
    // read up to BN rows, the rest from whatever follows in shared memory: columns that are never stored
    p.b_rows = p.BN < h.n_cols ? p.BN : pt_ceil_div(h.n_cols, 16) * 16;
    if (p.b_rows > p.BN) p.b_rows = p.BN;
    const size_t b_bytes = B_MN ? (size_t)pt_ceil_div(p.BN, 64) * 8192 : (size_t)p.b_rows * row_bytes;
    p.b_slot = (int)b_bytes;
    // epilogue staging: one slab of the tile's raster rows x 128 bytes per group (direct-store launches use none)
    p.staging = d->out_f32 ? 0 : (int)pt_align_up((size_t)(p.nr * Wp < 128 ? p.nr * Wp : 128) * 128, 1024);
    p.stats_warp = pt_ceil_div(p.BN, 64) * (int)kStatsChunkBytes;
    const size_t st_smem = c->stats_mode ? (size_t)8 * p.stats_warp : 0;        // statistics accumulators of the eight epilogue warps
    const size_t budget = 227 * 1024 - 2048 - 2 * (size_t)p.staging - a_tail - st_smem;
    const size_t w_all = (size_t)h.n_taps * p.k_chunks * b_bytes;
    p.resident = (p.n_tiles == 1 && w_all + 2 * (size_t)p.a_alloc <= budget) ? 1 : 0;
    size_t left = budget - (p.resident ? w_all : 0);
    bool two_pipes = false;
    if (!p.resident) {
        // ring: at least two A stages, the rest for weight stages (at least 3)
        p.stages_a = 2;
        if (left < 2 * (size_t)p.a_alloc + 3 * b_bytes) return PT_ERR_UNSUPPORTED;
        size_t sb = (left - 2 * (size_t)p.a_alloc) / b_bytes;
        p.stages_b = sb > kMaxStages ? kMaxStages : (int)sb;
        // two pipelines (one per tile parity) when each can have three weight stages and the CTAs get several tiles
        // (a launch that shares the SMs with others has fewer CTAs, each with more tiles)
        const int ctas_avail = (h.max_ctas > 0 && h.max_ctas < c->sm_count) ? h.max_ctas : c->sm_count;
        two_pipes = p.stages_b >= 6 && pt_ceil_div(p.N * p.row_tiles * p.n_tiles, ctas_avail) >= 2;
        if (two_pipes) p.stages_b = p.stages_b / 2 * 2;
        // Two pipelines on one weight stream (a single channel tile): every chunk of both tiles should have an activation stage
        // of its own -- a chunk that waits for the previous chunk's MMAs to free its stage exposes a DRAM round trip per tile
        // (28x28, 69 -> 93 channels, MN-major weights: two stages against four, 30 -> 22 us) -- as long as four weight stages
        // remain for the shared stream.
        const int want_a = 2 * p.k_chunks > 4 ? 4 : 2 * p.k_chunks;
        if (two_pipes && p.n_tiles == 1 && left >= (size_t)want_a * p.a_alloc + 4 * b_bytes) {
            const size_t sb2 = (left - (size_t)want_a * p.a_alloc) / b_bytes;
            if ((size_t)p.stages_b > sb2) p.stages_b = (int)sb2;
        }
        left -= (size_t)p.stages_b * b_bytes;
        int sa = (int)(left / p.a_alloc);
        p.stages_a = sa > 4 ? 4 : sa;
    } else {
        int sa = (int)(left / p.a_alloc);
        p.stages_a = sa > 4 ? 4 : sa;
        p.stages_b = 1;
    }
    if (p.stages_a < 2) return PT_ERR_UNSUPPORTED;
    // issuer warps: several only with resident weights; each needs an A stage of its own and an accumulator buffer
    p.n_issuers = 1;
    p.acc_per = 2;
    if (p.resident) {
        p.n_issuers = (p.stages_a >= 4 && 4 * p.BN <= 512) ? 4 : 2;
        p.acc_per = p.n_issuers * 2 * p.BN <= 512 ? 2 : 1;
    } else if (two_pipes) {
        p.n_issuers = 2;
        p.acc_per = 4 * p.BN <= 512 ? 2 : 1;
        p.shared_b = p.n_tiles == 1 ? 1 : 0;          // the tiles of a round then use the same weight columns
    }
    p.stages_a = p.stages_a / p.n_issuers * p.n_issuers;
    p.tmem_cols = pow2_cols(p.n_issuers * p.acc_per * p.BN);
    p.out = out; p.ld_out = h.ld_out; p.out_f32 = d->out_f32;
    p.oH = h.oH; p.oW = h.oW; p.o_step = h.o_step; p.o_h0 = h.o_h0; p.o_w0 = h.o_w0;
    p.tma_store = d->out_f32 ? 0 : 1;
    p.status = c->d_status;
    CUtensorMap tmA, tmB, tmC;
    memset(&tmC, 0, sizeof(tmC));
    if (h.row32) {
        if (!p.resident) return PT_ERR_UNSUPPORTED;
        if (!make_halo_in_map(c, &tmA, h.src, h.Cs, h.Ws, h.Hs, d->N, h.lds, Wp, box_h, 16)) return PT_ERR_CUDA;
        // weights [K][w_taps][16]: one 32-byte row per output channel and tap
        cuuint64_t dims[3] = {16, (cuuint64_t)h.w_taps, (cuuint64_t)h.n_cols};
        cuuint64_t strides[2] = {32, (cuuint64_t)h.w_taps * 32};
        cuuint32_t box[3] = {16, 1, (cuuint32_t)p.b_rows}, estr[3] = {1, 1, 1};
        CUresult r = ((EncodeTiledFn)c->encode_tiled)(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(w), dims, strides, box,
                                                      estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B,
                                                      CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (!map_ok(r, __LINE__)) return PT_ERR_CUDA;
    } else {
        if (!make_halo_in_map(c, &tmA, h.src, h.Cs, h.Ws, h.Hs, d->N, h.lds, Wp, box_h)) return PT_ERR_CUDA;
        if (!make_weight_map(c, &tmB, w, d->C, d->R * d->S, d->K, d->ldw, B_MN ? kKC : p.b_rows)) return PT_ERR_CUDA;
    }
    if (p.tma_store) {
        // the output view as a 4-D tensor (channels, raster columns, raster rows, images); strided when o_step > 1
        const size_t es = 2;
        char *base = (char *)out + ((size_t)h.o_h0 * h.oW + h.o_w0) * h.ld_out * es;
        cuuint64_t dims[4] = {(cuuint64_t)store_cols(h.n_cols, h.ld_out), (cuuint64_t)h.Q, (cuuint64_t)h.P, (cuuint64_t)d->N};
        cuuint64_t strides[3] = {(cuuint64_t)h.o_step * h.ld_out * es, (cuuint64_t)h.o_step * h.oW * h.ld_out * es,
                                 (cuuint64_t)h.oH * h.oW * h.ld_out * es};
        cuuint32_t box[4] = {64, (cuuint32_t)Wp, (cuuint32_t)p.nr, 1}, estr[4] = {1, 1, 1, 1};
        CUresult r = ((EncodeTiledFn)c->encode_tiled)(&tmC, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr,
                                                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                      CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (!map_ok(r, __LINE__)) return PT_ERR_CUDA;
    }
    const size_t smem = 2048 + 2 * (size_t)p.staging + (p.resident ? w_all : (size_t)p.stages_b * b_bytes) + (size_t)p.stages_a * p.a_alloc + a_tail +
                        st_smem;
    p.stats_off = (int)(smem - st_smem);
    void (*kernel)(CUtensorMap, CUtensorMap, CUtensorMap, HaloP) =
        (!B_MN && c->stats_mode) ? conv_halo_kernel<false, true> : conv_halo_kernel<B_MN, false>;
    const int kid = (!B_MN && c->stats_mode) ? 2 : (B_MN ? 1 : 0);
    static bool attr_set[3] = {false, false, false};
    if (!attr_set[kid]) {
        PT_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        attr_set[kid] = true;
    }
    const int total_tiles = p.N * p.row_tiles * p.n_tiles;
    int grid = total_tiles < c->sm_count ? total_tiles : c->sm_count;
    if (h.max_ctas > 0 && grid > h.max_ctas) grid = h.max_ctas;
    if (c->stats_mode) {
        if (!p.tma_store || B_MN) return PT_ERR_UNSUPPORTED;
        c->stats_parts = grid * 8;
        if ((size_t)c->stats_parts * 2 * p.ld_out * sizeof(float) > c->stats_cap) return PT_ERR_WORKSPACE;
        p.stats = c->stats_out;
    }
    PT_CUDA_OK(launch_pdl(kernel, dim3((unsigned)grid), dim3(kHaloThreads), smem, st, tmA, tmB, tmC, p));
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

// Stride-1 RxS forward (flip = false, src = x) or data gradient (flip = true, src = dy, padding R-1-pad).
void halo_spec_stride1(const pt_conv_desc *d, HaloSpec *h, const void *src, int Cs, int Ws, int Hs, int lds, int n_cols, int P, int Q,
                       int ld_out, int pad_h, int pad_w, bool flip)
{
    memset(h, 0, sizeof(*h));
    h->src = src; h->Cs = Cs; h->Ws = Ws; h->Hs = Hs; h->lds = lds;
    h->P = P; h->Q = Q; h->n_taps = d->R * d->S; h->span_h = d->R; h->span_w = d->S;
    h->lo_h = -pad_h; h->lo_w = -pad_w;
    for (int t = 0; t < h->n_taps && t < kMaxTaps; ++t) {
        h->tap_oh[t] = t / d->S; h->tap_ow[t] = t % d->S;
        h->tap_wt[t] = flip ? h->n_taps - 1 - t : t;
    }
    h->n_cols = n_cols; h->ld_out = ld_out;
    h->oH = P; h->oW = Q; h->o_step = 1; h->o_h0 = 0; h->o_w0 = 0;
}

// A CTA of a split weight gradient holds its tensor memory while it waits for the other splits of its tile. Two such CTAs
// on one SM could block each other's tensor-memory allocation (the second allocation waits for columns the first one
// frees only after a CTA that cannot start has arrived), so a split launch asks for more than half of an SM's shared
// memory: at most one of them per SM, whatever else runs beside it (kernels that wait for nobody always finish).
constexpr size_t kSplitSmemFloor = 116 * 1024;

// Taps handled by one weight-gradient CTA: they share the dy tile and get one TMEM accumulator of BN columns each.
// Bounded by the 512 TMEM columns and by a stage of 16 KB (dy) + taps x BN/64 x 8 KB (x) staying at or below 48 KB, so
// that at least four pipeline stages fit (measured: with two stages the kernel is slower than with one tap per CTA);
// the taps are then dealt out in equal groups.
int wgrad_taps_per_cta(int taps, int bn)
{
    int t = 512 / bn;
    const int by_smem = 4 / pt_ceil_div(bn, 64);
    if (t > by_smem) t = by_smem;
    if (t < 1) t = 1;
    if (t > taps) t = taps;
    const int groups = pt_ceil_div(taps, t);
    return pt_ceil_div(taps, groups);
}

int wgrad_splits(const pt_ctx *c, const pt_conv_desc *d, int P, int Q)
{
    int n_tiles;
    const int bn = tile_n(d->C, &n_tiles);
    const int tpc = wgrad_taps_per_cta(d->R * d->S, bn);
    const int tiles = pt_ceil_div(d->K, 128) * n_tiles * pt_ceil_div(d->R * d->S, tpc);
    const long long npix = (long long)d->N * P * Q;
    const int budget = (c->wgrad_ctas > 0 && c->wgrad_ctas < c->sm_count) ? c->wgrad_ctas : c->sm_count;
    long long s = budget / tiles;                          // at most one CTA per SM, one wave
    const long long max_s = (npix + 255) / 256;          // at least four 64-pixel stages per split
    if (s > max_s) s = max_s;
    if (s < 1) s = 1;
    if (s > 512) s = 512;
    return (int)s;
}

// Plan of the row-block weight gradient (stride-1 filters with at most 64 input channels); ok = 0 where the generic kernel is used.
struct WgRows {
    int ok;
    int bn, n_tiles, m_tiles, tpc, tap_groups, apc, acc_cols;
    int nr, Wp, RB, units, units_per_split, splits, ksteps, nb_a, stages;
    unsigned a_box, b_box;
    size_t stage_bytes, smem;
};

WgRows wgrad_rows_plan(const pt_ctx *c, const pt_conv_desc *d, int P, int Q)
{
    WgRows w;
    memset(&w, 0, sizeof(w));
    const int taps = d->R * d->S;
    if (d->stride != 1 || taps > kMaxTaps) return w;
    // a 1x1 filter has no halo to save, but the orientation (x on the M side, all of dy's channels on the N side: one tile
    // where the generic kernel needs two for K > 128) and the plain tiled loads (no im2col boxes on 96-byte pixel pitches)
    // still pay on large maps (56x56, 59 -> 143: 53 -> 31 us at 49 CTAs); small maps have too few units to split
    if (taps < 2 && P * Q < 784) return w;
    w.Wp = Q + d->S - 1;
    if (w.Wp > 256 || P < 1 || Q < 1) return w;
    // paired form only: the x tile is the M side (two taps x 64 channel lanes), dy's output channels the N side
    w.acc_cols = pt_ceil_div(d->K, 16) * 16;
    if (d->C > 64 || w.acc_cols > 256) return w;
    w.bn = tile_n(d->C, &w.n_tiles);
    w.m_tiles = 1;
    const int pairs = pt_ceil_div(taps, 2);
    int t = 512 / w.acc_cols;
    if (t > 16) t = 16;                                   // four issuer warps x four accumulators
    if (t > pairs) t = pairs;
    w.tap_groups = pt_ceil_div(pairs, t);
    w.apc = pt_ceil_div(pairs, w.tap_groups);
    w.tpc = 2 * w.apc;
    w.tap_groups = pt_ceil_div(taps, w.tpc);
    w.nb_a = pt_ceil_div(w.acc_cols, 64);
    const int nb_b = 1;
    // rows per unit: the least traffic per useful row (dy rows + x halo rows, the last unit of an image padded) times
    // the MMA steps spent per useful pixel, among the sizes that leave at least two stages
    double best = 1e30;
    for (int nr = 1; nr <= P && nr + d->R - 1 <= 256; ++nr) {
        const int ks = pt_ceil_div(nr * w.Wp, 16);
        const size_t a_box = (size_t)ks * 2048;
        const size_t b_box = pt_align_up(((size_t)(d->R - 1) * w.Wp + d->S + (size_t)ks * 16) * 128, 1024);
        const size_t stage = w.nb_a * a_box + nb_b * b_box;
        const int st = (int)((220 * 1024 - 2048) / stage);
        if (st < 2) break;
        const int rb = pt_ceil_div(P, nr);
        const double traffic = (double)(w.nb_a * nr + nb_b * (nr + d->R - 1)) * rb / P;
        const double steps = (double)ks * 16 * rb / ((double)P * w.Wp);
        const double cost = traffic * steps;
        if (cost < best) {
            best = cost;
            w.nr = nr; w.ksteps = ks; w.a_box = (unsigned)a_box; w.b_box = (unsigned)b_box;
            w.stages = st > kMaxStages ? kMaxStages : st;
            w.stage_bytes = stage;
        }
    }
    if (w.nr == 0) return w;
    w.RB = pt_ceil_div(P, w.nr);
    w.units = d->N * w.RB;
    const int tiles = w.m_tiles * w.n_tiles * w.tap_groups;
    const int budget = (c->wgrad_ctas > 0 && c->wgrad_ctas < c->sm_count) ? c->wgrad_ctas : c->sm_count;
    int s = budget / tiles;                                // at most one CTA per SM, one wave
    if (s > w.units / 2) s = w.units / 2;                  // at least two units per split
    if (s < 1) s = 1;
    if (s > 512) s = 512;
    w.units_per_split = pt_ceil_div(w.units, s);
    w.splits = pt_ceil_div(w.units, w.units_per_split);
    if (w.stages > w.units_per_split && w.units_per_split >= 2) w.stages = w.units_per_split;
    w.smem = 2048 + (size_t)w.stages * w.stage_bytes;
    if (w.smem < 2048 + 8 * 2 * 4096) w.smem = 2048 + 8 * 2 * 4096;    // the epilogue's staging slabs reuse the ring
    w.ok = 1;
    return w;
}

// Workspace of the split weight gradient: one padded 128 x BN fp32 tile per (tile, split).
size_t wgrad_partial_bytes(const pt_ctx *c, const pt_conv_desc *d, int P, int Q)
{
    const WgRows wr = wgrad_rows_plan(c, d, P, Q);
    if (wr.ok)
        return wr.splits <= 1 ? 0 : (size_t)wr.tap_groups * wr.apc * wr.splits * 128 * wr.acc_cols * sizeof(float);
    const int s = wgrad_splits(c, d, P, Q);
    if (s <= 1) return 0;
    int n_tiles;
    const int bn = tile_n(d->C, &n_tiles);
    const int tpc = wgrad_taps_per_cta(d->R * d->S, bn);
    return (size_t)n_tiles * pt_ceil_div(d->K, 128) * pt_ceil_div(d->R * d->S, tpc) * tpc * s * 128 * bn * sizeof(float);
}

// The splits' fp32 partial tiles as a 2-D tensor (BN columns, rows): box 32 x 32, 128-byte swizzle.
bool make_partial_map(const pt_ctx *c, CUtensorMap *tm, void *ws, int bn, size_t rows)
{
    if (!c->encode_tiled) return false;
    cuuint64_t dims[2] = {(cuuint64_t)bn, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)bn * 4};
    cuuint32_t box[2] = {32, 32}, estr[2] = {1, 1};
    CUresult r = ((EncodeTiledFn)c->encode_tiled)(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, ws, dims, strides, box, estr,
                                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return map_ok(r, __LINE__);
}

// Launches the weight-gradient kernel for a problem whose x operand is described by `tmX` (64 pixels x 64 channels boxes).
pt_status run_wgrad(pt_ctx *c, const pt_conv_desc *d, int P, int Q, int stride, int lo_h, int lo_w, const CUtensorMap &tmX,
                    const void *dy, float *out, void *ws, size_t ws_bytes, cudaStream_t st, bool x_tiled = false)
{
    WgradP p;
    memset(&p, 0, sizeof(p));
    p.x_tiled = x_tiled ? 1 : 0;
    p.K = d->K; p.C = d->C; p.taps = d->R * d->S; p.S = d->S;
    p.BN = tile_n(d->C, &p.n_tiles);
    p.m_tiles = pt_ceil_div(d->K, 128);
    p.tpc = wgrad_taps_per_cta(p.taps, p.BN);
    p.tap_groups = pt_ceil_div(p.taps, p.tpc);
    p.apc = p.tpc; p.acc_cols = p.BN;
    p.npix = d->N * P * Q;
    p.splits = wgrad_splits(c, d, P, Q);
    p.pix_per_split = pt_ceil_div(pt_ceil_div(p.npix, p.splits), 64) * 64;
    p.Pd = P; p.Qd = Q; p.stride = stride; p.lo_h = lo_h; p.lo_w = lo_w;
    p.tmem_cols = pow2_cols(p.tpc * p.BN);
    p.status = c->d_status;
    const int gx = p.n_tiles * p.m_tiles * p.tap_groups;
    p.out = out;
    CUtensorMap tmP;
    memset(&tmP, 0, sizeof(tmP));
    if (p.splits > 1) {
        const size_t need = (size_t)gx * p.tpc * p.splits * 128 * p.BN * sizeof(float);
        if (!ws || ws_bytes < need) return PT_ERR_WORKSPACE;
        p.partial = (float *)ws;
        // two self-resetting counters per tile from the context's ring (kernels of one stream run in order, and the ring
        // is far larger than the tiles of the few launches that can be in flight)
        if (2 * gx > 8192) return PT_ERR_UNSUPPORTED;
        if (c->sync_next + 2 * gx > 16384) c->sync_next = 0;
        p.sync = c->d_sync + c->sync_next;
        c->sync_next += 2 * gx;
        if (!make_partial_map(c, &tmP, ws, p.BN, (size_t)gx * p.tpc * p.splits * 128)) return PT_ERR_CUDA;
    }
    // A: dy as a 2-D tensor (K channels, N*P*Q pixels), box 64 channels x 64 pixels
    if (!c->encode_tiled) return PT_ERR_CUDA;
    CUtensorMap tmA;
    {
        cuuint64_t dims[2] = {(cuuint64_t)d->K, (cuuint64_t)p.npix};
        cuuint64_t strides[1] = {(cuuint64_t)d->ldy * 2};
        cuuint32_t box[2] = {64, 64}, estr[2] = {1, 1};
        CUresult r = ((EncodeTiledFn)c->encode_tiled)(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(dy), dims, strides, box,
                                                      estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                      CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (!map_ok(r, __LINE__)) return PT_ERR_CUDA;
    }
    size_t smem = 0;
    const size_t stage = 2 * 8192 + (size_t)p.tpc * pt_ceil_div(p.BN, 64) * 8192;
    p.stages = pick_stages(stage, pt_ceil_div(p.pix_per_split, 64), 0, &smem);
    if (smem < 2048 + 8 * 2 * 4096) smem = 2048 + 8 * 2 * 4096;        // the epilogue's staging slabs reuse the stage memory
    if (p.splits > 1 && smem < kSplitSmemFloor) smem = kSplitSmemFloor;
    static bool attr_set = false;
    if (!attr_set) {
        PT_CUDA_OK(cudaFuncSetAttribute(conv_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        attr_set = true;
    }
    dim3 grid((unsigned)gx, (unsigned)p.splits);
    if (c->test_skip == 1 && p.splits > 1) { p.test_skip = 1; c->test_skip = 0; }
    PT_CUDA_OK(launch_pdl(conv_wgrad_kernel, grid, dim3(kThreads), smem, st, tmA, tmX, tmP, p));
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

// Launches the row-block weight-gradient kernel; PT_ERR_UNSUPPORTED (nothing launched) where the plan declines the shape.
// `x_row_pixels` > 0 and (lo_h, lo_w): x is a view whose rows are x_row_pixels apart and whose raster origin for tap (0, 0)
// is at (lo_h, lo_w) instead of (-pad, -pad) -- the space-to-depth stem, whose "pixels" are overlapping 4-pixel windows.
pt_status run_wgrad_rows(pt_ctx *c, const pt_conv_desc *d, int P, int Q, const void *x, const void *dy, float *out, void *ws,
                         size_t ws_bytes, cudaStream_t st, int x_row_pixels = 0, int lo_h = 0, int lo_w = 0)
{
    const WgRows wr = wgrad_rows_plan(c, d, P, Q);
    if (!wr.ok || !c->encode_tiled) return PT_ERR_UNSUPPORTED;
    WgradP p;
    memset(&p, 0, sizeof(p));
    p.K = d->K; p.C = d->C; p.taps = d->R * d->S; p.S = d->S;
    p.BN = wr.bn; p.n_tiles = wr.n_tiles; p.m_tiles = wr.m_tiles;
    p.tpc = wr.tpc; p.tap_groups = wr.tap_groups;
    p.pair = 1; p.apc = wr.apc; p.acc_cols = wr.acc_cols;
    p.npix = d->N * P * Q;
    p.splits = wr.splits;
    p.Pd = P; p.Qd = Q; p.stride = 1; p.lo_h = -d->pad; p.lo_w = -d->pad;
    if (x_row_pixels > 0) { p.lo_h = lo_h; p.lo_w = lo_w; }
    p.nr = wr.nr; p.Wp = wr.Wp; p.RB = wr.RB; p.units = wr.units; p.units_per_split = wr.units_per_split;
    p.ksteps = wr.ksteps; p.nb_a = wr.nb_a; p.lo_span = d->R - 1; p.a_box = wr.a_box; p.b_box = wr.b_box;
    p.stages = wr.stages;
    p.tmem_cols = pow2_cols(p.apc * p.acc_cols);
    p.status = c->d_status;
    p.out = out;
    const int gx = p.n_tiles * p.m_tiles * p.tap_groups;
    CUtensorMap tmP, tmA, tmX;
    memset(&tmP, 0, sizeof(tmP));
    if (p.splits > 1) {
        const size_t need = (size_t)gx * p.apc * p.splits * 128 * p.acc_cols * sizeof(float);
        if (!ws || ws_bytes < need) return PT_ERR_WORKSPACE;
        p.partial = (float *)ws;
        if (2 * gx > 8192) return PT_ERR_UNSUPPORTED;
        if (c->sync_next + 2 * gx > 16384) c->sync_next = 0;
        p.sync = c->d_sync + c->sync_next;
        c->sync_next += 2 * gx;
        if (!make_partial_map(c, &tmP, ws, p.acc_cols, (size_t)gx * p.apc * p.splits * 128)) return PT_ERR_CUDA;
    }
    // dy: box of nr rows x Wp columns (Wp > Q: the extra columns are out of bounds and read as zeros); x: the halo box
    if (!make_halo_in_map(c, &tmA, dy, d->K, Q, P, d->N, d->ldy, wr.Wp, wr.nr)) return PT_ERR_UNSUPPORTED;
    if (!make_halo_in_map(c, &tmX, x, d->C, d->W, d->H, d->N, d->ldx, wr.Wp, wr.nr + d->R - 1, kKC, x_row_pixels)) return PT_ERR_UNSUPPORTED;
    static bool attr_set = false;
    if (!attr_set) {
        PT_CUDA_OK(cudaFuncSetAttribute(conv_wgrad_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        attr_set = true;
    }
    dim3 grid((unsigned)gx, (unsigned)p.splits);
    const size_t smem = (p.splits > 1 && wr.smem < kSplitSmemFloor) ? kSplitSmemFloor : wr.smem;
    if (c->test_skip == 1 && p.splits > 1) { p.test_skip = 1; c->test_skip = 0; }
    PT_CUDA_OK(launch_pdl(conv_wgrad_rows_kernel, grid, dim3(kThreads), smem, st, tmA, tmX, tmP, p));
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

// Stride-2 data gradient of a bf16 dx with even H and W: the input pixels split by the parity (a, b) of (h, w) into four
// stride-1 correlations over dy (pixel h = 2i + a receives tap r iff a + pad - r is even, from dy row i + (a + pad - r)/2).
// Each parity with taps is one halo-kernel launch that TMA-stores into the strided view of dx holding that parity; if some
// parity has no tap (1x1 stride 2), dx is cleared first. Returns PT_ERR_UNSUPPORTED for shapes the halo kernel declines
// (nothing has been launched then).
pt_status dgrad_stride2_halo(pt_ctx *c, const pt_conv_desc *d, int P, int Q, const void *dy, const void *w, void *dx, cudaStream_t st)
{
    HaloSpec hs[4];
    int n_launch = 0;
    bool any_empty = false;
    for (int ab = 0; ab < 4; ++ab) {
        const int pa = ab >> 1, pb = ab & 1;
        HaloSpec &h = hs[n_launch];
        memset(&h, 0, sizeof(h));
        int oh[kMaxTaps], ow[kMaxTaps], nt = 0;
        for (int r = 0; r < d->R; ++r) {
            if ((pa + d->pad - r) & 1) continue;
            for (int sft = 0; sft < d->S; ++sft) {
                if ((pb + d->pad - sft) & 1) continue;
                if (nt >= kMaxTaps) return PT_ERR_UNSUPPORTED;
                oh[nt] = (pa + d->pad - r) / 2; ow[nt] = (pb + d->pad - sft) / 2;
                h.tap_wt[nt] = r * d->S + sft;
                ++nt;
            }
        }
        if (nt == 0) { any_empty = true; continue; }
        int min_oh = oh[0], min_ow = ow[0], max_oh = oh[0], max_ow = ow[0];
        for (int t = 0; t < nt; ++t) {
            min_oh = oh[t] < min_oh ? oh[t] : min_oh; max_oh = oh[t] > max_oh ? oh[t] : max_oh;
            min_ow = ow[t] < min_ow ? ow[t] : min_ow; max_ow = ow[t] > max_ow ? ow[t] : max_ow;
        }
        for (int t = 0; t < nt; ++t) { h.tap_oh[t] = oh[t] - min_oh; h.tap_ow[t] = ow[t] - min_ow; }
        h.src = dy; h.Cs = d->K; h.Ws = Q; h.Hs = P; h.lds = d->ldy;
        h.P = d->H / 2; h.Q = d->W / 2;
        h.n_taps = nt; h.span_h = max_oh - min_oh + 1; h.span_w = max_ow - min_ow + 1;
        h.lo_h = min_oh; h.lo_w = min_ow;
        h.n_cols = d->C; h.ld_out = d->ldx;
        h.oH = d->H; h.oW = d->W; h.o_step = 2; h.o_h0 = pa; h.o_w0 = pb;
        if (h.Q + h.span_w - 1 > 128) return PT_ERR_UNSUPPORTED;
        ++n_launch;
    }
    if (n_launch == 0) return PT_ERR_UNSUPPORTED;
    // a 1x1 filter on tiny images: one image fills less than half of a 128-row tile and the reduction is deep, so the
    // pixel-linear tiles of the im2col kernel do better
    if (d->R * d->S == 1 && (d->H / 2) * (d->W / 2) < 64) return PT_ERR_UNSUPPORTED;
    if (any_empty) PT_CUDA_OK(cudaMemsetAsync(dx, 0, (size_t)d->N * d->H * d->W * d->ldx * 2, st));
    // The parity classes write disjoint pixels of dx and read the same inputs: launches 1.. go to the context's helper
    // streams (forked from and joined back to the caller's stream by events) so that their fills and drains overlap.
    if (n_launch > 1 && !c->fork_ev) {
        bool ok = cudaEventCreateWithFlags(&c->fork_ev, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < 3 && ok; ++i)
            ok = cudaStreamCreateWithFlags(&c->fork_stream[i], cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->join_ev[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) { (void)cudaGetLastError(); return PT_ERR_CUDA; }
    }
    if (n_launch > 1) {
        // each parity launch would fill the device on its own and they would run one after the other, each paying its start
        // and drain; sharing the SMs in proportion to their taps lets them run side by side
        // (measured: 28x28 <- 14x14, 200 channels: 40.7 -> 26.0 us; with three or more tiles per CTA it no longer pays)
        int taps_total = 0;
        for (int i = 0; i < n_launch; ++i) taps_total += hs[i].n_taps;
        const int wp = hs[0].Q + 1, nr = 128 / wp < hs[0].P ? 128 / wp : hs[0].P;
        int n_tiles;
        (void)tile_n(d->C, &n_tiles);
        const bool few_tiles = nr > 0 && d->N * pt_ceil_div(hs[0].P, nr) * n_tiles <= 2 * c->sm_count;
        for (int i = 0; i < n_launch && few_tiles; ++i) {
            hs[i].max_ctas = c->sm_count * hs[i].n_taps / taps_total;
            if (hs[i].max_ctas < 8) hs[i].max_ctas = 8;
        }
    }
    if (n_launch > 1) PT_CUDA_OK(cudaEventRecord(c->fork_ev, st));
    pt_status first = PT_OK;
    for (int i = 0; i < n_launch; ++i) {
        cudaStream_t si = i == 0 ? st : c->fork_stream[i - 1];
        if (i > 0) PT_CUDA_OK(cudaStreamWaitEvent(si, c->fork_ev, 0));
        pt_status r = launch_halo<true>(c, d, hs[i], w, dx, si);
        if (i > 0) {                                   // join even after a failure, so that a capture stays well formed
            PT_CUDA_OK(cudaEventRecord(c->join_ev[i - 1], si));
            PT_CUDA_OK(cudaStreamWaitEvent(st, c->join_ev[i - 1], 0));
        }
        if (r != PT_OK && first == PT_OK)
            first = (r == PT_ERR_UNSUPPORTED && i == 0 && !any_empty) ? r : (r == PT_ERR_UNSUPPORTED ? PT_ERR_CUDA : r);
        if (first != PT_OK && i == 0) return first;    // nothing forked yet
    }
    return first;
}

}  // namespace

bool pt_sm100_conv_supported(const pt_ctx *c, const pt_conv_desc *d, int which)
{
    if (!c->encode_tiled || !c->encode_im2col) return false;
    if (d->stride > 8 || d->pad > 100 || d->R * d->S > kMaxTaps) return false;
    if (which == PT_CONV_FWD) return true;
    if (which == PT_CONV_DGRAD) return (d->stride == 1 && d->pad <= d->R - 1 && d->pad <= d->S - 1) || d->stride == 2;
    return true;
}

// The stem's weight gradient as the generic kernel sees it: U taps of 64 "channels".
static pt_conv_desc stem_virtual_desc(const pt_conv_desc *d, const StemPlan &sp)
{
    pt_conv_desc v = *d;
    v.C = 64; v.R = sp.U; v.S = 1;
    return v;
}

// The same for the row-block kernel: a stride-1 U x 1 filter over Q x Hs "pixels" of 64 lanes whose rows are Wp real pixels
// (16 lanes each) apart; pixel j of a row is the window of real pixels j .. j+3.
static pt_conv_desc stem_rows_desc(const pt_conv_desc *d, const StemPlan &sp)
{
    pt_conv_desc v = stem_virtual_desc(d, sp);
    v.stride = 1; v.W = sp.Q; v.H = sp.Hs; v.ldx = 16;
    return v;
}

// CTAs the weight gradient of `d` launches at the context's current CTA limit: tiles x splits; *waits = 1 if they wait for
// one another (splits > 1).
int pt_sm100_wgrad_ctas(const pt_ctx *c, const pt_conv_desc *d, int *waits)
{
    const StemPlan sp = stem_plan(d);
    pt_conv_desc v = sp.ok ? stem_virtual_desc(d, sp) : *d;
    const int P = sp.ok ? sp.P : pt_out_dim(d->H, d->R, d->stride, d->pad), Q = sp.ok ? sp.Q : pt_out_dim(d->W, d->S, d->stride, d->pad);
    int tiles, splits;
    const pt_conv_desc vr = sp.ok ? stem_rows_desc(d, sp) : v;
    const WgRows wr = wgrad_rows_plan(c, &vr, P, Q);
    if (wr.ok) {
        tiles = wr.n_tiles * wr.m_tiles * wr.tap_groups;
        splits = wr.splits;
    } else {
        int n_tiles;
        const int bn = tile_n(v.C, &n_tiles);
        const int tpc = wgrad_taps_per_cta(v.R * v.S, bn);
        tiles = pt_ceil_div(v.K, 128) * n_tiles * pt_ceil_div(v.R * v.S, tpc);
        splits = wgrad_splits(c, &v, P, Q);
    }
    if (waits) *waits = splits > 1 ? 1 : 0;
    return tiles * splits;
}

size_t pt_sm100_conv_workspace(const pt_ctx *c, const pt_conv_desc *d, int which)
{
    const StemPlan sp = stem_plan(d);
    if (sp.ok && which == PT_CONV_FWD) return sp.xs_bytes + pt_align_up(sp.w2_elems * 2, 1024);
    if (sp.ok && which == PT_CONV_WGRAD) {
        const pt_conv_desc v = stem_virtual_desc(d, sp), vr = stem_rows_desc(d, sp);
        const size_t pa = wgrad_partial_bytes(c, &v, sp.P, sp.Q), pb = wgrad_partial_bytes(c, &vr, sp.P, sp.Q);
        return sp.xs_bytes + pt_align_up(sp.w2_elems * 4, 1024) + (pa > pb ? pa : pb);
    }
    if (which != PT_CONV_WGRAD) return 0;
    const int P = pt_out_dim(d->H, d->R, d->stride, d->pad), Q = pt_out_dim(d->W, d->S, d->stride, d->pad);
    return wgrad_partial_bytes(c, d, P, Q);
}

pt_status pt_sm100_conv(pt_ctx *c, const pt_conv_desc *d, int which, const void *a, const void *b, void *out, void *ws,
                        size_t ws_bytes, cudaStream_t st)
{
    const int P = pt_out_dim(d->H, d->R, d->stride, d->pad), Q = pt_out_dim(d->W, d->S, d->stride, d->pad);
    CUtensorMap tmA, tmB;
    const StemPlan sp = stem_plan(d);
    if (which == PT_CONV_WGRAD) {
        if (sp.ok) {
            // stem: space-to-depth copy of x, generic wgrad over U taps x 64 lanes, then back to [K][R][S][C]
            char *wsb = (char *)ws;
            __nv_bfloat16 *xs = (__nv_bfloat16 *)wsb;
            float *dw2 = (float *)(wsb + sp.xs_bytes);
            char *part = wsb + sp.xs_bytes + pt_align_up(sp.w2_elems * 4, 1024);
            const pt_conv_desc v = stem_virtual_desc(d, sp);
            const size_t tot = (size_t)d->N * sp.Hs * sp.Wp;
            stem_s2d_x_kernel_launch((unsigned)((tot + 255) / 256), st, (const __nv_bfloat16 *)a, xs, d->N, d->H, d->W, d->C, sp.Hs, sp.Ws,
                                     sp.Wp, sp.pl);
            c->launches += 1;
            // the row-block kernel first: the windows of a unit of rows are staged once for all U vertical taps and two taps share
            // an MMA (M = 128 lanes where the generic kernel has 55 output channels on its M side)
            const pt_conv_desc vr = stem_rows_desc(d, sp);
            pt_status r = run_wgrad_rows(c, &vr, sp.P, sp.Q, xs, b, dw2, part, ws_bytes - (size_t)(part - wsb), st, sp.Wp, -sp.pl, 0);
            if (r == PT_ERR_UNSUPPORTED) {
                CUtensorMap tmX;
                const int up_h = (sp.P - 1) - sp.pl - (sp.Hs - 1);
                if (!make_im2col_map(c, &tmX, xs, 64, sp.Q, sp.Hs, d->N, 16, 0, -sp.pl, 0, up_h, 1, 64, sp.Wp)) return PT_ERR_CUDA;
                r = run_wgrad(c, &v, sp.P, sp.Q, 1, -sp.pl, 0, tmX, b, dw2, part, ws_bytes - (size_t)(part - wsb), st);
            }
            if (r != PT_OK) return r;
            const int n = d->K * d->R * d->S * d->C;
            stem_dw_back_kernel<<<(n + 255) / 256, 256, 0, st>>>(dw2, (float *)out, d->K, d->R, d->S, d->C, sp.U, sp.off);
            c->launches += 1;
            PT_CUDA_OK(cudaGetLastError());
            return PT_OK;
        }
        {
            const pt_status r = run_wgrad_rows(c, d, P, Q, a, b, (float *)out, ws, ws_bytes, st);
            if (r != PT_ERR_UNSUPPORTED) return r;
        }
        CUtensorMap tmX;
        const int up_w = (Q - 1) * d->stride - d->pad - (d->W - 1), up_h = (P - 1) * d->stride - d->pad - (d->H - 1);
        const bool plain = d->R == 1 && d->S == 1 && d->stride == 1 && d->pad == 0;     // pixels of x and dy coincide
        if (plain) {
            if (!make_act2d_map(c, &tmX, a, d->C, (long long)d->N * d->H * d->W, d->ldx, 64)) return PT_ERR_CUDA;
        } else if (!make_im2col_map(c, &tmX, a, d->C, d->W, d->H, d->N, d->ldx, -d->pad, -d->pad, up_w, up_h, d->stride, 64)) return PT_ERR_CUDA;
        return run_wgrad(c, d, P, Q, d->stride, -d->pad, -d->pad, tmX, b, (float *)out, ws, ws_bytes, st, plain);
    }

    GemmP p;
    memset(&p, 0, sizeof(p));
    p.status = c->d_status;
    p.out = out;
    p.out_f32 = d->out_f32;
    if (which == PT_CONV_FWD && sp.ok) {
        char *wsb = (char *)ws;
        __nv_bfloat16 *xs = (__nv_bfloat16 *)wsb, *w2 = (__nv_bfloat16 *)(wsb + sp.xs_bytes);
        const size_t tot = (size_t)d->N * sp.Hs * sp.Wp;
        stem_s2d_x_kernel_launch((unsigned)((tot + 255) / 256), st, (const __nv_bfloat16 *)a, xs, d->N, d->H, d->W, d->C, sp.Hs, sp.Ws, sp.Wp,
                                 sp.pl);
        stem_s2d_w_kernel<<<(unsigned)((sp.w2_elems + 255) / 256), 256, 0, st>>>((const __nv_bfloat16 *)b, w2, d->K, d->R, d->S, d->C, d->ldw,
                                                                              sp.U, sp.V, sp.off);
        c->launches += 2;
        // (plain launches: the convolution below loads w2 before its dependency wait, which is safe because stem_s2d_w_kernel
        // does not release its dependents before it has completed)
        if (!d->out_f32) {
            // row-block form on 32-byte pixels: the U x V taps are row shifts of one staged tile (each xs byte read once)
            HaloSpec h;
            memset(&h, 0, sizeof(h));
            h.src = xs; h.Cs = 16; h.Ws = sp.Wp; h.Hs = sp.Hs; h.lds = 16;
            h.P = sp.P; h.Q = sp.Q;
            h.n_taps = sp.U * sp.V; h.span_h = sp.U; h.span_w = sp.V;
            h.lo_h = -sp.pl; h.lo_w = 0;
            for (int t = 0; t < h.n_taps; ++t) { h.tap_oh[t] = t / sp.V; h.tap_ow[t] = t % sp.V; h.tap_wt[t] = (t / sp.V) * 4 + t % sp.V; }
            h.n_cols = d->K; h.ld_out = d->ldy;
            h.oH = sp.P; h.oW = sp.Q; h.o_step = 1; h.o_h0 = 0; h.o_w0 = 0;
            h.row32 = 1; h.w_taps = sp.U * 4;
            const pt_status r = launch_halo<false>(c, d, h, w2, out, st);
            if (r != PT_ERR_UNSUPPORTED) return r;
        }
        p.M_total = d->N * sp.P * sp.Q;
        p.n_cols = d->K;
        p.BN = tile_n(d->K, &p.n_tiles);
        p.c_red = 64;
        p.k_chunks = 1;
        p.taps = sp.U;
        for (int t = 0; t < p.taps; ++t) { p.tap_oh[t] = (unsigned char)t; p.tap_ow[t] = 0; p.tap_wt[t] = (unsigned short)t; }
        p.Pd = sp.P; p.Qd = sp.Q; p.stride = 1; p.lo_h = -sp.pl; p.lo_w = 0;
        p.oH = sp.P; p.oW = sp.Q; p.o_step = 1; p.o_h0 = 0; p.o_w0 = 0; p.ld_out = d->ldy; p.zero_mask = 0;
        p.tmem_cols = pow2_cols(p.BN);
        const int up_h = (sp.P - 1) - sp.pl - (sp.Hs - 1);
        if (!make_im2col_map(c, &tmA, xs, 64, sp.Q, sp.Hs, d->N, 16, 0, -sp.pl, 0, up_h, 1, kBM, sp.Wp)) return PT_ERR_CUDA;
        if (!make_weight_map(c, &tmB, w2, 64, sp.U, d->K, 64, p.BN)) return PT_ERR_CUDA;
        return launch_gemm<false>(c, tmA, tmB, p, st);
    }
    // A halo tile is whole raster rows of ONE image in at most 128 MMA rows: on small maps most of the tile is padding (7x7:
    // 49 useful rows of 128), and the pixel-linear tiles of the im2col kernel do better (7x7, 345 -> 374: 23 us against 30)
    const int raster_h = which == PT_CONV_FWD ? P : d->H, raster_w = which == PT_CONV_FWD ? Q : d->W;
    const int halo_wp = raster_w + d->S - 1;
    const int halo_nr = halo_wp <= 128 ? (128 / halo_wp < raster_h ? 128 / halo_wp : raster_h) : 1;
    const bool sparse_tiles = 2 * raster_h * raster_w < pt_ceil_div(raster_h, halo_nr) * 128;
    if (!sparse_tiles && which == PT_CONV_FWD && d->stride == 1 && d->R * d->S > 1 && d->R * d->S <= kMaxTaps) {
        HaloSpec h;
        halo_spec_stride1(d, &h, a, d->C, d->W, d->H, d->ldx, d->K, P, Q, d->ldy, d->pad, d->pad, false);
        pt_status r = launch_halo<false>(c, d, h, b, out, st);
        if (r != PT_ERR_UNSUPPORTED) return r;
    }
    if (!sparse_tiles && which == PT_CONV_DGRAD && d->stride == 1 && d->R * d->S > 1 && d->R * d->S <= kMaxTaps && d->pad <= d->R - 1 &&
        d->pad <= d->S - 1) {
        // dx = correlation of dy (padding R-1-pad) with the taps visited flipped
        HaloSpec h;
        halo_spec_stride1(d, &h, a, d->K, Q, P, d->ldy, d->C, d->H, d->W, d->ldx, d->R - 1 - d->pad, d->S - 1 - d->pad, true);
        pt_status r = launch_halo<true>(c, d, h, b, out, st);
        if (r != PT_ERR_UNSUPPORTED) return r;
    }
    if (which == PT_CONV_DGRAD && d->stride == 2 && !d->out_f32 && (d->H % 2 == 0) && (d->W % 2 == 0)) {
        pt_status r = dgrad_stride2_halo(c, d, P, Q, a, b, out, st);
        if (r != PT_ERR_UNSUPPORTED) return r;
    }
    if (which == PT_CONV_FWD) {
        // raster = output pixels (P x Q per image); source = x
        p.M_total = d->N * P * Q;
        p.n_cols = d->K;
        p.BN = tile_n(d->K, &p.n_tiles, pt_ceil_div(p.M_total, kBM), c->sm_count);
        p.c_red = d->C;
        p.k_chunks = pt_ceil_div(d->C, kKC);
        p.taps = d->R * d->S;
        for (int t = 0; t < p.taps; ++t) { p.tap_oh[t] = (unsigned char)(t / d->S); p.tap_ow[t] = (unsigned char)(t % d->S); p.tap_wt[t] = (unsigned short)t; }
        p.Pd = P; p.Qd = Q; p.stride = d->stride; p.lo_h = -d->pad; p.lo_w = -d->pad;
        p.oH = P; p.oW = Q; p.o_step = 1; p.o_h0 = 0; p.o_w0 = 0; p.ld_out = d->ldy; p.zero_mask = 0;
        p.tmem_cols = pow2_cols(p.BN);
        // the box of base positions must hold exactly P x Q positions at the traversal stride
        const int up_w = (Q - 1) * d->stride - d->pad - (d->W - 1), up_h = (P - 1) * d->stride - d->pad - (d->H - 1);
        if (d->R == 1 && d->S == 1 && d->stride == 1 && d->pad == 0) {
            p.a_tiled = 1;
            if (!make_act2d_map(c, &tmA, a, d->C, (long long)d->N * d->H * d->W, d->ldx, kBM)) return PT_ERR_CUDA;
        } else if (!make_im2col_map(c, &tmA, a, d->C, d->W, d->H, d->N, d->ldx, -d->pad, -d->pad, up_w, up_h, d->stride, kBM)) return PT_ERR_CUDA;
        if (!make_weight_map(c, &tmB, b, d->C, d->R * d->S, d->K, d->ldw, p.BN)) return PT_ERR_CUDA;
        return launch_gemm<false>(c, tmA, tmB, p, st);
    }
    if (which != PT_CONV_DGRAD) return PT_ERR_UNSUPPORTED;
    p.n_cols = d->C;
    p.BN = tile_n(d->C, &p.n_tiles, pt_ceil_div(d->N * d->H * d->W / (d->stride * d->stride), kBM), c->sm_count);
    p.c_red = d->K;
    p.k_chunks = pt_ceil_div(d->K, kKC);
    p.tmem_cols = pow2_cols(p.BN);
    p.oH = d->H; p.oW = d->W; p.ld_out = d->ldx;
    if (!make_weight_map(c, &tmB, b, d->C, d->R * d->S, d->K, d->ldw, kKC)) return PT_ERR_CUDA;
    if (d->stride == 1) {
        // raster = input pixels (H x W per image); source = dy with padding R-1-pad and the taps visited flipped:
        // dx[h,w] = sum_{r',s'} dy[h - (R-1-pad) + r', w - (S-1-pad) + s'] * w[R-1-r', S-1-s']
        const int ph = d->R - 1 - d->pad, pw = d->S - 1 - d->pad;
        if (ph < 0 || pw < 0) return PT_ERR_UNSUPPORTED;
        p.M_total = d->N * d->H * d->W;
        p.taps = d->R * d->S;
        for (int t = 0; t < p.taps; ++t) {
            p.tap_oh[t] = (unsigned char)(t / d->S); p.tap_ow[t] = (unsigned char)(t % d->S);
            p.tap_wt[t] = (unsigned short)(p.taps - 1 - t);
        }
        p.Pd = d->H; p.Qd = d->W; p.stride = 1; p.lo_h = -ph; p.lo_w = -pw;
        p.o_step = 1; p.o_h0 = 0; p.o_w0 = 0; p.zero_mask = 0;
        const int up_w = (d->W - 1) - pw - (Q - 1), up_h = (d->H - 1) - ph - (P - 1);
        if (d->R == 1 && d->S == 1 && d->pad == 0) {
            p.a_tiled = 1;
            if (!make_act2d_map(c, &tmA, a, d->K, (long long)d->N * P * Q, d->ldy, kBM)) return PT_ERR_CUDA;
        } else if (!make_im2col_map(c, &tmA, a, d->K, Q, P, d->N, d->ldy, -pw, -ph, up_w, up_h, 1, kBM)) return PT_ERR_CUDA;
        return launch_gemm<true>(c, tmA, tmB, p, st);
    }
    if (d->stride != 2) return PT_ERR_UNSUPPORTED;
    // Stride 2: the input pixels split by the parity (a, b) of (h, w) into four stride-1 problems over dy.
    // Pixel h = 2i + a receives tap r iff (a + pad - r) is even, from dy row p = i + (a + pad - r)/2.
    // Parities no tap reaches are zero-filled by the epilogue of the first launched parity.
    struct Par { int a, b, nt; int oh[kMaxTaps], ow[kMaxTaps], wt[kMaxTaps]; };
    Par par[4];
    int empty_mask = 0, first = -1;
    for (int ab = 0; ab < 4; ++ab) {
        Par &q = par[ab];
        q.a = ab >> 1; q.b = ab & 1; q.nt = 0;
        for (int r = 0; r < d->R; ++r) {
            if ((q.a + d->pad - r) & 1) continue;
            for (int s = 0; s < d->S; ++s) {
                if ((q.b + d->pad - s) & 1) continue;
                q.oh[q.nt] = (q.a + d->pad - r) / 2;      // exact: the difference is even (may be negative)
                q.ow[q.nt] = (q.b + d->pad - s) / 2;
                q.wt[q.nt] = r * d->S + s;
                ++q.nt;
            }
        }
        const int rows = (d->H - q.a + 1) / 2, cols = (d->W - q.b + 1) / 2;
        if (rows <= 0 || cols <= 0) { q.nt = -1; continue; }          // no pixel has this parity
        if (q.nt == 0) empty_mask |= 1 << ab; else if (first < 0) first = ab;
    }
    if (first < 0) return PT_ERR_UNSUPPORTED;
    if (empty_mask && (par[first].a != 0 || par[first].b != 0)) return PT_ERR_UNSUPPORTED;   // cells are anchored at parity (0,0)
    for (int ab = 0; ab < 4; ++ab) {
        Par &q = par[ab];
        if (q.nt <= 0) continue;
        int min_oh = q.oh[0], min_ow = q.ow[0];
        for (int t = 0; t < q.nt; ++t) { min_oh = q.oh[t] < min_oh ? q.oh[t] : min_oh; min_ow = q.ow[t] < min_ow ? q.ow[t] : min_ow; }
        const int rows = (d->H - q.a + 1) / 2, cols = (d->W - q.b + 1) / 2;
        p.M_total = d->N * rows * cols;
        p.taps = q.nt;
        for (int t = 0; t < q.nt; ++t) {
            p.tap_oh[t] = (unsigned char)(q.oh[t] - min_oh); p.tap_ow[t] = (unsigned char)(q.ow[t] - min_ow);
            p.tap_wt[t] = (unsigned short)q.wt[t];
        }
        p.Pd = rows; p.Qd = cols; p.stride = 1; p.lo_h = min_oh; p.lo_w = min_ow;
        p.o_step = 2; p.o_h0 = q.a; p.o_w0 = q.b;
        p.zero_mask = (ab == first) ? empty_mask : 0;
        const int up_w = (cols - 1) + min_ow - (Q - 1), up_h = (rows - 1) + min_oh - (P - 1);
        if (!make_im2col_map(c, &tmA, a, d->K, Q, P, d->N, d->ldy, min_ow, min_oh, up_w, up_h, 1, kBM)) return PT_ERR_CUDA;
        pt_status s = launch_gemm<true>(c, tmA, tmB, p, st);
        if (s != PT_OK) return s;
    }
    return PT_OK;
}

// Sets the limit of the bounded device-side waits of this file's kernels (the variable lives in this translation unit).
pt_status pt_sm100_set_wait_limit_ns(unsigned long long ns, cudaStream_t st)
{
    PT_CUDA_OK(cudaMemcpyToSymbolAsync(g_wait_limit_ns, &ns, sizeof(ns), 0, cudaMemcpyHostToDevice, st));
    PT_CUDA_OK(cudaStreamSynchronize(st));
    return PT_OK;
}

#ifdef PT_DEVICE_TRACE
extern "C" int pt_debug_wgrad_trace(unsigned long long *host_out)
{
    return (int)cudaMemcpyFromSymbol(host_out, g_wg_trace, sizeof(unsigned long long) * 8 * 64);
}
extern "C" int pt_debug_chain_trace(unsigned long long *host_out, int reset)
{
    cudaError_t e = cudaMemcpyFromSymbol(host_out, g_chain_trace, sizeof(unsigned long long) * 256 * 12);
    if (reset) {
        static const unsigned long long zeros[256 * 12] = {0};
        const unsigned int z = 0;
        (void)cudaMemcpyToSymbol(g_chain_trace, zeros, sizeof(zeros));
        (void)cudaMemcpyToSymbol(g_chain_seq, &z, sizeof(z));
    }
    return (int)e;
}
extern "C" int pt_debug_gemm_trace(unsigned long long *host_out)
{
    return (int)cudaMemcpyFromSymbol(host_out, g_gemm_trace, sizeof(unsigned long long) * 8 * 64);
}
extern "C" int pt_debug_halo_trace(unsigned long long *host_out)
{
    return (int)cudaMemcpyFromSymbol(host_out, g_halo_trace, sizeof(unsigned long long) * 8 * 64);
}
#endif
