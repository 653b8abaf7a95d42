// tcgen05 / TMEM / TMA implicit-GEMM convolutions for sm_100a.
//
// conv_gemm_kernel  (fwd, dgrad):  D[pixel][channel] = sum over taps and reduction channels.
//   A operand: 128 output pixels x 64 reduction channels per stage, fetched by ONE im2col-mode TMA load
//              (the TMA unit walks the output-pixel raster with the conv stride and adds the tap offset,
//              zero-filling the padding halo and the channels past the true, ragged channel count).
//   B operand: the bf16 weight shadow [K][R*S][ldw].
//              fwd   : rows = output channels, 64 input channels contiguous  -> K-major tile, one 3-D TMA box.
//              dgrad : rows = 64 output channels (the reduction), input channels contiguous -> MN-major tiles
//                      straight from the same shadow, taps visited flipped. No transposed copy of the weights.
//   Accumulator: fp32 in TMEM, 128 lanes x BN columns (BN = the ragged channel count rounded up to 16, <= 256).
//   Roles: warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2..5 = epilogue
//          (tcgen05.ld -> bf16/fp32 -> predicated stores at the true channel count).
// Every mbarrier wait is bounded; on expiry the CTA records PT_DEV_TIMEOUT in the status word, drains and exits.
#include "pt_internal.h"
#include "pt_sm100_ptx.cuh"
#include <cudaTypedefs.h>

using namespace sm100;

namespace {

constexpr int kBM = 128;            // output pixels per CTA tile
constexpr int kKC = 64;             // reduction channels per stage (one 128-byte swizzle row)
constexpr int kMaxStages = 8;
constexpr int kThreads = 192;

struct GemmP {
    int M_total;        // output pixels of this launch's raster
    int n_cols;         // true number of output channels
    int BN;             // tile width (multiple of 16)
    int n_tiles;        // tiles along the channel dimension
    int c_red;          // true number of reduction channels
    int k_chunks;       // ceil(c_red / 64)
    int taps, S;        // R*S and S
    int Pd, Qd;         // raster of output pixels (rows, columns) per image
    int stride;         // traversal stride of the raster in the source tensor
    int lo_h, lo_w;     // source coordinate of raster position (0,0) for tap (0,0)
    int flip;           // dgrad: weight tap = taps-1-tap
    int stages;
    int tmem_cols;
    // output pixel mapping: pixel (n, i, j) of the raster -> out[((n*oH + i*o_step + o_h0)*oW + j*o_step + o_w0)*ld_out]
    int oH, oW, o_step, o_h0, o_w0;
    int ld_out, out_f32;
    int zero_mask;      // stride-2 dgrad: bit (a*2+b) set => also write zeros to the pixel at parity (a,b) of each 2x2 cell
    void *out;
    unsigned int *status;
};

struct __align__(8) Ctl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t accum;
    uint32_t tmem_base;
    int abort_flag;
};

template <bool B_MN>
__global__ void __launch_bounds__(kThreads) conv_gemm_kernel(const __grid_constant__ CUtensorMap tmA,
                                                              const __grid_constant__ CUtensorMap tmB, const GemmP p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Ctl *ctl = reinterpret_cast<Ctl *>(smem_raw);
    // stage buffers start at the first 1024-byte boundary after the control block
    const uint32_t smem_base = smem_u32(smem_raw);
    const uint32_t data_base = (smem_base + (uint32_t)sizeof(Ctl) + 1023u) & ~1023u;
    const uint32_t a_bytes = kBM * kKC * 2;
    const uint32_t b_bytes = B_MN ? (uint32_t)((p.BN + 63) / 64) * 8192u : (uint32_t)p.BN * 128u;
    const uint32_t stage_bytes = a_bytes + ((b_bytes + 1023u) & ~1023u);
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tile = blockIdx.x % p.n_tiles, m_tile = blockIdx.x / p.n_tiles;
    const int m0 = m_tile * kBM, n0 = n_tile * p.BN;
    const int iters = p.taps * p.k_chunks;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 1);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        mbar_init(smem_u32(&ctl->accum), 1);
        ctl->abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer
            const int q = m0 % p.Qd, t = m0 / p.Qd, pp = t % p.Pd, n = t / p.Pd;
            const int w0 = q * p.stride + p.lo_w, h0 = pp * p.stride + p.lo_h;
            int issued = 0;
            for (int it = 0; it < iters; ++it) {
                const int s = it % p.stages, ph = (it / p.stages) & 1;
                if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1, abort_flag, p.status, 1)) break;
                const int tap = it / p.k_chunks, kc = it - tap * p.k_chunks;
                const int r = tap / p.S, sft = tap - r * p.S;
                const uint32_t bar = smem_u32(&ctl->full[s]);
                const uint32_t a_dst = data_base + (uint32_t)s * stage_bytes, b_dst = a_dst + a_bytes;
                mbar_arrive_expect_tx(bar, a_bytes + b_bytes);
                tma_load_im2col_4d(a_dst, &tmA, bar, kc * kKC, w0, h0, n, (uint16_t)sft, (uint16_t)r);
                const int wtap = p.flip ? p.taps - 1 - tap : tap;
                if (!B_MN) {
                    tma_load_3d(b_dst, &tmB, bar, kc * kKC, wtap, n0);
                } else {
                    for (int nb = 0; nb < (p.BN + 63) / 64; ++nb)
                        tma_load_3d(b_dst + (uint32_t)nb * 8192u, &tmB, bar, n0 + nb * 64, wtap, kc * kKC);
                }
                issued = it + 1;
            }
            if (*abort_flag) {
                // drain: give the copies already issued a bounded time to land before the CTA's smem is released
                for (int it = max(0, issued - p.stages); it < issued; ++it) {
                    const int s = it % p.stages, ph = (it / p.stages) & 1;
                    const uint64_t t0 = globaltimer_ns();
                    while (!mbar_try_wait(smem_u32(&ctl->full[s]), ph) && globaltimer_ns() - t0 < 20000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer
            const uint32_t idesc = make_idesc_bf16(kBM, p.BN, 0, B_MN ? 1 : 0);
            bool ok = true;
            for (int it = 0; it < iters && ok; ++it) {
                const int s = it % p.stages, ph = (it / p.stages) & 1;
                ok = mbar_wait(smem_u32(&ctl->full[s]), ph, abort_flag, p.status, 2);
                if (!ok) break;
                tc_fence_after();
                const int kc = it % p.k_chunks;
                const int rem = p.c_red - kc * kKC;
                const int ksteps = rem >= kKC ? 4 : (rem + 15) / 16;
                const uint32_t a_src = data_base + (uint32_t)s * stage_bytes, b_src = a_src + a_bytes;
#pragma unroll 1
                for (int k = 0; k < ksteps; ++k) {
                    const uint64_t ad = make_desc(a_src + (uint32_t)k * 32u, 16u, 1024u);
                    const uint64_t bd = B_MN ? make_desc(b_src + (uint32_t)k * 2048u, 8192u, 1024u)
                                             : make_desc(b_src + (uint32_t)k * 32u, 16u, 1024u);
                    umma_bf16(tmem_base, ad, bd, idesc, (it | k) != 0 ? 1u : 0u);
                }
                umma_commit(smem_u32(&ctl->empty[s]));       // frees the stage when these MMAs have read it
            }
            if (ok) umma_commit(smem_u32(&ctl->accum));      // accumulator complete
        }
    } else {
        // ---------------- epilogue: warp w may touch TMEM lanes 32*(w%4) .. +31
        const int quarter = warp & 3;
        const bool ok = mbar_wait(smem_u32(&ctl->accum), 0, abort_flag, p.status, 3);
        tc_fence_after();
        if (ok) {
            const int m = m0 + quarter * 32 + lane;
            const bool row_ok = m < p.M_total;
            size_t row_off = 0;
            int cell_h = 0, cell_w = 0, img = 0;
            if (row_ok) {
                const int j = m % p.Qd, t = m / p.Qd, i = t % p.Pd;
                img = t / p.Pd;
                cell_h = i * p.o_step;
                cell_w = j * p.o_step;
                row_off = ((size_t)(img * p.oH + cell_h + p.o_h0) * p.oW + cell_w + p.o_w0) * (size_t)p.ld_out;
            }
            const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
            for (int c0 = 0; c0 < p.BN; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(lane_addr + (uint32_t)c0, v);
                tmem_ld_wait();
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
            // stride-2 data gradient: pixels of this 2x2 cell that no tap reaches are written as zeros here
            if (row_ok && p.zero_mask && n_tile == 0) {
                for (int ab = 0; ab < 4; ++ab) {
                    if (!((p.zero_mask >> ab) & 1)) continue;
                    const int hh = cell_h + (ab >> 1), ww = cell_w + (ab & 1);
                    if (hh >= p.oH || ww >= p.oW) continue;
                    const size_t off = ((size_t)(img * p.oH + hh) * p.oW + ww) * (size_t)p.ld_out;
                    if (p.out_f32) {
                        float *o = (float *)p.out + off;
                        for (int e = 0; e < p.n_cols; ++e) o[e] = 0.f;
                    } else {
                        __nv_bfloat16 *o = (__nv_bfloat16 *)p.out + off;
                        int e = 0;
                        for (; e + 8 <= p.n_cols; e += 8) *reinterpret_cast<uint4 *>(o + e) = make_uint4(0, 0, 0, 0);
                        for (; e < p.n_cols; ++e) o[e] = __float2bfloat16_rn(0.f);
                    }
                }
            }
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
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
                     int up_w, int up_h, int stride, int pixels)
{
    if (!c->encode_im2col) return false;
    if (lo_w < -128 || lo_h < -128 || up_w < -128 || up_h < -128 || lo_w > 127 || lo_h > 127 || up_w > 127 || up_h > 127) return false;
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
    cuuint64_t strides[3] = {(cuuint64_t)ld * 2, (cuuint64_t)W * ld * 2, (cuuint64_t)H * W * ld * 2};
    int lo[2] = {lo_w, lo_h}, up[2] = {up_w, up_h};
    cuuint32_t estr[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
    CUresult r = ((EncodeIm2colFn)c->encode_im2col)(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, lo,
                                                    up, (cuuint32_t)kKC, (cuuint32_t)pixels, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
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
    return r == CUDA_SUCCESS;
}

int tile_n(int cols, int *n_tiles)
{
    int nt = pt_ceil_div(cols, 256);
    int bn = pt_ceil_div(pt_ceil_div(cols, nt), 16) * 16;
    *n_tiles = pt_ceil_div(cols, bn);
    return bn;
}

int pow2_cols(int bn)
{
    int c = 32;
    while (c < bn) c <<= 1;
    return c;
}

template <bool B_MN>
pt_status launch_gemm(pt_ctx *c, const CUtensorMap &tmA, const CUtensorMap &tmB, GemmP &p, cudaStream_t st)
{
    const size_t a_bytes = kBM * kKC * 2;
    const size_t b_bytes = B_MN ? (size_t)pt_ceil_div(p.BN, 64) * 8192 : pt_align_up((size_t)p.BN * 128, 1024);
    const size_t stage = a_bytes + b_bytes;
    int stages = (int)((110 * 1024 - 2048) / stage);           // two CTAs per SM
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) stages = 2;
    const int iters = p.taps * p.k_chunks;
    if (stages > iters) stages = iters < 2 ? 2 : iters;
    p.stages = stages;
    const size_t smem = 2048 + (size_t)stages * stage;
    static bool attr_set[2] = {false, false};
    if (!attr_set[B_MN ? 1 : 0]) {
        PT_CUDA_OK(cudaFuncSetAttribute(conv_gemm_kernel<B_MN>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        attr_set[B_MN ? 1 : 0] = true;
    }
    const int m_tiles = pt_ceil_div(p.M_total, kBM);
    conv_gemm_kernel<B_MN><<<m_tiles * p.n_tiles, kThreads, smem, st>>>(tmA, tmB, p);
    c->launches += 1;
    PT_CUDA_OK(cudaGetLastError());
    return PT_OK;
}

}  // namespace

bool pt_sm100_conv_supported(const pt_ctx *c, const pt_conv_desc *d, int which)
{
    if (!c->encode_tiled || !c->encode_im2col) return false;
    if (d->stride > 8 || d->pad > 100 || d->R > 128 || d->S > 128) return false;
    if (which == PT_CONV_FWD) return true;
    if (which == PT_CONV_DGRAD) return d->stride == 1;
    return false;
}

size_t pt_sm100_conv_workspace(const pt_ctx *, const pt_conv_desc *, int) { return 0; }

pt_status pt_sm100_conv(pt_ctx *c, const pt_conv_desc *d, int which, const void *a, const void *b, void *out, void *ws,
                        size_t ws_bytes, cudaStream_t st)
{
    (void)ws; (void)ws_bytes;
    const int P = pt_out_dim(d->H, d->R, d->stride, d->pad), Q = pt_out_dim(d->W, d->S, d->stride, d->pad);
    GemmP p;
    memset(&p, 0, sizeof(p));
    p.status = c->d_status;
    p.out = out;
    p.out_f32 = d->out_f32;
    p.taps = d->R * d->S;
    p.S = d->S;
    CUtensorMap tmA, tmB;
    if (which == PT_CONV_FWD) {
        // raster = output pixels (P x Q per image); source = x
        p.M_total = d->N * P * Q;
        p.n_cols = d->K;
        p.BN = tile_n(d->K, &p.n_tiles);
        p.c_red = d->C;
        p.k_chunks = pt_ceil_div(d->C, kKC);
        p.Pd = P; p.Qd = Q; p.stride = d->stride; p.lo_h = -d->pad; p.lo_w = -d->pad; p.flip = 0;
        p.oH = P; p.oW = Q; p.o_step = 1; p.o_h0 = 0; p.o_w0 = 0; p.ld_out = d->ldy; p.zero_mask = 0;
        p.tmem_cols = pow2_cols(p.BN);
        // the box of base positions must hold exactly P x Q positions at the traversal stride
        const int up_w = (Q - 1) * d->stride - d->pad - (d->W - 1), up_h = (P - 1) * d->stride - d->pad - (d->H - 1);
        if (!make_im2col_map(c, &tmA, a, d->C, d->W, d->H, d->N, d->ldx, -d->pad, -d->pad, up_w, up_h, d->stride, kBM)) return PT_ERR_CUDA;
        if (!make_weight_map(c, &tmB, b, d->C, d->R * d->S, d->K, d->ldw, p.BN)) return PT_ERR_CUDA;
        return launch_gemm<false>(c, tmA, tmB, p, st);
    }
    if (which == PT_CONV_DGRAD && d->stride == 1) {
        // raster = input pixels (H x W per image); source = dy with padding R-1-pad and flipped taps
        const int ph = d->R - 1 - d->pad, pw = d->S - 1 - d->pad;
        if (ph < 0 || pw < 0) return PT_ERR_UNSUPPORTED;
        p.M_total = d->N * d->H * d->W;
        p.n_cols = d->C;
        p.BN = tile_n(d->C, &p.n_tiles);
        p.c_red = d->K;
        p.k_chunks = pt_ceil_div(d->K, kKC);
        p.Pd = d->H; p.Qd = d->W; p.stride = 1; p.lo_h = -ph; p.lo_w = -pw; p.flip = 1;
        p.oH = d->H; p.oW = d->W; p.o_step = 1; p.o_h0 = 0; p.o_w0 = 0; p.ld_out = d->ldx; p.zero_mask = 0;
        p.tmem_cols = pow2_cols(p.BN);
        const int up_w = (d->W - 1) - pw - (Q - 1), up_h = (d->H - 1) - ph - (P - 1);
        if (!make_im2col_map(c, &tmA, a, d->K, Q, P, d->N, d->ldy, -pw, -ph, up_w, up_h, 1, kBM)) return PT_ERR_CUDA;
        if (!make_weight_map(c, &tmB, b, d->C, d->R * d->S, d->K, d->ldw, kKC)) return PT_ERR_CUDA;
        return launch_gemm<true>(c, tmA, tmB, p, st);
    }
    return PT_ERR_UNSUPPORTED;
}
