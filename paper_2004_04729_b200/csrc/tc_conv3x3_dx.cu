// Dense tensor-core input gradient of 3x3 convolutions (stride 1, pad 1), bf16 operands:
//   dX[b][ci][y][x] = Delta * sum_(co,ky,kx) q[b][co][y+1-ky][x+1-kx] * W[co][ci][ky][kx]
//
// The nine taps are nine accumulating GEMMs (M = 128 input channels, N = 128 positions,
// K = output channels in stages of 64) that all read ONE expanded copy of the codes. The codes
// of a stage are expanded to bf16 once, transposed to [position][co] (a K-major operand whose
// rows are positions), and a tap is then only a different start row of the operand: the
// 128-byte swizzle is a function of the absolute shared-memory address, so a descriptor may
// start at any row. Positions are numbered in a row space h = b * HP + p in which the images
// are HP >= P + W + 1 apart; the rows of a gap are zero, which gives the zero padding above
// and below an image. Left/right padding cannot be a row offset, so the expanded tile exists
// three times: as it is (kx = 1), with the rows of column 0 zeroed (kx = 0, whose source
// column x+1 would otherwise wrap into the next image row) and with the rows of column W-1
// zeroed (kx = 2).
//
// Per stage: the int8 codes are staged by cp.async (rows of the [co][position] plane when the
// plane pitch allows 16-byte copies, else whole [64 co][P] slabs of the images the tile
// touches), sixteen warps expand them into the three copies, one thread issues 36 MMAs per
// 128-channel accumulator, one thread streams the weight tiles (prepared once per call as
// ready-to-use swizzled images) with bulk copies. All waits are bounded.
#include "tc_common.cuh"

namespace dbp {

namespace {

using namespace tc;

constexpr int kXW = 16;                  // expander warps (also the epilogue)
constexpr int kX = kXW * 32;
constexpr int kThreadsS = kX + 64;       // + MMA warp + loader warp
constexpr int kNA = 4;                   // ring of weight tiles
constexpr int kTile = 16384;             // 128 x 64 bf16
constexpr int kRawPitch = 256;           // bytes per staged code row (row mode)

struct Sx3P {
    const int8_t *codes;           // [B][Cout][P]
    const __nv_bfloat16 *Wimg;     // [Cout/64][9][mt_pad] tiles of [128 ci][64 co], swizzled
    const float *delta_p;
    void *dX;
    int dx_f32;
    int B, Cin, Cout, W, P;
    int HP;                        // distance of two images in row space
    int HL;                        // rows staged before the tile (>= W + 1)
    int RQ;                        // rows of one expanded copy (multiple of 8)
    int raw_bytes;                 // bytes of one staging buffer
    int nq;                        // sets of the three expanded copies: 2 (expansion of a stage overlaps the MMAs of the one before) where they fit, else 1
    int nimg;                      // slab mode: images staged per tile
    int mt_pad;                    // 128-channel tiles the weight images provide
    int total;                     // B * HP
    int *err_flag;
};

struct PipeS {
    unsigned long long raw_full[2], qt_full[2], qt_empty[2], a_full[kNA], a_empty[kNA], acc;
    unsigned tmem_base;
};

__device__ __forceinline__ void st_global_v8(void *dst, const unsigned (&w)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                 "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
}
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, unsigned bytes, unsigned long long *bar) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ unsigned pack_bf16(unsigned a, unsigned b, float delta) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(a) * delta, __uint_as_float(b) * delta);
    return *reinterpret_cast<const unsigned *>(&h);
}

// MODE 0: P % 16 == 0 (row staging, 16-position store groups); 1: P % 4 == 0; 2: any P (slabs)
template <int MODE>
__device__ __forceinline__ void store_run(const Sx3P &p, const unsigned (&v)[32], float delta, int ci, int hfirst) {
    constexpr int GS = MODE == 0 ? 8 : MODE == 1 ? 4 : 1;
    int b = hfirst / p.HP, pp = hfirst - b * p.HP;
    if (MODE == 0 && !p.dx_f32) {
#pragma unroll
        for (int j0 = 0; j0 < 32; j0 += 16) {
            if (hfirst + j0 < p.total && pp < p.P) {
                unsigned w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) w[e] = pack_bf16(v[j0 + 2 * e], v[j0 + 2 * e + 1], delta);
                st_global_v8(static_cast<__nv_bfloat16 *>(p.dX) + (static_cast<long long>(b) * p.Cin + ci) * p.P + pp, w);
            }
            pp += 16;
            if (pp >= p.HP) { pp -= p.HP; ++b; }
        }
        return;
    }
#pragma unroll
    for (int j0 = 0; j0 < 32; j0 += GS) {
        if (hfirst + j0 < p.total && pp < p.P) {
            const long long o = (static_cast<long long>(b) * p.Cin + ci) * p.P + pp;
            if (p.dx_f32) {
                float *dst = static_cast<float *>(p.dX) + o;
                if (GS == 8) {
                    unsigned w[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) w[e] = __float_as_uint(__uint_as_float(v[j0 + e]) * delta);
                    st_global_v8(dst, w);
                } else if (GS == 4) {
                    *reinterpret_cast<float4 *>(dst) =
                        make_float4(__uint_as_float(v[j0]) * delta, __uint_as_float(v[j0 + 1]) * delta,
                                    __uint_as_float(v[(j0 + 2) & 31]) * delta, __uint_as_float(v[(j0 + 3) & 31]) * delta);
                } else {
                    dst[0] = __uint_as_float(v[j0]) * delta;
                }
            } else {
                __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.dX) + o;
                if (GS == 4) {
                    *reinterpret_cast<uint2 *>(dst) = make_uint2(pack_bf16(v[j0], v[j0 + 1], delta),
                                                                 pack_bf16(v[(j0 + 2) & 31], v[(j0 + 3) & 31], delta));
                } else {
                    dst[0] = __float2bfloat16_rn(__uint_as_float(v[j0]) * delta);
                }
            }
        }
        pp += GS;
        if (pp >= p.HP) { pp -= p.HP; ++b; }     // groups never straddle an image end
    }
}

template <int MT, int MODE>
__global__ void __launch_bounds__(kThreadsS) tc3_dx_shift_kernel(const Sx3P p) {
    chain_wait();        // launched chained: earlier kernels' writes are visible from here on
    chain_release();
    constexpr bool SLAB = MODE != 0;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char *a_s = smem;                              // kNA weight tiles
    unsigned char *qt = a_s + kNA * kTile;                  // three copies of [RQ rows][64 co]
    const unsigned copy_bytes = static_cast<unsigned>(p.RQ) * 128u;
    unsigned char *raw_s = qt + p.nq * 3 * copy_bytes;      // two staging buffers
    __shared__ PipeS pipe;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h0 = blockIdx.x * 128;
    const int m0 = blockIdx.y * MT;
    const int nch = p.Cout / 64;

    if (threadIdx.x == 0) {
        mbar_init(&pipe.raw_full[0], kX);
        mbar_init(&pipe.raw_full[1], kX);
        for (int b = 0; b < 2; ++b) { mbar_init(&pipe.qt_full[b], kX); mbar_init(&pipe.qt_empty[b], 1); }
        for (int s = 0; s < kNA; ++s) { mbar_init(&pipe.a_full[s], 1); mbar_init(&pipe.a_empty[s], 1); }
        mbar_init(&pipe.acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kXW) tmem_alloc(&pipe.tmem_base, MT * 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_d = pipe.tmem_base;

    if (warp < kXW) {
        const int t = threadIdx.x;
        const int hlo = h0 - p.HL;                           // row of the tile's first staged row
        const int b_lo = (hlo > 0 ? hlo : 0) / p.HP;         // slab mode: first staged image
        // ---- expansion: my rows are (t & 63) + 64 * pass, my chunk of eight co is t >> 6
        const int ch = t >> 6;
        int src_off[4];                 // where my eight bytes start in the staging buffer; -1: zero row
        unsigned zmask = 0;             // bit pass: row is column 0; bit 4 + pass: row is column W - 1
#pragma unroll
        for (int pass = 0; pass < 4; ++pass) {
            const int r = (t & 63) + 64 * pass, h = hlo + r;
            src_off[pass] = -1;
            if (r < p.RQ && h >= 0 && h < p.total) {
                const int b = h / p.HP, pp = h - b * p.HP;
                if (pp < p.P) {
                    const int xs = pp % p.W;
                    if (xs == 0) zmask |= 1u << pass;
                    if (xs == p.W - 1) zmask |= 16u << pass;
                    src_off[pass] = SLAB ? ((b - b_lo) * 64 + ch * 8) * p.P + pp : ch * 8 * kRawPitch + r;
                }
            }
        }
        // ---- staging copies of a stage
        // row mode: chunk column j of rows co = (t >> 4) + 32 i
        const int j = t & 15;
        long long rsrc = -1;
        // slab mode: 16-byte chunks t + 512 i of the nimg slabs
        int s_dst[4];
        long long s_src[4];
        if (!SLAB) {
            const int h = hlo + 16 * j;
            if (16 * j < p.RQ && h >= 0 && h < p.total) {
                const int b = h / p.HP, pp = h - b * p.HP;
                if (pp < p.P) rsrc = static_cast<long long>(b) * p.Cout * p.P + pp;
            }
        } else {
            const int per_img = 4 * p.P;                     // 64 * P / 16
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int idx = t + kX * i;
                s_dst[i] = -1;
                s_src[i] = -1;
                if (idx < p.nimg * per_img) {
                    const int img = idx / per_img, k = idx - img * per_img;
                    s_dst[i] = img * 64 * p.P + 16 * k;
                    if (b_lo + img < p.B) s_src[i] = static_cast<long long>(b_lo + img) * p.Cout * p.P + 16 * k;
                }
            }
        }
        auto issue_raw = [&](int c) {
            unsigned char *raw = raw_s + (c & 1) * p.raw_bytes;
            if (!SLAB) {
                if (16 * j < p.RQ) {
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int co = (t >> 4) + 32 * i;
                        const bool v = rsrc >= 0;
                        cp_async16(raw + co * kRawPitch + 16 * j,
                                   v ? p.codes + rsrc + static_cast<long long>(c * 64 + co) * p.P : p.codes, v);
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (s_dst[i] >= 0) {
                        const bool v = s_src[i] >= 0;
                        cp_async16(raw + s_dst[i], v ? p.codes + s_src[i] + static_cast<long long>(c) * 64 * p.P : p.codes, v);
                    }
                }
            }
            mbar_arrive_on_cp_async(&pipe.raw_full[c & 1]);
        };
        const int stride = SLAB ? p.P : kRawPitch;
        bool ok = true;
        issue_raw(0);
        if (nch > 1) issue_raw(1);
        for (int c = 0; c < nch; ++c) {
            ok = ok && mbar_wait(&pipe.raw_full[c & 1], (c >> 1) & 1, p.err_flag);
            const int qb = p.nq == 2 ? (c & 1) : 0, qu = p.nq == 2 ? (c >> 1) : c;   // copy set and its earlier uses
            if (qu > 0) ok = ok && mbar_wait(&pipe.qt_empty[qb], (qu - 1) & 1, p.err_flag);
            unsigned char *qtb = qt + qb * 3 * copy_bytes;
            const unsigned char *raw = raw_s + (c & 1) * p.raw_bytes;
#pragma unroll
            for (int pass = 0; pass < 4; ++pass) {
                const int r = (t & 63) + 64 * pass;
                if (r < p.RQ) {
                    uint4 e = make_uint4(0u, 0u, 0u, 0u);
                    if (src_off[pass] >= 0) {
                        const unsigned char *s = raw + src_off[pass];
                        const unsigned w0 = s[0] | (s[stride] << 8) | (s[2 * stride] << 16) | (s[3 * stride] << 24);
                        const unsigned w1 = s[4 * stride] | (s[5 * stride] << 8) | (s[6 * stride] << 16) | (s[7 * stride] << 24);
                        e = expand8(make_uint2(w0, w1));
                    }
                    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
                    const unsigned o = swz(r, ch);
                    *reinterpret_cast<uint4 *>(qtb + copy_bytes + o) = e;
                    *reinterpret_cast<uint4 *>(qtb + o) = ((zmask >> pass) & 1u) ? z : e;
                    *reinterpret_cast<uint4 *>(qtb + 2 * copy_bytes + o) = ((zmask >> (4 + pass)) & 1u) ? z : e;
                }
            }
            fence_async_proxy();
            mbar_arrive(&pipe.qt_full[qb]);
            if (c + 2 < nch) {
                asm volatile("bar.sync 1, %0;" ::"n"(kX) : "memory");   // everyone is done with this buffer
                issue_raw(c + 2);
            }
        }
        // ---------------- epilogue: lanes = input channels, columns = rows h. Warp w takes lane
        // quarter w % 4 and the 32 columns w / 4 of every accumulator.
        if (mbar_wait(&pipe.acc, 0, p.err_flag)) {
            tc_fence_after();
            const float delta = *p.delta_p;
            const int q = warp & 3, cg = warp >> 2;
#pragma unroll 1
            for (int m = 0; m < MT; ++m) {
                const int ci = (m0 + m) * 128 + q * 32 + lane;
                unsigned v[32];
                tmem_ld32(tmem_d + (static_cast<unsigned>(q * 32) << 16) + m * 128 + cg * 32, v);
                const int hfirst = h0 + cg * 32;
                if (ci < p.Cin && hfirst < p.total) store_run<MODE>(p, v, delta, ci, hfirst);
            }
        }
    } else if (warp == kXW) {
        if (lane == 0) {
            constexpr unsigned idesc = make_idesc(128, 128, false, false);
            const unsigned qt_addr = smem_u32(qt), a_addr = smem_u32(a_s);
            bool ok = true;
            int ia = 0;
            for (int c = 0; c < nch && ok; ++c) {
                const int qb = p.nq == 2 ? (c & 1) : 0, qu = p.nq == 2 ? (c >> 1) : c;
                ok = mbar_wait(&pipe.qt_full[qb], qu & 1, p.err_flag);
                fence_async_proxy();
                tc_fence_after();
                for (int tap = 0; tap < 9 && ok; ++tap) {
                    const int ky = tap / 3, kx = tap - ky * 3;
                    const int row = p.HL + (1 - ky) * p.W + (1 - kx);          // source row of the tile's row 0
                    const unsigned long long bd = make_desc(qt_addr + (qb * 3 + kx) * copy_bytes + row * 128, 16, 1024);
                    for (int m = 0; m < MT && ok; ++m, ++ia) {
                        const int sa = ia % kNA;
                        ok = mbar_wait(&pipe.a_full[sa], (ia / kNA) & 1, p.err_flag);
                        tc_fence_after();
                        const unsigned long long ad = make_desc(a_addr + sa * kTile, 16, 1024);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_bf16(tmem_d + m * 128, ad + 2 * k, bd + 2 * k, idesc, (c > 0 || tap > 0 || k > 0) ? 1u : 0u);
                        mma_commit(&pipe.a_empty[sa]);
                    }
                }
                mma_commit(&pipe.qt_empty[qb]);
            }
            mma_commit(&pipe.acc);
        }
    } else if (lane == 0) {
        // weight tiles in the order the MMAs use them
        bool ok = true;
        int ia = 0;
        for (int c = 0; c < nch && ok; ++c)
            for (int tap = 0; tap < 9 && ok; ++tap)
                for (int m = 0; m < MT && ok; ++m, ++ia) {
                    const int sa = ia % kNA;
                    ok = mbar_wait(&pipe.a_empty[sa], ((ia / kNA) & 1) ^ 1, p.err_flag);
                    if (ok)
                        bulk_load(a_s + sa * kTile,
                                  p.Wimg + (static_cast<long long>(c * 9 + tap) * p.mt_pad + m0 + m) * (kTile / 2),
                                  kTile, &pipe.a_full[sa]);
                }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kXW) {
        __syncwarp();
        tmem_dealloc(tmem_d, MT * 128);
    }
}

// weights [Cout][Cin][3][3] -> tiles [Cout/64][tap][mt_pad] of [128 ci][64 co] bf16 in the
// swizzled layout the MMA reads (zero beyond Cin); one thread per 16-byte chunk
__global__ void __launch_bounds__(256) w_images_dx_kernel(const __nv_bfloat16 *__restrict__ W, __nv_bfloat16 *__restrict__ out,
                                                          int Cout, int Cin, int mt_pad, long long nchunks) {
    chain_wait();        // launched chained: earlier kernels' writes are visible from here on
    chain_release();
    const unsigned short *w = reinterpret_cast<const unsigned short *>(W);
    for (long long idx = blockIdx.x * 256ll + threadIdx.x; idx < nchunks; idx += gridDim.x * 256ll) {
        const long long img = idx >> 10;
        const int within = static_cast<int>(idx & 1023), r = within & 127, ch = within >> 7;
        const int m = static_cast<int>(img % mt_pad), tap = static_cast<int>((img / mt_pad) % 9);
        const int c = static_cast<int>(img / (9ll * mt_pad));
        const int ci = m * 128 + r;
        unsigned short h[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int co = c * 64 + ch * 8 + e;
            h[e] = (ci < Cin && co < Cout) ? __ldg(w + (static_cast<long long>(co) * Cin + ci) * 9 + tap) : 0;
        }
        *reinterpret_cast<uint4 *>(reinterpret_cast<unsigned char *>(out) + img * kTile + swz(r, ch)) =
            make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
    }
}

template <int MT, int MODE>
int run_s(dbp_ctx *ctx, const Sx3P &p, dim3 grid, size_t smem) {
    if (cudaFuncSetAttribute(tc3_dx_shift_kernel<MT, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem)) != cudaSuccess)
        return DBP_ECUDA;
    if (launch_chained(tc3_dx_shift_kernel<MT, MODE>, grid, dim3(kThreadsS), smem, ctx->stream, p) != cudaSuccess) return DBP_ECUDA;
    return cuda_ok(cudaGetLastError());
}
template <int MT>
int run_mode(dbp_ctx *ctx, const Sx3P &p, int mode, dim3 grid, size_t smem) {
    return mode == 0 ? run_s<MT, 0>(ctx, p, grid, smem) : mode == 1 ? run_s<MT, 1>(ctx, p, grid, smem)
                                                                     : run_s<MT, 2>(ctx, p, grid, smem);
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

}  // namespace

// DBP_EUNSUPPORTED: the shape does not fit this kernel (the caller uses the generic one)
int launch_tc3_dx_shift(dbp_ctx *ctx, const int8_t *codes, const void *W, const float *delta_p,
                        const ConvShape &s, void *dX, bool dx_bf16, int *err_flag) {
    const long long P = s.H * s.W;
    if (s.Cout % 64 != 0 || s.Cin % 8 != 0 || s.W > 63 || s.W < 2 || P > (1 << 20)) return DBP_EUNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(dX) & 31u) != 0 || (reinterpret_cast<uintptr_t>(codes) & 15u) != 0) return DBP_EUNSUPPORTED;
    Sx3P p{};
    p.codes = codes; p.delta_p = delta_p; p.dX = dX; p.dx_f32 = dx_bf16 ? 0 : 1;
    p.B = static_cast<int>(s.B); p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.W = static_cast<int>(s.W); p.P = static_cast<int>(P);
    p.err_flag = err_flag;
    const int mode = P % 16 == 0 ? 0 : P % 4 == 0 ? 1 : 2;
    const int halo = p.W + 1;
    if (mode == 0) {
        p.HL = round_up(halo, 16);
        p.HP = p.P + round_up(halo, 16);
    } else {
        p.HL = halo;
        p.HP = mode == 1 ? round_up(p.P + halo, 4) : p.P + halo;
    }
    p.RQ = round_up(p.HL + 128 + halo, 8);
    if (p.RQ > 256) return DBP_EUNSUPPORTED;
    const long long total = static_cast<long long>(s.B) * p.HP;
    if (total >= (1ll << 30)) return DBP_EUNSUPPORTED;
    p.total = static_cast<int>(total);
    if (mode == 0) {
        p.raw_bytes = 64 * kRawPitch;
        p.nimg = 0;
    } else {
        if ((static_cast<long long>(s.Cout) * P) % 16 != 0) return DBP_EUNSUPPORTED;
        p.nimg = (p.RQ - 1 + p.HP - 1) / p.HP + 1;
        if (static_cast<long long>(p.nimg) * 4 * P > 4 * kX) return DBP_EUNSUPPORTED;
        p.raw_bytes = round_up(p.nimg * 64 * p.P, 16);
    }
    const int mt_total = static_cast<int>((s.Cin + 127) / 128);
    const int tiles = (p.total + 127) / 128;
    // several accumulators per CTA share one expansion of the codes. A CTA costs about one unit for
    // the expansion and one per accumulator, and the grid runs in waves of one CTA per SM: take the
    // count with the least waves x cost (ties: fewer accumulators, more CTAs)
    int mt = 1;
    long long best = -1;
    for (int cand = 1; cand <= 4; cand <<= 1) {
        if (cand > 1 && cand > mt_total) break;
        const long long ctas = static_cast<long long>(tiles) * ((mt_total + cand - 1) / cand);
        const long long cost = ((ctas + ctx->sm_count - 1) / ctx->sm_count) * (1 + cand);
        if (best < 0 || cost < best) { best = cost; mt = cand; }
    }
    const int gy = (mt_total + mt - 1) / mt;
    p.mt_pad = gy * mt;
    const size_t smem1 = static_cast<size_t>(kNA) * kTile + 3 * static_cast<size_t>(p.RQ) * 128 + 2 * static_cast<size_t>(p.raw_bytes) + 1024;
    if (smem1 > 227 * 1024) return DBP_EUNSUPPORTED;
    p.nq = (p.Cout > 64 && smem1 + 3 * static_cast<size_t>(p.RQ) * 128 <= 226 * 1024) ? 2 : 1;
    const size_t smem = smem1 + (p.nq - 1) * 3 * static_cast<size_t>(p.RQ) * 128;
    const long long nchunks = static_cast<long long>(p.Cout / 64) * 9 * p.mt_pad * 1024;
    int rc = ws_reserve(ctx, ctx->w_taps, static_cast<size_t>(nchunks) * 16);
    if (rc) return rc;
    __nv_bfloat16 *wimg = static_cast<__nv_bfloat16 *>(ctx->w_taps.ptr);
    {
        long long blocks = (nchunks + 255) / 256;
        if (blocks > ctx->sm_count * 8) blocks = ctx->sm_count * 8;
        if ((rc = cuda_ok(launch_chained(w_images_dx_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, ctx->stream,
                                         static_cast<const __nv_bfloat16 *>(W), wimg, p.Cout, p.Cin, p.mt_pad, nchunks))))
            return rc;
    }
    p.Wimg = wimg;
    dim3 grid(static_cast<unsigned>(tiles), static_cast<unsigned>(gy));
    return mt == 4 ? run_mode<4>(ctx, p, mode, grid, smem) : mt == 2 ? run_mode<2>(ctx, p, mode, grid, smem)
                                                                      : run_mode<1>(ctx, p, mode, grid, smem);
}

}  // namespace dbp
