// Sparse weight-gradient product dW = delta~^T * X (Eq. (qdw) and its convolutional analogue).
//
// One CTA owns a block of dW -- CO_T output channels x CI_T input channels x all taps -- in
// registers and streams position tiles of its share of the batch through shared memory:
//   * the X tile, transposed to [position (with halo)][ci] in 16-byte chunks (XOR-swizzled so
//     that both the transposing stores and the row loads are bank-conflict free);
//   * the code bytes [co][position] of its output channels.
// A warp owns CPG output channels. For each it ballots "code != 0" over 32 positions at a
// time and walks the set bits: per non-zero code and tap, one shared load of VG consecutive
// input channels of the shifted position and VG FMAs per lane. Delta is applied once, at the
// end, when the partial block is added to dW with fp32 reductions (CTAs that share an output
// block split the batch between them).
#include "dbp_internal.cuh"

namespace dbp {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;

struct Dw2Params {
    const int8_t *codes;   // [B][Cout][H][W]
    const void *X;         // [B][Cin][H][W]
    const float *delta_p;
    float *dW;             // [Cout][Cin][KK]
    int B, Cin, Cout, H, W;
    int TH, TW, tiles_y, tiles_x;   // 3x3: spatial tile; 1x1: TH = 1, TW = rows per tile
    int pt_pad;                     // tile positions rounded up to 32
    long long total_rows;           // 1x1: B * H * W
    long long ntiles;
    int splits;
};

template <int BYTES>
struct Raw;
template <>
struct Raw<4> { using T = unsigned; };
template <>
struct Raw<8> { using T = uint2; };
template <>
struct Raw<16> { using T = uint4; };

template <typename XT, int LB>
struct Lanes;
template <int LB>
struct Lanes<float, LB> {
    static constexpr int VG = LB / 4;
    __device__ static void get(const unsigned *w, float (&f)[VG]) {
#pragma unroll
        for (int i = 0; i < VG; ++i) f[i] = __uint_as_float(w[i]);
    }
};
template <int LB>
struct Lanes<__nv_bfloat16, LB> {
    static constexpr int VG = LB / 2;
    __device__ static void get(const unsigned *w, float (&f)[VG]) {
#pragma unroll
        for (int i = 0; i < VG / 2; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

__device__ __forceinline__ unsigned ld_bits(const float *p) { return __float_as_uint(__ldg(p)); }
__device__ __forceinline__ unsigned ld_bits(const __nv_bfloat16 *p) {
    return __ldg(reinterpret_cast<const unsigned short *>(p));
}

// 16 bytes = 4 fp32 or 8 bf16 channels of one position, gathered with channel stride cs
__device__ __forceinline__ uint4 gather_chunk(const float *src, long long cs, int nvalid) {
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (nvalid > 0) v.x = ld_bits(src);
    if (nvalid > 1) v.y = ld_bits(src + cs);
    if (nvalid > 2) v.z = ld_bits(src + 2 * cs);
    if (nvalid > 3) v.w = ld_bits(src + 3 * cs);
    return v;
}
__device__ __forceinline__ uint4 gather_chunk(const __nv_bfloat16 *src, long long cs, int nvalid) {
    unsigned h[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) h[j] = (j < nvalid) ? ld_bits(src + j * cs) : 0u;
    return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
}

template <int KS, int LB, int CPG, typename XT>
__global__ void __launch_bounds__(kThreads) conv_dw2_kernel(const Dw2Params p) {
    constexpr int PAD = (KS - 1) / 2;
    constexpr int KK = KS * KS;
    constexpr int ES = sizeof(XT);
    constexpr int VG = LB / ES;
    constexpr int CI_T = 32 * VG;
    constexpr int ROWB = 32 * LB;          // bytes of one position's channel row
    constexpr int CHUNKS = ROWB / 16;
    constexpr int CPC = 16 / ES;           // channels per 16-byte chunk
    constexpr int CO_T = kWarps * CPG;
    using RawT = typename Raw<LB>::T;

    extern __shared__ __align__(16) unsigned char smem[];
    const int TWp = p.TW + 2 * PAD, THp = p.TH + 2 * PAD;
    const int nhp = THp * TWp;
    unsigned char *Xs = smem;                                                    // [nhp][ROWB]
    int8_t *ct = reinterpret_cast<int8_t *>(Xs + static_cast<size_t>(nhp) * ROWB);   // [CO_T][pt_pad]
    unsigned short *hpos = reinterpret_cast<unsigned short *>(ct + static_cast<size_t>(CO_T) * p.pt_pad);  // [pt_pad]
    long long *xbase = reinterpret_cast<long long *>(
        (reinterpret_cast<uintptr_t>(hpos + p.pt_pad) + 7) & ~uintptr_t(7));      // [pt_pad] (1x1 only)
    long long *cbase = xbase + p.pt_pad;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int co0 = blockIdx.x * CO_T, ci0 = blockIdx.y * CI_T;
    const long long P = static_cast<long long>(p.H) * p.W;
    const XT *X = static_cast<const XT *>(p.X);
    const int lane_off = lane * LB;        // my byte offset inside a channel row (before swizzle)

    float acc[CPG][KK][VG];
#pragma unroll
    for (int a = 0; a < CPG; ++a)
#pragma unroll
        for (int t = 0; t < KK; ++t)
#pragma unroll
            for (int v = 0; v < VG; ++v) acc[a][t][v] = 0.f;

    const int tpi = p.tiles_y * p.tiles_x;
    for (long long tile = blockIdx.z; tile < p.ntiles; tile += p.splits) {
        int b = 0, y0 = 0, x0 = 0, npos;
        long long r0 = 0;
        if (KS == 1) {
            r0 = tile * p.TW;
            const long long left = p.total_rows - r0;
            npos = left < p.TW ? static_cast<int>(left) : p.TW;
        } else {
            b = static_cast<int>(tile / tpi);
            const int t = static_cast<int>(tile - static_cast<long long>(b) * tpi);
            y0 = (t / p.tiles_x) * p.TH;
            x0 = (t % p.tiles_x) * p.TW;
            npos = p.TH * p.TW;
        }
        __syncthreads();   // previous tile fully consumed
        // ---- per-position tables
        for (int i = threadIdx.x; i < p.pt_pad; i += kThreads) {
            if (KS == 1) {
                const long long r = r0 + i;
                const long long bb = r / P, pp = r - bb * P;
                xbase[i] = bb * p.Cin * P + pp;
                cbase[i] = bb * p.Cout * P + pp;
                hpos[i] = static_cast<unsigned short>(i);
            } else {
                const int ly = i / p.TW, lx = i - ly * p.TW;
                const bool ok = i < npos && y0 + ly < p.H && x0 + lx < p.W;
                hpos[i] = ok ? static_cast<unsigned short>((ly + PAD) * TWp + lx + PAD) : 0xffff;
            }
        }
        if (KS == 1) __syncthreads();
        // ---- X tile, transposed: item = (16-byte channel chunk, position)
        if (KS == 1) {
            for (int c16 = warp; c16 < CHUNKS; c16 += kWarps) {
                const int ci = ci0 + c16 * CPC;
                const int nvalid = p.Cin - ci;
                for (int hp = lane; hp < nhp; hp += 32) {
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (hp < npos && nvalid > 0) v = gather_chunk(X + xbase[hp] + ci * P, P, nvalid);
                    *reinterpret_cast<uint4 *>(Xs + static_cast<size_t>(hp) * ROWB + ((c16 ^ (hp & 7)) << 4)) = v;
                }
            }
        } else {
            for (int row = warp; row < CHUNKS * THp; row += kWarps) {
                const int c16 = row / THp, ty = row - c16 * THp;
                const int ci = ci0 + c16 * CPC;
                const int nvalid = p.Cin - ci;
                const int y = y0 + ty - PAD;
                const bool row_ok = nvalid > 0 && y >= 0 && y < p.H;
                const XT *src = X + ((static_cast<long long>(b) * p.Cin + ci) * p.H + y) * p.W;
                for (int tx = lane; tx < TWp; tx += 32) {
                    const int x = x0 + tx - PAD;
                    const int hp = ty * TWp + tx;
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (row_ok && x >= 0 && x < p.W) v = gather_chunk(src + x, P, nvalid);
                    *reinterpret_cast<uint4 *>(Xs + static_cast<size_t>(hp) * ROWB + ((c16 ^ (hp & 7)) << 4)) = v;
                }
            }
        }
        // ---- code bytes of my output channels
        for (int c = warp; c < CO_T; c += kWarps) {
            const int co = co0 + c;
            for (int i = lane; i < p.pt_pad; i += 32) {
                int8_t code = 0;
                if (co < p.Cout && i < npos) {
                    if (KS == 1) {
                        code = p.codes[cbase[i] + co * P];
                    } else {
                        const int ly = i / p.TW, lx = i - ly * p.TW;
                        const int y = y0 + ly, x = x0 + lx;
                        if (y < p.H && x < p.W)
                            code = p.codes[((static_cast<long long>(b) * p.Cout + co) * p.H + y) * p.W + x];
                    }
                }
                ct[c * p.pt_pad + i] = code;
            }
        }
        __syncthreads();
        // ---- walk the non-zero codes of my channels
#pragma unroll
        for (int a = 0; a < CPG; ++a) {
            const int8_t *row = ct + (warp * CPG + a) * p.pt_pad;
            for (int pos0 = 0; pos0 < p.pt_pad; pos0 += 32) {
                const int code = row[pos0 + lane];
                unsigned m = __ballot_sync(kFull, code != 0);
                const float cf = static_cast<float>(code);
                while (m) {
                    const int j = __ffs(m) - 1;
                    m &= m - 1;
                    const float c = __shfl_sync(kFull, cf, j);
                    const int hp = hpos[pos0 + j];
#pragma unroll
                    for (int ky = 0; ky < KS; ++ky) {
#pragma unroll
                        for (int kx = 0; kx < KS; ++kx) {
                            const int xp = hp + (ky - PAD) * TWp + (kx - PAD);
                            const int off = (((lane_off >> 4) ^ (xp & 7)) << 4) | (lane_off & 15);
                            const RawT raw = *reinterpret_cast<const RawT *>(Xs + static_cast<size_t>(xp) * ROWB + off);
                            float xv[VG];
                            Lanes<XT, LB>::get(reinterpret_cast<const unsigned *>(&raw), xv);
#pragma unroll
                            for (int v = 0; v < VG; ++v)
                                acc[a][ky * KS + kx][v] = fmaf(c, xv[v], acc[a][ky * KS + kx][v]);
                        }
                    }
                }
            }
        }
    }

    const float delta = *p.delta_p;
#pragma unroll
    for (int a = 0; a < CPG; ++a) {
        const int co = co0 + warp * CPG + a;
        if (co >= p.Cout) continue;
#pragma unroll
        for (int v = 0; v < VG; ++v) {
            const int ci = ci0 + lane * VG + v;
            if (ci >= p.Cin) continue;
#pragma unroll
            for (int t = 0; t < KK; ++t) {
                const float val = acc[a][t][v] * delta;
                if (val != 0.f) atomicAdd(p.dW + (static_cast<long long>(co) * p.Cin + ci) * KK + t, val);
            }
        }
    }
}

template <int KS, int LB, int CPG, typename XT>
int launch_one(dbp_ctx *ctx, Dw2Params &p, const ConvShape &s) {
    constexpr int PAD = (KS - 1) / 2;
    constexpr int VG = LB / static_cast<int>(sizeof(XT));
    constexpr int CI_T = 32 * VG;
    constexpr int CO_T = kWarps * CPG;
    constexpr int PT = 128;
    if (KS == 1) {
        p.TH = 1;
        p.TW = PT;
        p.total_rows = s.B * s.H * s.W;
        p.ntiles = (p.total_rows + PT - 1) / PT;
        p.tiles_y = p.tiles_x = 1;
    } else {
        int tw = static_cast<int>(s.W < PT ? s.W : PT);
        int th_max = PT / tw;
        if (th_max > s.H) th_max = static_cast<int>(s.H);
        const int ty = static_cast<int>((s.H + th_max - 1) / th_max);
        p.TW = tw;
        p.TH = static_cast<int>((s.H + ty - 1) / ty);
        p.tiles_y = ty;
        p.tiles_x = static_cast<int>((s.W + tw - 1) / tw);
        p.ntiles = s.B * p.tiles_y * p.tiles_x;
    }
    p.pt_pad = (p.TH * p.TW + 31) & ~31;
    const int nhp = (p.TH + 2 * PAD) * (p.TW + 2 * PAD);
    const size_t smem = static_cast<size_t>(nhp) * 32 * LB + static_cast<size_t>(CO_T) * p.pt_pad +
                        static_cast<size_t>(p.pt_pad) * (2 + 16) + 16;
    if (smem > 220 * 1024 || nhp >= 0xffff) return DBP_EUNSUPPORTED;
    const long long out_blocks = ((s.Cout + CO_T - 1) / CO_T) * ((s.Cin + CI_T - 1) / CI_T);
    long long splits = (2LL * ctx->sm_count) / out_blocks;
    if (splits < 1) splits = 1;
    if (splits > p.ntiles) splits = p.ntiles;
    if (splits > 65535) splits = 65535;
    p.splits = static_cast<int>(splits);
    auto kern = conv_dw2_kernel<KS, LB, CPG, XT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return DBP_ECUDA;
    dim3 grid(static_cast<unsigned>((s.Cout + CO_T - 1) / CO_T), static_cast<unsigned>((s.Cin + CI_T - 1) / CI_T),
              static_cast<unsigned>(splits));
    note_launch();
    kern<<<grid, kThreads, smem, ctx->stream>>>(p);
    return cuda_ok(cudaGetLastError());
}

template <typename XT>
int launch_by_shape(dbp_ctx *ctx, Dw2Params &p, const ConvShape &s) {
    constexpr int ES = sizeof(XT);
    const long long row_bytes = s.Cin * ES;
    // channels per lane VG = LB/ES; accumulators per lane = CPG * k*k * VG (64..72)
    if (s.k == 3) {
        if (row_bytes >= 512) return launch_one<3, 16, 8 / (16 / ES), XT>(ctx, p, s);
        if (row_bytes >= 256) return launch_one<3, 8, 8 / (8 / ES), XT>(ctx, p, s);
        return launch_one<3, 4, 8 / (4 / ES), XT>(ctx, p, s);
    }
    const bool wide = s.Cout > 64;   // more channels per warp when there are enough to fill a CTA
    if (row_bytes >= 512) return wide ? launch_one<1, 16, 64 / (16 / ES), XT>(ctx, p, s)
                                      : launch_one<1, 16, 4, XT>(ctx, p, s);
    if (row_bytes >= 256) return wide ? launch_one<1, 8, 16, XT>(ctx, p, s) : launch_one<1, 8, 4, XT>(ctx, p, s);
    return wide ? launch_one<1, 4, 16, XT>(ctx, p, s) : launch_one<1, 4, 4, XT>(ctx, p, s);
}

}  // namespace

int launch_conv_dw_streamed(dbp_ctx *ctx, const int8_t *codes, const void *X, int dtype,
                            const float *delta_p, const ConvShape &s, float *dW) {
    Dw2Params p;
    p.codes = codes; p.X = X; p.delta_p = delta_p; p.dW = dW;
    p.B = static_cast<int>(s.B); p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.H = static_cast<int>(s.H); p.W = static_cast<int>(s.W);
    p.total_rows = 0;
    if (cudaMemsetAsync(dW, 0, sizeof(float) * s.Cout * s.Cin * s.k * s.k, ctx->stream) != cudaSuccess)
        return DBP_ECUDA;
    return dtype == DBP_F32 ? launch_by_shape<float>(ctx, p, s) : launch_by_shape<__nv_bfloat16>(ctx, p, s);
}

}  // namespace dbp
