// Sparse input-gradient product dX = delta~ * W (Eq. (qda) and its convolutional analogue),
// gather form, weights streamed through shared memory.
//
// One CTA owns a tile of output positions of one image (3x3) or a run of flattened
// (image, position) rows (1x1 / linear) and a chunk of CI_T input channels. It loops over
// chunks of CC output channels: the chunk's weights W[co][tap][ci-chunk] and code bytes are
// staged in shared memory; per input position the non-zero codes of the chunk are compacted
// (warp ballot + prefix popcount) into a short list of (weight-row offset, code) entries;
// then every warp walks, for each of its output positions, the lists of the (up to 9)
// neighbouring input positions: one shared load of the weight vector and VG FMAs per lane
// and per non-zero code. Accumulators stay in registers across all chunks; Delta is applied
// once at the end and the tile leaves through shared memory so that stores are coalesced.
#include "dbp_internal.cuh"

namespace dbp {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kWarps = 8;
constexpr int kCC = 32;   // output channels per chunk (one ballot)

struct Dx2Params {
    const int8_t *codes;   // [B][Cout][H][W]
    const void *w_taps;    // [Cout][KK][Cin], fp32 or bf16
    const float *delta_p;
    void *dX;
    int B, Cin, Cout, H, W;
    int TH, TW, tiles_y, tiles_x;   // 3x3: spatial tile; 1x1: TH = 1, TW = positions per tile
    int plane_stride;               // bytes per output channel of the shared code tile
    long long total_rows;           // 1x1: B * H * W
};

template <int BYTES>
struct LdsVec;
template <>
struct LdsVec<4> { using T = unsigned; };
template <>
struct LdsVec<8> { using T = uint2; };
template <>
struct LdsVec<16> { using T = uint4; };

// fp32 words / packed bf16 pairs -> VG floats
template <typename WT, int LB>
struct Unpack;
template <int LB>
struct Unpack<float, LB> {
    static constexpr int VG = LB / 4;
    __device__ static void get(const unsigned *w, float (&f)[VG]) {
#pragma unroll
        for (int i = 0; i < VG; ++i) f[i] = __uint_as_float(w[i]);
    }
};
template <int LB>
struct Unpack<__nv_bfloat16, LB> {
    static constexpr int VG = LB / 2;
    __device__ static void get(const unsigned *w, float (&f)[VG]) {
#pragma unroll
        for (int i = 0; i < VG / 2; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc, bool valid) {
    const unsigned d = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    const int n = valid ? 16 : 0;   // src-size 0: the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(d), "l"(gsrc), "r"(n));
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}

// KS: 1 or 3. LB: bytes of weights each lane loads per entry. NPW: output positions per warp.
template <int KS, int LB, int NPW, typename WT, typename OutT>
__global__ void __launch_bounds__(kWarps * 32, 2) conv_dx2_kernel(const Dx2Params p) {
    constexpr int PAD = (KS - 1) / 2;
    constexpr int KK = KS * KS;
    constexpr int ES = sizeof(WT);
    constexpr int VG = LB / ES;            // input channels per lane
    constexpr int CI_T = 32 * VG;
    constexpr int ROWB = 32 * LB;          // bytes of one weight row (one co, one tap)
    constexpr int PT = kWarps * NPW;       // output positions per tile
    using Vec = typename LdsVec<LB>::T;

    extern __shared__ __align__(16) unsigned char smem[];
    const int TWp = p.TW + 2 * PAD, THp = p.TH + 2 * PAD;
    const int nhp = THp * TWp;             // input positions (with halo) of the tile
    unsigned char *w_s = smem;                                             // [CC*KK][ROWB]
    unsigned *lists = reinterpret_cast<unsigned *>(w_s + kCC * KK * ROWB); // [nhp][CC]
    int8_t *codes_s = reinterpret_cast<int8_t *>(lists + static_cast<size_t>(nhp) * kCC);  // [CC][plane_stride]
    unsigned char *cnt = reinterpret_cast<unsigned char *>(codes_s + kCC * p.plane_stride);  // [nhp]
    float *stage = reinterpret_cast<float *>(smem);                        // reused at the end
    __shared__ long long code_base[KS == 1 ? kWarps * NPW : 1];   // 1x1: offset of (image, position) in a [B][C][P] tensor, channel 0, C = Cout
    __shared__ long long out_base[KS == 1 ? kWarps * NPW : 1];    // the same with C = Cin

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int ci0 = blockIdx.y * CI_T;
    // tile origin
    int b = 0, y0 = 0, x0 = 0;
    long long r0 = 0;
    int npos;
    if (KS == 1) {
        r0 = static_cast<long long>(blockIdx.x) * PT;
        const long long left = p.total_rows - r0;
        npos = left < PT ? static_cast<int>(left) : PT;
    } else {
        const int tpi = p.tiles_y * p.tiles_x;
        b = blockIdx.x / tpi;
        const int t = blockIdx.x - b * tpi;
        y0 = (t / p.tiles_x) * p.TH;
        x0 = (t % p.tiles_x) * p.TW;
        npos = p.TH * p.TW;
    }
    const long long P = static_cast<long long>(p.H) * p.W;
    if (KS == 1) {
        for (int i = threadIdx.x; i < PT; i += kWarps * 32) {
            const long long r = r0 + i;
            const long long bb = r / P, pp = r - bb * P;
            code_base[i] = bb * p.Cout * P + pp;
            out_base[i] = bb * p.Cin * P + pp;
        }
    }

    float acc[NPW][VG];
#pragma unroll
    for (int i = 0; i < NPW; ++i)
#pragma unroll
        for (int v = 0; v < VG; ++v) acc[i][v] = 0.f;

    // halo'd index of my output positions (position i*8 + warp), -1 when outside the image
    int hp_of[NPW];
#pragma unroll
    for (int i = 0; i < NPW; ++i) {
        const int pos = i * kWarps + warp;
        if (KS == 1) {
            hp_of[i] = pos < npos ? pos : -1;
        } else {
            const int ly = pos / p.TW, lx = pos - ly * p.TW;
            hp_of[i] = (pos < npos && y0 + ly < p.H && x0 + lx < p.W) ? (ly + PAD) * TWp + lx + PAD : -1;
        }
    }

    const unsigned char *wt = static_cast<const unsigned char *>(p.w_taps);
    for (int co0 = 0; co0 < p.Cout; co0 += kCC) {
        __syncthreads();   // previous chunk fully consumed
        // ---- stage weights of the chunk: rows (co_local, tap), 16-byte pieces
        constexpr int PIECES = ROWB / 16;
        for (int i = threadIdx.x; i < kCC * KK * PIECES; i += kWarps * 32) {
            const int row = i / PIECES, piece = i - row * PIECES;
            const int co = co0 + row / KK;
            const int ci = ci0 + piece * (16 / ES);
            const bool ok = co < p.Cout && ci < p.Cin;
            const long long src = ((static_cast<long long>(co0) * KK + row) * p.Cin + ci) * ES;
            cp_async16(w_s + row * ROWB + piece * 16, ok ? wt + src : wt, ok);
        }
        // ---- stage code bytes of the chunk
        if (KS == 1) {
            for (int c = warp; c < kCC; c += kWarps) {
                const int co = co0 + c;
                for (int hp = lane; hp < nhp; hp += 32) {
                    int8_t code = 0;
                    if (co < p.Cout && hp < npos) code = p.codes[code_base[hp] + co * P];
                    codes_s[c * p.plane_stride + hp] = code;
                }
            }
        } else {
            for (int row = warp; row < kCC * THp; row += kWarps) {
                const int c = row / THp, ty = row - c * THp;
                const int co = co0 + c, y = y0 + ty - PAD;
                const bool row_ok = co < p.Cout && y >= 0 && y < p.H;
                const int8_t *src = p.codes + ((static_cast<long long>(b) * p.Cout + co) * p.H + y) * p.W;
                for (int tx = lane; tx < TWp; tx += 32) {
                    const int x = x0 + tx - PAD;
                    codes_s[c * p.plane_stride + ty * TWp + tx] = (row_ok && x >= 0 && x < p.W) ? src[x] : int8_t(0);
                }
            }
        }
        cp_async_wait_all();
        __syncthreads();
        // ---- compact: one warp per input position, one lane per output channel of the chunk
        for (int hp = warp; hp < nhp; hp += kWarps) {
            const int code = codes_s[lane * p.plane_stride + hp];
            const unsigned m = __ballot_sync(kFull, code != 0);
            if (code != 0) {
                const unsigned fb = __float_as_uint(static_cast<float>(code)) & 0xffff0000u;  // exact: |code| <= 127
                lists[hp * kCC + __popc(m & ((1u << lane) - 1u))] = fb | static_cast<unsigned>(lane * (KK * ROWB / 16));
            }
            if (lane == 0) cnt[hp] = static_cast<unsigned char>(__popc(m));
        }
        __syncthreads();
        // ---- gather
#pragma unroll
        for (int i = 0; i < NPW; ++i) {
            const int hp = hp_of[i];
            if (hp < 0) continue;       // warp-uniform
#pragma unroll
            for (int ky = 0; ky < KS; ++ky) {
#pragma unroll
                for (int kx = 0; kx < KS; ++kx) {
                    const int nb = hp + (PAD - ky) * TWp + (PAD - kx);
                    const int n = cnt[nb];
                    const unsigned *lp = lists + nb * kCC;
                    const unsigned char *wtap = w_s + (ky * KS + kx) * ROWB + lane * LB;
                    for (int e = 0; e < n; ++e) {
                        const unsigned ent = lp[e];
                        const float c = __uint_as_float(ent & 0xffff0000u);
                        const Vec raw = *reinterpret_cast<const Vec *>(wtap + ((ent & 0xffffu) << 4));
                        float w[VG];
                        Unpack<WT, LB>::get(reinterpret_cast<const unsigned *>(&raw), w);
#pragma unroll
                        for (int v = 0; v < VG; ++v) acc[i][v] = fmaf(c, w[v], acc[i][v]);
                    }
                }
            }
        }
    }
    __syncthreads();
    // ---- Delta, transpose through shared memory, coalesced stores
    const float delta = *p.delta_p;
    constexpr int SS = PT + 1;
#pragma unroll
    for (int i = 0; i < NPW; ++i) {
        const int pos = i * kWarps + warp;
#pragma unroll
        for (int v = 0; v < VG; ++v) stage[(lane * VG + v) * SS + pos] = acc[i][v] * delta;
    }
    __syncthreads();
    OutT *out = static_cast<OutT *>(p.dX);
    for (int i = threadIdx.x; i < CI_T * PT; i += kWarps * 32) {
        const int c = i / PT, pos = i - c * PT;
        const int ci = ci0 + c;
        if (ci >= p.Cin || pos >= npos) continue;
        long long dst;
        if (KS == 1) {
            dst = out_base[pos] + ci * P;
        } else {
            const int ly = pos / p.TW, lx = pos - ly * p.TW;
            const int y = y0 + ly, x = x0 + lx;
            if (y >= p.H || x >= p.W) continue;
            dst = ((static_cast<long long>(b) * p.Cin + ci) * p.H + y) * p.W + x;
        }
        out[dst] = static_cast<OutT>(stage[c * SS + pos]);
    }
}

template <int KS, int LB, int NPW, typename WT, typename OutT>
int launch_one(dbp_ctx *ctx, Dx2Params &p, const ConvShape &s) {
    constexpr int PAD = (KS - 1) / 2;
    constexpr int KK = KS * KS;
    constexpr int VG = LB / static_cast<int>(sizeof(WT));
    constexpr int CI_T = 32 * VG;
    constexpr int PT = kWarps * NPW;
    if (KS == 1) {
        p.TH = 1;
        p.TW = PT;
        p.total_rows = s.B * s.H * s.W;
    } else {
        int tw = static_cast<int>(s.W < PT ? s.W : PT);
        int th_max = PT / tw;
        if (th_max > s.H) th_max = static_cast<int>(s.H);
        const int ty = static_cast<int>((s.H + th_max - 1) / th_max);
        p.TW = tw;
        p.TH = static_cast<int>((s.H + ty - 1) / ty);
        p.tiles_y = ty;
        p.tiles_x = static_cast<int>((s.W + tw - 1) / tw);
    }
    const int nhp = (p.TH + 2 * PAD) * (p.TW + 2 * PAD);
    int ps = (nhp + 3) & ~3;
    if (((ps / 4) & 1) == 0) ps += 4;      // odd word stride: the 32 lanes hit 32 banks
    p.plane_stride = ps;
    size_t work = static_cast<size_t>(kCC) * KK * 32 * LB + static_cast<size_t>(nhp) * kCC * 4 +
                  static_cast<size_t>(kCC) * ps + nhp + 16;
    const size_t stage = static_cast<size_t>(CI_T) * (PT + 1) * 4;
    const size_t smem = work > stage ? work : stage;
    if (smem > 220 * 1024) return DBP_EUNSUPPORTED;
    auto kern = conv_dx2_kernel<KS, LB, NPW, WT, OutT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return DBP_ECUDA;
    const long long tiles = KS == 1 ? (p.total_rows + PT - 1) / PT
                                    : s.B * p.tiles_y * p.tiles_x;
    dim3 grid(static_cast<unsigned>(tiles), static_cast<unsigned>((s.Cin + CI_T - 1) / CI_T));
    note_launch();
    kern<<<grid, kWarps * 32, smem, ctx->stream>>>(p);
    return cuda_ok(cudaGetLastError());
}

template <int KS, typename WT, typename OutT>
int launch_by_width(dbp_ctx *ctx, Dx2Params &p, const ConvShape &s) {
    const long long row_bytes = s.Cin * static_cast<long long>(sizeof(WT));
    // bytes per lane: the widest load that the layer's channel count fills
    if (KS == 3) {   // 3x3 keeps all nine taps of a chunk resident: narrower rows
        if (row_bytes >= 256) return launch_one<KS, 8, 16, WT, OutT>(ctx, p, s);
        return launch_one<KS, 4, 16, WT, OutT>(ctx, p, s);
    }
    if (row_bytes >= 512) return launch_one<KS, 16, 16 / (16 / static_cast<int>(sizeof(WT)) / 4), WT, OutT>(ctx, p, s);
    if (row_bytes >= 256) return launch_one<KS, 8, 16, WT, OutT>(ctx, p, s);
    return launch_one<KS, 4, 16, WT, OutT>(ctx, p, s);
}

}  // namespace

// Returns DBP_EUNSUPPORTED when the shape does not fit this kernel (the caller then uses
// the generic one): weight rows must be 16-byte multiples.
int launch_conv_dx_streamed(dbp_ctx *ctx, const int8_t *codes, const void *w_taps, int w_dtype,
                            const float *delta_p, const ConvShape &s, void *dX, bool dx_bf16) {
    const long long es = w_dtype == DBP_F32 ? 4 : 2;
    if ((s.Cin * es) % 16 != 0) return DBP_EUNSUPPORTED;
    Dx2Params p;
    p.codes = codes; p.w_taps = w_taps; p.delta_p = delta_p; p.dX = dX;
    p.B = static_cast<int>(s.B); p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.H = static_cast<int>(s.H); p.W = static_cast<int>(s.W);
    p.tiles_y = p.tiles_x = 1;
    p.total_rows = 0;
    if (w_dtype == DBP_F32) {
        if (dx_bf16) return DBP_EUNSUPPORTED;
        return s.k == 1 ? launch_by_width<1, float, float>(ctx, p, s) : launch_by_width<3, float, float>(ctx, p, s);
    }
    if (dx_bf16)
        return s.k == 1 ? launch_by_width<1, __nv_bfloat16, __nv_bfloat16>(ctx, p, s)
                        : launch_by_width<3, __nv_bfloat16, __nv_bfloat16>(ctx, p, s);
    return s.k == 1 ? launch_by_width<1, __nv_bfloat16, float>(ctx, p, s)
                    : launch_by_width<3, __nv_bfloat16, float>(ctx, p, s);
}

}  // namespace dbp
