// Sparse backward products driven by the int8 NSD codes (Eqs. (qda), (qdw) and their
// convolutional analogues): only non-zero codes cost arithmetic (the p_nz * m k n term of
// Section 3.4), Delta is applied once per output, accumulation is fp32.
//
// A linear layer is the 1x1 convolution with H = W = 1 (the memory layouts coincide), so one
// pair of kernels covers linear, 1x1, 3x3 and 5x5 (the 5x5 layers of LeNet-5-like networks run here only).
#include "dbp_internal.cuh"

namespace dbp {

namespace {

constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// ------------------------------------------------------------------ weights as [Cout][tap][Cin]
__device__ __forceinline__ void store_as(float *p, float v) { *p = v; }
__device__ __forceinline__ void store_as(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T, typename O>
__global__ void weight_taps_kernel(const T *__restrict__ W, O *__restrict__ out, long long Cout,
                                   long long Cin, int KK) {
    const long long n = Cout * Cin * KK;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long ci = i % Cin;
        const long long t = (i / Cin) % KK;
        const long long co = i / (Cin * KK);
        store_as(out + i, to_f32(W[(co * Cin + ci) * KK + t]));
    }
}

// ------------------------------------------------------------------ dX (gather form)
// One CTA: one image, a TH x TW tile of output positions, a chunk of CI_T = 32*VEC input
// channels. The tile's codes (all Cout, with halo) sit in shared memory as bytes. A warp
// takes one output position at a time; lanes hold VEC consecutive input channels. For each
// tap and each group of 32 output channels the warp ballots "code != 0" and walks the set
// bits: one vector load of W[co][tap][ci..] and VEC FMAs per non-zero code.
struct DxParams {
    const int8_t *codes;
    const float *w_taps;
    const float *delta_p;
    void *dX;
    int B, Cin, Cout, H, W;
    int TH, TW, tiles_y, tiles_x;
    int plane_stride;   // bytes per output channel in the shared code tile
    int stage_stride;   // floats per input channel in the shared output tile
};

template <int VEC>
struct VecLoad;
template <>
struct VecLoad<1> {
    __device__ static void ld(const float *p, float (&w)[1]) { w[0] = __ldg(p); }
};
template <>
struct VecLoad<2> {
    __device__ static void ld(const float *p, float (&w)[2]) {
        const float2 q = __ldg(reinterpret_cast<const float2 *>(p));
        w[0] = q.x; w[1] = q.y;
    }
};
template <>
struct VecLoad<4> {
    __device__ static void ld(const float *p, float (&w)[4]) {
        const float4 q = __ldg(reinterpret_cast<const float4 *>(p));
        w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
    }
};

template <int KS, int VEC, typename OutT>
__global__ void __launch_bounds__(256) conv_dx_kernel(const DxParams p) {
    constexpr int PAD = (KS - 1) / 2;
    constexpr int KK = KS * KS;
    constexpr int CI_T = 32 * VEC;
    extern __shared__ __align__(16) unsigned char smem[];
    const int TWp = p.TW + 2 * PAD;
    const int THp = p.TH + 2 * PAD;
    const int npos = p.TH * p.TW;
    int8_t *tile = reinterpret_cast<int8_t *>(smem);
    float *stage = reinterpret_cast<float *>(smem + ((static_cast<size_t>(p.Cout) * p.plane_stride + 15) & ~size_t(15)));

    const int tiles_per_img = p.tiles_y * p.tiles_x;
    const int b = blockIdx.x / tiles_per_img;
    const int t = blockIdx.x % tiles_per_img;
    const int y0 = (t / p.tiles_x) * p.TH;
    const int x0 = (t % p.tiles_x) * p.TW;
    const int ci0 = blockIdx.y * CI_T;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // stage the code tile (zero outside the image)
    const int plane_elems = THp * TWp;
    for (int i = threadIdx.x; i < p.Cout * plane_elems; i += blockDim.x) {
        const int co = i / plane_elems;
        const int r = i - co * plane_elems;
        const int ty = r / TWp, tx = r - ty * TWp;
        const int y = y0 + ty - PAD, x = x0 + tx - PAD;
        int8_t c = 0;
        if (y >= 0 && y < p.H && x >= 0 && x < p.W)
            c = p.codes[((static_cast<long long>(b) * p.Cout + co) * p.H + y) * p.W + x];
        tile[co * p.plane_stride + r] = c;
    }
    __syncthreads();

    const float delta = *p.delta_p;
    const int ci = ci0 + lane * VEC;
    const bool ci_ok = ci < p.Cin;     // Cin % VEC == 0, so a lane's vector is all-in or all-out
    for (int pos = warp; pos < npos; pos += 8) {
        const int ly = pos / p.TW, lx = pos - ly * p.TW;
        if (y0 + ly >= p.H || x0 + lx >= p.W) continue;   // warp-uniform
        float acc[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
#pragma unroll
        for (int ky = 0; ky < KS; ++ky) {
#pragma unroll
            for (int kx = 0; kx < KS; ++kx) {
                // code position (y - ky + PAD, x - kx + PAD) in tile coordinates
                const int toff = (ly - ky + 2 * PAD) * TWp + (lx - kx + 2 * PAD);
                const int tap = ky * KS + kx;
                for (int co0 = 0; co0 < p.Cout; co0 += 32) {
                    const int co = co0 + lane;
                    const int code = (co < p.Cout) ? tile[co * p.plane_stride + toff] : 0;
                    unsigned m = __ballot_sync(kFull, code != 0);
                    const float cf = static_cast<float>(code);
                    while (m) {
                        const int j = __ffs(m) - 1;
                        m &= m - 1;
                        const float c = __shfl_sync(kFull, cf, j);
                        if (ci_ok) {
                            float w[VEC];
                            VecLoad<VEC>::ld(p.w_taps + (static_cast<long long>(co0 + j) * KK + tap) * p.Cin + ci, w);
#pragma unroll
                            for (int v = 0; v < VEC; ++v) acc[v] = fmaf(c, w[v], acc[v]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int v = 0; v < VEC; ++v) stage[(lane * VEC + v) * p.stage_stride + pos] = acc[v] * delta;
    }
    __syncthreads();

    // coalesced write of the [CI_T][TH][TW] tile
    OutT *out = static_cast<OutT *>(p.dX);
    for (int i = threadIdx.x; i < CI_T * npos; i += blockDim.x) {
        const int c = i / npos, pos = i - c * npos;
        const int ly = pos / p.TW, lx = pos - ly * p.TW;
        const int y = y0 + ly, x = x0 + lx;
        if (ci0 + c < p.Cin && y < p.H && x < p.W)
            out[((static_cast<long long>(b) * p.Cin + ci0 + c) * p.H + y) * p.W + x] =
                static_cast<OutT>(stage[c * p.stage_stride + pos]);
    }
}

// ------------------------------------------------------------------ dW (native walk)
// One CTA: 32 output channels x CI_T input channels of dW, kept in registers across all the
// position tiles the CTA visits (a slice of the batch); X tiles are staged transposed,
// [position][ci] with a 16-byte-chunk XOR swizzle, so that a lane reads 4 consecutive input
// channels of one position with one 128-bit shared load. A group of G = CI_T/4 lanes owns one
// output channel at a time and walks its non-zero codes: 9 (or 1) loads and 36 (or 4) FMAs
// per non-zero. Partial sums of the CTAs that share an output block meet through fp32 atomics.
struct DwParams {
    const int8_t *codes;
    const void *X;
    const float *delta_p;
    float *dW;
    int B, Cin, Cout, H, W;
    int TH, TW, tiles_y, tiles_x;
    int splits;
};

template <int KS, int CI_T, typename T>
__global__ void __launch_bounds__(512) conv_dw_kernel(const DwParams p) {
    constexpr int PAD = (KS - 1) / 2;
    constexpr int KK = KS * KS;
    constexpr int G = CI_T / 4;            // lanes per group: 16 or 32
    constexpr int NG = 512 / G;            // groups per CTA: 32 or 16
    constexpr int CPG = 32 / NG;           // output channels per group: 1 or 2
    extern __shared__ __align__(16) unsigned char smem[];
    const int TWp = p.TW + 2 * PAD, THp = p.TH + 2 * PAD;
    const int npos = p.TH * p.TW;
    const int npos_pad = (npos + 31) & ~31;
    float *Xs = reinterpret_cast<float *>(smem);                               // [THp*TWp][CI_T]
    int8_t *ct = reinterpret_cast<int8_t *>(smem + static_cast<size_t>(THp) * TWp * CI_T * 4);  // [32][npos_pad]

    const int co0 = blockIdx.x * 32;
    const int ci0 = blockIdx.y * CI_T;
    const int lane = threadIdx.x & 31;
    const int gl = threadIdx.x % G;        // lane inside the group
    const int grp = threadIdx.x / G;
    const int gbase = lane - gl;           // first lane of my group inside the warp
    const unsigned gmask = (G == 32) ? kFull : (0xffffu << gbase);
    const T *X = static_cast<const T *>(p.X);

    float acc[CPG][KK][4];
#pragma unroll
    for (int a = 0; a < CPG; ++a)
#pragma unroll
        for (int t = 0; t < KK; ++t)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[a][t][v] = 0.f;

    const int tiles_per_img = p.tiles_y * p.tiles_x;
    const long long ntiles = static_cast<long long>(p.B) * tiles_per_img;
    for (long long tile = blockIdx.z; tile < ntiles; tile += p.splits) {
        const int b = static_cast<int>(tile / tiles_per_img);
        const int tt = static_cast<int>(tile % tiles_per_img);
        const int y0 = (tt / p.tiles_x) * p.TH, x0 = (tt % p.tiles_x) * p.TW;
        __syncthreads();
        // X tile, transposed: item = (chunk of 4 ci, position); consecutive threads take
        // consecutive x so that each of the 4 loads is coalesced
        const int nxp = THp * TWp;
        for (int i = threadIdx.x; i < nxp * (CI_T / 4); i += 512) {
            const int c4 = i / nxp, xp = i - c4 * nxp;
            const int ty = xp / TWp, tx = xp - ty * TWp;
            const int y = y0 + ty - PAD, x = x0 + tx - PAD;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (y >= 0 && y < p.H && x >= 0 && x < p.W) {
                const int ci = ci0 + c4 * 4;
                const long long base = ((static_cast<long long>(b) * p.Cin + ci) * p.H + y) * p.W + x;
                const long long cs = static_cast<long long>(p.H) * p.W;
                if (ci + 0 < p.Cin) v.x = to_f32(X[base]);
                if (ci + 1 < p.Cin) v.y = to_f32(X[base + cs]);
                if (ci + 2 < p.Cin) v.z = to_f32(X[base + 2 * cs]);
                if (ci + 3 < p.Cin) v.w = to_f32(X[base + 3 * cs]);
            }
            *reinterpret_cast<float4 *>(Xs + static_cast<size_t>(xp) * CI_T + ((c4 ^ (xp & 7)) << 2)) = v;
        }
        // codes of my 32 output channels
        for (int i = threadIdx.x; i < 32 * npos_pad; i += 512) {
            const int c = i / npos_pad, pos = i - c * npos_pad;
            const int ly = pos / p.TW, lx = pos - ly * p.TW;
            const int y = y0 + ly, x = x0 + lx;
            int8_t code = 0;
            if (pos < npos && co0 + c < p.Cout && y < p.H && x < p.W)
                code = p.codes[((static_cast<long long>(b) * p.Cout + co0 + c) * p.H + y) * p.W + x];
            ct[c * npos_pad + pos] = code;
        }
        __syncthreads();

#pragma unroll
        for (int a = 0; a < CPG; ++a) {
            const int c = grp * CPG + a;   // local output channel of my group
            for (int pos0 = 0; pos0 < npos_pad; pos0 += G) {
                const int pos = pos0 + gl;
                const int code = (pos < npos_pad) ? ct[c * npos_pad + pos] : 0;
                const float cf = static_cast<float>(code);
                unsigned m = (__ballot_sync(kFull, code != 0) & gmask) >> gbase;
                while (__any_sync(kFull, m != 0)) {
                    const bool on = (m != 0);
                    const int j = on ? (__ffs(m) - 1) : 0;
                    m &= m - 1;
                    const float cv = __shfl_sync(kFull, cf, gbase + j);
                    if (on) {
                        const int q = pos0 + j;
                        const int ly = q / p.TW, lx = q - ly * p.TW;
#pragma unroll
                        for (int ky = 0; ky < KS; ++ky)
#pragma unroll
                            for (int kx = 0; kx < KS; ++kx) {
                                const int xp = (ly + ky) * TWp + lx + kx;
                                const float4 xv = *reinterpret_cast<const float4 *>(
                                    Xs + static_cast<size_t>(xp) * CI_T + ((gl ^ (xp & 7)) << 2));
                                float *r = acc[a][ky * KS + kx];
                                r[0] = fmaf(cv, xv.x, r[0]);
                                r[1] = fmaf(cv, xv.y, r[1]);
                                r[2] = fmaf(cv, xv.z, r[2]);
                                r[3] = fmaf(cv, xv.w, r[3]);
                            }
                    }
                }
            }
        }
    }

    const float delta = *p.delta_p;
#pragma unroll
    for (int a = 0; a < CPG; ++a) {
        const int co = co0 + grp * CPG + a;
        if (co >= p.Cout) continue;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int ci = ci0 + gl * 4 + v;
            if (ci >= p.Cin) continue;
#pragma unroll
            for (int t = 0; t < KK; ++t)
                atomicAdd(p.dW + (static_cast<long long>(co) * p.Cin + ci) * KK + t, acc[a][t][v] * delta);
        }
    }
}

// ------------------------------------------------------------------ db, ReLU', max-pool routing
__global__ void __launch_bounds__(256) bias_grad_kernel(const int8_t *__restrict__ codes,
                                                        const float *__restrict__ delta_p, int B,
                                                        int Cout, long long P, float *__restrict__ db) {
    const int co = blockIdx.x;
    long long s = 0;
    for (int b = 0; b < B; ++b) {
        const int8_t *src = codes + (static_cast<long long>(b) * Cout + co) * P;
        for (long long i = threadIdx.x; i < P; i += 256) s += src[i];
    }
    __shared__ long long sh[8];
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFull, s, o);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long tot = 0;
        for (int w = 0; w < 8; ++w) tot += sh[w];
        db[co] = static_cast<float>(tot) * (*delta_p);
    }
}

// delta_z = delta_a (.) f'(z), the derivative given as one byte per element; four elements per thread where
// the size and the pointers allow
__global__ void __launch_bounds__(256) relu_backward_kernel(const float *__restrict__ da, const uint8_t *__restrict__ mask,
                                                            float *__restrict__ dz, long long n, int vec) {
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (vec) {
        const long long n4 = n >> 2;
        for (; i < n4; i += stride) {
            const float4 a = __ldg(reinterpret_cast<const float4 *>(da) + i);
            const uchar4 m = __ldg(reinterpret_cast<const uchar4 *>(mask) + i);
            reinterpret_cast<float4 *>(dz)[i] = make_float4(m.x ? a.x : 0.f, m.y ? a.y : 0.f, m.z ? a.z : 0.f, m.w ? a.w : 0.f);
        }
        return;
    }
    for (; i < n; i += stride) dz[i] = mask[i] ? da[i] : 0.f;
}

// Routing of a pooled gradient g [planes][h][w] to out [planes][2h][2w]: one thread per window, which writes
// its four outputs (two pairs); argmax in {0,1,2,3} is the row-major position of the forward maximum
__global__ void __launch_bounds__(256) maxpool_backward_kernel(const float *__restrict__ g, const int8_t *__restrict__ am,
                                                               float *__restrict__ out, long long planes, int h, int w) {
    const long long n = planes * h * w;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long row = i / w;                    // (plane, y)
        const int x = static_cast<int>(i - row * w);
        const long long pl = row / h;
        const int y = static_cast<int>(row - pl * h);
        const float v = __ldg(g + i);
        const int which = am[i];
        float *o = out + ((pl * 2 * h + 2 * y) * 2ll * w + 2 * x);
        *reinterpret_cast<float2 *>(o) = make_float2(which == 0 ? v : 0.f, which == 1 ? v : 0.f);
        *reinterpret_cast<float2 *>(o + 2 * w) = make_float2(which == 2 ? v : 0.f, which == 3 ? v : 0.f);
    }
}

void pick_tile(const ConvShape &s, int max_pos, int &TH, int &TW) {
    TW = static_cast<int>(s.W < 64 ? s.W : 64);
    if (TW > max_pos) TW = max_pos;
    TH = max_pos / TW;
    if (TH > s.H) TH = static_cast<int>(s.H);
    if (TH < 1) TH = 1;
}

int blocks_for(long long n, int threads, int cap) {
    long long b = (n + threads - 1) / threads;
    if (b < 1) b = 1;
    if (b > cap) b = cap;
    return static_cast<int>(b);
}

}  // namespace

int launch_weight_taps(dbp_ctx *ctx, const void *W, int dtype, const ConvShape &s, void *w_taps,
                       bool to_f32) {
    const int KK = s.k * s.k;
    const long long n = s.Cout * s.Cin * KK;
    const int blocks = blocks_for(n, 256, ctx->sm_count * 8);
    if (dtype == DBP_F32)
        { note_launch(); weight_taps_kernel<float, float><<<blocks, 256, 0, ctx->stream>>>(
            static_cast<const float *>(W), static_cast<float *>(w_taps), s.Cout, s.Cin, KK); }
    else if (to_f32)
        { note_launch(); weight_taps_kernel<__nv_bfloat16, float><<<blocks, 256, 0, ctx->stream>>>(
            static_cast<const __nv_bfloat16 *>(W), static_cast<float *>(w_taps), s.Cout, s.Cin, KK); }
    else
        { note_launch(); weight_taps_kernel<__nv_bfloat16, __nv_bfloat16><<<blocks, 256, 0, ctx->stream>>>(
            static_cast<const __nv_bfloat16 *>(W), static_cast<__nv_bfloat16 *>(w_taps), s.Cout, s.Cin, KK); }
    return cuda_ok(cudaGetLastError());
}

template <int KS, int VEC, typename OutT>
static int launch_dx_t(dbp_ctx *ctx, const DxParams &p, size_t smem) {
    auto kern = conv_dx_kernel<KS, VEC, OutT>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return DBP_ECUDA;
    }
    const int CI_T = 32 * VEC;
    dim3 grid(static_cast<unsigned>(p.B * p.tiles_y * p.tiles_x), static_cast<unsigned>((p.Cin + CI_T - 1) / CI_T));
    note_launch();
    kern<<<grid, 256, smem, ctx->stream>>>(p);
    return cuda_ok(cudaGetLastError());
}

int launch_conv_dx(dbp_ctx *ctx, const int8_t *codes, const float *w_taps, const float *delta_p,
                   const ConvShape &s, void *dX, bool dx_bf16) {
    DxParams p;
    p.codes = codes; p.w_taps = w_taps; p.delta_p = delta_p; p.dX = dX;
    p.B = static_cast<int>(s.B); p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.H = static_cast<int>(s.H); p.W = static_cast<int>(s.W);
    const int vec = (s.Cin % 128 == 0 || (s.Cin % 4 == 0 && s.Cin > 64)) ? 4 : (s.Cin % 2 == 0 && s.Cin >= 64) ? 2 : 1;
    const int pad = (s.k - 1) / 2;
    // shrink the tile until codes + output staging fit in shared memory
    int max_pos = 128;
    size_t smem = 0;
    for (;;) {
        pick_tile(s, max_pos, p.TH, p.TW);
        int ps = ((p.TH + 2 * pad) * (p.TW + 2 * pad) + 3) & ~3;
        if (((ps / 4) & 1) == 0) ps += 4;          // odd word stride: lanes hit distinct banks
        p.plane_stride = ps;
        p.stage_stride = p.TH * p.TW + 1;
        smem = ((static_cast<size_t>(p.Cout) * ps + 15) & ~size_t(15)) +
               static_cast<size_t>(32 * vec) * p.stage_stride * 4;
        if (smem <= 200 * 1024 || max_pos == 1) break;
        max_pos /= 2;
    }
    if (smem > 227 * 1024) return DBP_EUNSUPPORTED;
    p.tiles_y = (p.H + p.TH - 1) / p.TH;
    p.tiles_x = (p.W + p.TW - 1) / p.TW;
#define DBP_DX(KS, VEC)                                                                         \
    (dx_bf16 ? launch_dx_t<KS, VEC, __nv_bfloat16>(ctx, p, smem) : launch_dx_t<KS, VEC, float>(ctx, p, smem))
    if (s.k == 1) return vec == 4 ? DBP_DX(1, 4) : vec == 2 ? DBP_DX(1, 2) : DBP_DX(1, 1);
    if (s.k == 5) return vec == 4 ? DBP_DX(5, 4) : vec == 2 ? DBP_DX(5, 2) : DBP_DX(5, 1);
    return vec == 4 ? DBP_DX(3, 4) : vec == 2 ? DBP_DX(3, 2) : DBP_DX(3, 1);
#undef DBP_DX
}

template <int KS, int CI_T, typename T>
static int launch_dw_t(dbp_ctx *ctx, const DwParams &p, size_t smem, dim3 grid) {
    auto kern = conv_dw_kernel<KS, CI_T, T>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return DBP_ECUDA;
    }
    note_launch();
    kern<<<grid, 512, smem, ctx->stream>>>(p);
    return cuda_ok(cudaGetLastError());
}

int launch_conv_dw(dbp_ctx *ctx, const int8_t *codes, const void *X, int dtype,
                   const float *delta_p, const ConvShape &s, float *dW) {
    DwParams p;
    p.codes = codes; p.X = X; p.delta_p = delta_p; p.dW = dW;
    p.B = static_cast<int>(s.B); p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.H = static_cast<int>(s.H); p.W = static_cast<int>(s.W);
    // 5x5: 25 taps x 4 channels of accumulators per thread leave no room for a second output channel per group
    const int ci_t = (s.Cin <= 64 || s.k == 5) ? 64 : 128;
    const int pad = (s.k - 1) / 2;
    int max_pos = 128;
    size_t smem = 0;
    for (;;) {
        pick_tile(s, max_pos, p.TH, p.TW);
        const int npos_pad = (p.TH * p.TW + 31) & ~31;
        smem = static_cast<size_t>(p.TH + 2 * pad) * (p.TW + 2 * pad) * ci_t * 4 + 32 * static_cast<size_t>(npos_pad);
        if (smem <= 200 * 1024 || max_pos == 1) break;
        max_pos /= 2;
    }
    p.tiles_y = (p.H + p.TH - 1) / p.TH;
    p.tiles_x = (p.W + p.TW - 1) / p.TW;
    const long long ntiles = s.B * p.tiles_y * p.tiles_x;
    const long long out_blocks = ((s.Cout + 31) / 32) * ((s.Cin + ci_t - 1) / ci_t);
    long long splits = (2LL * ctx->sm_count + out_blocks - 1) / out_blocks;
    if (splits > ntiles) splits = ntiles;
    if (splits < 1) splits = 1;
    if (splits > 65535) splits = 65535;
    p.splits = static_cast<int>(splits);
    cudaError_t e = cudaMemsetAsync(dW, 0, sizeof(float) * s.Cout * s.Cin * s.k * s.k, ctx->stream);
    if (e != cudaSuccess) return DBP_ECUDA;
    dim3 grid(static_cast<unsigned>((s.Cout + 31) / 32), static_cast<unsigned>((s.Cin + ci_t - 1) / ci_t),
              static_cast<unsigned>(splits));
#define DBP_DW(KS, CT)                                                                       \
    (dtype == DBP_F32 ? launch_dw_t<KS, CT, float>(ctx, p, smem, grid)                       \
                      : launch_dw_t<KS, CT, __nv_bfloat16>(ctx, p, smem, grid))
    if (s.k == 1) return ci_t == 64 ? DBP_DW(1, 64) : DBP_DW(1, 128);
    if (s.k == 5) return DBP_DW(5, 64);
    return ci_t == 64 ? DBP_DW(3, 64) : DBP_DW(3, 128);
#undef DBP_DW
}

int launch_bias_grad(dbp_ctx *ctx, const int8_t *codes, const float *delta_p, const ConvShape &s,
                     float *db) {
    note_launch();
    bias_grad_kernel<<<static_cast<unsigned>(s.Cout), 256, 0, ctx->stream>>>(
        codes, delta_p, static_cast<int>(s.B), static_cast<int>(s.Cout), s.H * s.W, db);
    return cuda_ok(cudaGetLastError());
}

int launch_relu_backward(dbp_ctx *ctx, const float *da, const uint8_t *mask, float *dz, long long n) {
    note_launch();
    const int vec = (n % 4 == 0) && ((reinterpret_cast<uintptr_t>(da) | reinterpret_cast<uintptr_t>(dz)) % 16 == 0) &&
                    (reinterpret_cast<uintptr_t>(mask) % 4 == 0);
    relu_backward_kernel<<<blocks_for(vec ? n / 4 : n, 256, ctx->sm_count * 8), 256, 0, ctx->stream>>>(da, mask, dz, n, vec);
    return cuda_ok(cudaGetLastError());
}

int launch_maxpool_backward(dbp_ctx *ctx, const float *g, const int8_t *argmax, float *out,
                            long long planes, long long h, long long w) {
    note_launch();
    maxpool_backward_kernel<<<blocks_for(planes * h * w, 256, ctx->sm_count * 8), 256, 0, ctx->stream>>>(
        g, argmax, out, planes, static_cast<int>(h), static_cast<int>(w));
    return cuda_ok(cudaGetLastError());
}

}  // namespace dbp
