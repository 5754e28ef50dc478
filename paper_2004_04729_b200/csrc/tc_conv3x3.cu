// Dense tensor-core path for the two backward products of 3x3 convolutions (stride 1, pad 1)
// with bf16 operands. Each product is nine accumulating GEMMs, one per tap, in which the
// operand that is shifted by the tap is always the quantized gradient: its int8 codes are
// staged once per tile (with a halo) in shared memory, and for every tap a shifted, border-
// masked copy is expanded to bf16 directly in the 128-byte-swizzled layout the MMA reads.
// The dense operand (weights for dX, activations for dW) is copied unshifted by cp.async.
//
//   dX[ci][p]        = Delta sum_tap sum_co Wr[tap][ci][co] * q[co][p + s_tap]     (per image)
//       M = ci (128 per accumulator, up to four accumulators), N = 128 positions, K = co
//   dW[tap][co][ci]  = Delta sum_(b,p) X[ci][p] * q[co][p - s_tap]
//       M = ci (128), N = 32 output channels per tap (nine accumulators), K = positions
//
// Eight producer warps build tiles, a ninth issues the MMAs. All waits are bounded.
#include "tc_common.cuh"

namespace dbp {

namespace {

using namespace tc;

constexpr int kProdWarps = 8;
constexpr int kProd = kProdWarps * 32;
constexpr int kThreads3 = kProd + 32;

struct P3 {
    const int8_t *codes;           // [B][Cout][H][W]
    const __nv_bfloat16 *Wr;       // dX: weights as [tap][Cin][Cout]
    const __nv_bfloat16 *X;        // dW: [B][Cin][H][W]
    const float *delta_p;
    void *dX;
    float *partials;               // dW: [split][tap][Cout][Cin]
    int dx_f32;
    int B, Cin, Cout, H, W, P;
    int tiles_per_img;             // dX: 128-position tiles per image; dW: 64-position stages per image
    int raw_words;                 // 32-bit words per row of the staged code tile
    int raw_pitch;                 // odd number of words between rows (bank-conflict free)
    long long per_split, nstages;  // dW
    int *err_flag;
};

// Eight consecutive code bytes of a staged row starting at byte offset `off`.
__device__ __forceinline__ uint2 bytes8(const unsigned *row, int off) {
    const int wi = off >> 2;
    const unsigned sel = 0x3210u + 0x1111u * static_cast<unsigned>(off & 3);
    const unsigned w0 = row[wi], w1 = row[wi + 1], w2 = row[wi + 2];
    return make_uint2(__byte_perm(w0, w1, sel), __byte_perm(w1, w2, sel));
}

// One 32-bit word (four positions a..a+3 of plane `plane`) of the staged code tile; zero
// outside [0, P). Planes start 4-byte aligned when P % 4 == 0.
__device__ __forceinline__ unsigned load_code_word(const int8_t *plane, int a, int P, bool row_ok, bool aligned4) {
    if (!row_ok || a + 3 < 0 || a >= P) return 0u;
    if (aligned4 && a >= 0 && a + 3 < P) return __ldg(reinterpret_cast<const unsigned *>(plane + a));
    unsigned w = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (a + j >= 0 && a + j < P) w |= (static_cast<unsigned>(__ldg(plane + a + j)) & 0xffu) << (8 * j);
    return w;
}

// byte masks (0xff = keep) for the eight positions n0..n0+7 of a tile starting at position p0:
// .x/.y keep the positions whose column x allows a source at x+1 (x <= W-2); z/w at x-1 (x >= 1)
__device__ __forceinline__ uint4 column_masks(int p0, int n0, int W) {
    unsigned m[4] = {0, 0, 0, 0};
    int x = (p0 + n0) % W;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (x <= W - 2) m[i >> 2] |= 0xffu << (8 * (i & 3));
        if (x >= 1) m[2 + (i >> 2)] |= 0xffu << (8 * (i & 3));
        if (++x == W) x = 0;
    }
    return make_uint4(m[0], m[1], m[2], m[3]);
}

struct Pipe3 {
    unsigned long long a_full[4], a_empty[4], b_full[4], b_empty[4], acc;
    unsigned tmem_base;
};

constexpr int kNA = 4;   // ring of dense-operand tiles
constexpr int kRawMaxWords = 68;

// ------------------------------------------------------------------------------------ dX
template <int MT>
__global__ void __launch_bounds__(kThreads3) tc3_dx_kernel(const P3 p) {
    constexpr int NB = 3;                         // ring of shifted code tiles
    constexpr int TILE = 16384;                   // 128 x 64 bf16
    constexpr unsigned PANEL = 64 * 128;          // bytes between the two 64-position groups
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char *a_s = smem;                            // kNA tiles [128 ci][64 co], K-major
    unsigned char *b_s = a_s + kNA * TILE;                // NB tiles [64 co][128 positions], MN-major
    unsigned *raw_s = reinterpret_cast<unsigned *>(b_s + NB * TILE);   // 2 x [64 rows][raw_pitch]
    __shared__ Pipe3 pipe;
    __shared__ uint4 masks[16];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x / p.tiles_per_img;
    const int p0 = (blockIdx.x - b * p.tiles_per_img) * 128;
    const int ci_base = blockIdx.y * (MT * 128);
    const int nchunks = (p.Cout + 63) / 64;
    const int halo = p.W + 1;
    const int a0 = ((p0 - halo) >> 2) << 2;       // position of byte 0 of a staged row (floor to 4)

    if (threadIdx.x == 0) {
        for (int s = 0; s < kNA; ++s) { mbar_init(&pipe.a_full[s], kProd); mbar_init(&pipe.a_empty[s], 1); }
        for (int s = 0; s < NB; ++s) { mbar_init(&pipe.b_full[s], kProd); mbar_init(&pipe.b_empty[s], 1); }
        mbar_init(&pipe.acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 16) masks[threadIdx.x] = column_masks(p0, threadIdx.x * 8, p.W);
    if (warp == kProdWarps) tmem_alloc(&pipe.tmem_base, MT * 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_d = pipe.tmem_base;

    if (warp < kProdWarps) {
        const bool aligned4 = (p.P & 3) == 0;
        // staged code tile: 64 rows x raw_words words; thread t owns row t/4, words t%4 + 4 i
        const int rrow = threadIdx.x >> 2, rw0 = threadIdx.x & 3;
        const int nword = (p.raw_words - rw0 + 3) >> 2;          // my words in a row (<= 17)
        const int8_t *img_base = p.codes + static_cast<long long>(b) * p.Cout * p.P;
        unsigned pre[17];                          // staged-tile words of the next chunk
        auto fetch = [&](int c) {
            const int co = c * 64 + rrow;
            const int8_t *plane = img_base + static_cast<long long>(co < p.Cout ? co : 0) * p.P;
#pragma unroll
            for (int i = 0; i < 17; ++i)
                pre[i] = (i < nword) ? load_code_word(plane, a0 + 4 * (rw0 + 4 * i), p.P, co < p.Cout, aligned4) : 0u;
        };
        fetch(0);
        bool ok = true;
        int ia = 0, ib = 0;
        for (int c = 0; c < nchunks; ++c) {
            unsigned *raw = raw_s + (c & 1) * (64 * p.raw_pitch);
#pragma unroll
            for (int i = 0; i < 17; ++i)
                if (i < nword) raw[rrow * p.raw_pitch + rw0 + 4 * i] = pre[i];
            asm volatile("bar.sync 1, %0;" ::"n"(kProd) : "memory");
            if (c + 1 < nchunks) fetch(c + 1);
#pragma unroll 1
            for (int tap = 0; tap < 9 && ok; ++tap, ++ib) {
                const int ky = tap / 3, kx = tap - ky * 3;
                const int shift = (1 - ky) * p.W + (1 - kx);
                const int sb = ib % NB;
                ok = mbar_wait(&pipe.b_empty[sb], ((ib / NB) & 1) ^ 1, p.err_flag);
                unsigned char *bt = b_s + sb * TILE;
                // 2 row groups x 16 chunks = 32 warp tasks; lanes = 32 consecutive co rows
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int task = warp * 4 + t;
                    const int ch = task & 15, row = (task >> 4) * 32 + lane;
                    uint2 c8 = bytes8(raw + row * p.raw_pitch, p0 + ch * 8 + shift - a0);
                    const uint4 m = masks[ch];
                    if (kx == 0) { c8.x &= m.x; c8.y &= m.y; }
                    if (kx == 2) { c8.x &= m.z; c8.y &= m.w; }
                    *reinterpret_cast<uint4 *>(bt + (ch >> 3) * PANEL + swz(row, ch & 7)) = expand8(c8);
                }
                fence_async_proxy();
                mbar_arrive(&pipe.b_full[sb]);
                // weights of this tap and chunk: MT tiles [128 ci][64 co]
                for (int m = 0; m < MT && ok; ++m, ++ia) {
                    const int sa = ia % kNA;
                    ok = mbar_wait(&pipe.a_empty[sa], ((ia / kNA) & 1) ^ 1, p.err_flag);
                    unsigned char *at = a_s + sa * TILE;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int idx = threadIdx.x + i * kProd;      // 1024 chunks of 16 bytes
                        const int row = idx >> 3, ch = idx & 7;
                        const int ci = ci_base + m * 128 + row, co = c * 64 + ch * 8;
                        const bool v = ci < p.Cin && co < p.Cout;      // Cout % 8 == 0
                        cp_async16(at + swz(row, ch),
                                   v ? p.Wr + (static_cast<long long>(tap) * p.Cin + ci) * p.Cout + co : p.Wr, v);
                    }
                    mbar_arrive_on_cp_async(&pipe.a_full[sa]);
                }
            }
        }
        // ---------------- epilogue: lanes = ci, columns = positions; warp w takes lane quarter
        // w % 4 and column half w / 4
        if (mbar_wait(&pipe.acc, 0, p.err_flag)) {
            tc_fence_after();
            const float delta = *p.delta_p;
            const int q = warp & 3, half = warp >> 2;
            const bool vec = (p.P & 7) == 0;
            for (int m = 0; m < MT; ++m) {
                const int ci = ci_base + m * 128 + q * 32 + lane;
#pragma unroll 1
                for (int cc = 0; cc < 2; ++cc) {
                    const int n0 = half * 64 + cc * 32;
                    unsigned v[32];
                    tmem_ld32(tmem_d + (static_cast<unsigned>(q * 32) << 16) + m * 128 + n0, v);
                    const long long base = (static_cast<long long>(b) * p.Cin + ci) * p.P + p0 + n0;
                    const int nvalid = p.P - (p0 + n0);      // positions of this run inside the image
                    if (ci >= p.Cin || nvalid <= 0) {
                        // nothing to store for this lane / run
                    } else if (p.dx_f32) {
                        float *dst = static_cast<float *>(p.dX) + base;
                        if (vec && nvalid >= 32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<float4 *>(dst + j) =
                                    make_float4(__uint_as_float(v[j]) * delta, __uint_as_float(v[j + 1]) * delta,
                                                __uint_as_float(v[j + 2]) * delta, __uint_as_float(v[j + 3]) * delta);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < nvalid) dst[j] = __uint_as_float(v[j]) * delta;
                        }
                    } else {
                        __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.dX) + base;
                        if (vec && nvalid >= 32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 8) {
                                unsigned w[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[j + 2 * e]) * delta,
                                                                                   __uint_as_float(v[j + 2 * e + 1]) * delta);
                                    w[e] = *reinterpret_cast<const unsigned *>(&h);
                                }
                                *reinterpret_cast<uint4 *>(dst + j) = make_uint4(w[0], w[1], w[2], w[3]);
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < nvalid) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]) * delta);
                        }
                    }
                }
            }
        }
    } else if (lane == 0) {
        constexpr unsigned idesc = make_idesc(128, 128, false, true);
        bool ok = true;
        int ia = 0, ib = 0;
        for (int c = 0; c < nchunks && ok; ++c) {
            for (int tap = 0; tap < 9 && ok; ++tap, ++ib) {
                const int sb = ib % NB;
                ok = mbar_wait(&pipe.b_full[sb], (ib / NB) & 1, p.err_flag);
                fence_async_proxy();
                tc_fence_after();
                const unsigned long long bd = make_desc(smem_u32(b_s + sb * TILE), PANEL, 1024);
                for (int m = 0; m < MT && ok; ++m, ++ia) {
                    const int sa = ia % kNA;
                    ok = mbar_wait(&pipe.a_full[sa], (ia / kNA) & 1, p.err_flag);
                    fence_async_proxy();
                    tc_fence_after();
                    const unsigned long long ad = make_desc(smem_u32(a_s + sa * TILE), 16, 1024);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        mma_bf16(tmem_d + m * 128, ad + 2 * k, bd + 128 * k, idesc, (c > 0 || tap > 0 || k > 0) ? 1u : 0u);
                    mma_commit(&pipe.a_empty[sa]);
                }
                mma_commit(&pipe.b_empty[sb]);
            }
        }
        mma_commit(&pipe.acc);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kProdWarps) {
        __syncwarp();
        tmem_dealloc(tmem_d, MT * 128);
    }
}

// weights [Cout][Cin][3][3] -> [tap][Cin][Cout]
__global__ void weight_rows_kernel(const __nv_bfloat16 *__restrict__ W, __nv_bfloat16 *__restrict__ out,
                                   long long Cout, long long Cin) {
    const long long n = Cout * Cin * 9;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long co = i % Cout, ci = (i / Cout) % Cin, t = i / (Cout * Cin);
        out[i] = W[(co * Cin + ci) * 9 + t];
    }
}

// ------------------------------------------------------------------------------------ dW
// One stage = 64 consecutive positions of one image. A = X tile [128 ci][64 positions] (native,
// K-major), B_tap = shifted codes [32 co][64 positions] (K-major), nine accumulators of 32 columns.
// GX: positions per aligned group of X: 8 (P % 8 == 0), 4 (P % 4 == 0) or 1
template <int GX>
__global__ void __launch_bounds__(kThreads3) tc3_dw_kernel(const P3 p) {
    constexpr int NB = 2;
    constexpr int A_TILE = 16384;                 // 128 x 64 bf16
    constexpr int B_TAP = 32 * 128;               // 32 x 64 bf16
    constexpr int B_STAGE = 9 * B_TAP;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char *a_s = smem;
    unsigned char *b_s = a_s + kNA * A_TILE;
    unsigned *raw_s = reinterpret_cast<unsigned *>(b_s + NB * B_STAGE);   // 2 x [32 rows][raw_pitch]
    __shared__ Pipe3 pipe;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ci0 = blockIdx.x * 128, co0 = blockIdx.y * 32;
    const long long s0 = blockIdx.z * p.per_split;
    long long s1 = s0 + p.per_split;
    if (s1 > p.nstages) s1 = p.nstages;
    const int niter = s1 > s0 ? static_cast<int>(s1 - s0) : 0;
    const int halo = p.W + 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kNA; ++s) { mbar_init(&pipe.a_full[s], kProd); mbar_init(&pipe.a_empty[s], 1); }
        for (int s = 0; s < NB; ++s) { mbar_init(&pipe.b_full[s], kProd); mbar_init(&pipe.b_empty[s], 1); }
        mbar_init(&pipe.acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProdWarps) tmem_alloc(&pipe.tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_d = pipe.tmem_base;

    if (warp < kProdWarps) {
        const bool aligned4 = (p.P & 3) == 0;
        // staged code tile: 32 rows x raw_words words; thread t owns row t/8, words t%8 + 8 i
        const int rrow = threadIdx.x >> 3, rw0 = threadIdx.x & 7;
        const int nword = (p.raw_words - rw0 + 7) >> 3;         // my words in a row (<= 9)
        const bool rrow_ok = co0 + rrow < p.Cout;
        const int8_t *row_base = p.codes + static_cast<long long>(co0 + (rrow_ok ? rrow : 0)) * p.P;
        const long long img_codes = static_cast<long long>(p.Cout) * p.P, img_x = static_cast<long long>(p.Cin) * p.P;
        // X tile: my four 16-byte chunks are (row = t/8 + 32 i, chunk = t%8)
        const int xch = threadIdx.x & 7;
        // position of a stage: image and first position, advanced incrementally
        int bimg = static_cast<int>(s0 / p.tiles_per_img);
        int k0 = static_cast<int>(s0 - static_cast<long long>(bimg) * p.tiles_per_img) * 64;
        int nb = bimg, nk0 = k0;                                 // the stage being prefetched
        unsigned pre[9];
        auto fetch = [&]() {
            const int a0 = ((nk0 - halo) >> 2) << 2;
            const int8_t *plane = row_base + nb * img_codes;
#pragma unroll
            for (int i = 0; i < 9; ++i)
                pre[i] = (i < nword) ? load_code_word(plane, a0 + 4 * (rw0 + 8 * i), p.P, rrow_ok, aligned4) : 0u;
        };
        auto advance = [&](int &bb, int &kk) {
            kk += 64;
            if (kk >= p.tiles_per_img * 64) { kk = 0; ++bb; }
        };
        if (niter > 0) fetch();
        bool ok = true;
        for (int it = 0; it < niter; ++it) {
            const int a0 = ((k0 - halo) >> 2) << 2;
            unsigned *raw = raw_s + (it & 1) * (32 * p.raw_pitch);
#pragma unroll
            for (int i = 0; i < 9; ++i)
                if (i < nword) raw[rrow * p.raw_pitch + rw0 + 8 * i] = pre[i];
            asm volatile("bar.sync 1, %0;" ::"n"(kProd) : "memory");
            advance(nb, nk0);
            if (it + 1 < niter) fetch();
            if (ok) {
                // ---- X tile: 128 ci rows x 8 chunks of 8 positions
                const int sa = it % kNA;
                ok = mbar_wait(&pipe.a_empty[sa], ((it / kNA) & 1) ^ 1, p.err_flag);
                unsigned char *at = a_s + sa * A_TILE;
                const int pp = k0 + xch * 8;
                const __nv_bfloat16 *xsrc = p.X + bimg * img_x + pp;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = (threadIdx.x >> 3) + 32 * i;
                    const int ci = ci0 + row;
                    const __nv_bfloat16 *src = xsrc + static_cast<long long>(ci) * p.P;
                    if (GX == 8) {   // whole 16-byte groups, aligned
                        const bool v = ci < p.Cin && pp < p.P;
                        cp_async16(at + swz(row, xch), v ? src : p.X, v);
                    } else if (GX == 4) {   // two aligned 8-byte halves, each inside the image or not
                        const bool v0 = ci < p.Cin && pp < p.P, v1 = ci < p.Cin && pp + 4 < p.P;
                        cp_async_small<8>(at + swz(row, xch), v0 ? src : p.X, v0);
                        cp_async_small<8>(at + swz(row, xch) + 8, v1 ? src + 4 : p.X, v1);
                    } else {
                        unsigned short h[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            h[j] = (ci < p.Cin && pp + j < p.P) ? __ldg(reinterpret_cast<const unsigned short *>(src) + j) : 0;
                        *reinterpret_cast<uint4 *>(at + swz(row, xch)) =
                            make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
                    }
                }
                if (GX > 1) {
                    mbar_arrive_on_cp_async(&pipe.a_full[sa]);
                } else {
                    fence_async_proxy();
                    mbar_arrive(&pipe.a_full[sa]);
                }
                // ---- nine shifted code tiles; warp w builds chunk w of every tap, lanes = co rows
                const int sb = it % NB;
                ok = ok && mbar_wait(&pipe.b_empty[sb], ((it / NB) & 1) ^ 1, p.err_flag);
                unsigned char *bt = b_s + sb * B_STAGE + swz(lane, warp);
                const unsigned *rrow_s = raw + lane * p.raw_pitch;
                const int off0 = k0 + warp * 8 - a0;
                // source column is x' - (kx-1): kx = 0 needs x' <= W-2, kx = 2 needs x' >= 1
                const uint4 m = column_masks(k0, warp * 8, p.W);
#pragma unroll
                for (int ky = 0; ky < 3; ++ky) {
                    // X[p + (ky-1) W + (kx-1)] pairs with q[p]: with p' the X position, q index is p' - s
                    const int offy = off0 - (ky - 1) * p.W;
                    uint2 c0 = bytes8(rrow_s, offy + 1), c1 = bytes8(rrow_s, offy), c2 = bytes8(rrow_s, offy - 1);
                    c0.x &= m.x; c0.y &= m.y;
                    c2.x &= m.z; c2.y &= m.w;
                    *reinterpret_cast<uint4 *>(bt + (ky * 3 + 0) * B_TAP) = expand8(c0);
                    *reinterpret_cast<uint4 *>(bt + (ky * 3 + 1) * B_TAP) = expand8(c1);
                    *reinterpret_cast<uint4 *>(bt + (ky * 3 + 2) * B_TAP) = expand8(c2);
                }
                fence_async_proxy();
                mbar_arrive(&pipe.b_full[sb]);
            }
            advance(bimg, k0);
        }
        // ---------------- epilogue: lanes = ci, columns = (tap, co); partials [split][tap][Cout][Cin]
        if (niter > 0 && mbar_wait(&pipe.acc, 0, p.err_flag)) {
            tc_fence_after();
            const int q = warp & 3;
            const int ci = ci0 + q * 32 + lane;
            for (int tap = warp >> 2; tap < 9; tap += 2) {
                unsigned v[32];
                tmem_ld32(tmem_d + (static_cast<unsigned>(q * 32) << 16) + tap * 32, v);
                if (ci < p.Cin) {
                    float *dst = p.partials + ((static_cast<long long>(blockIdx.z) * 9 + tap) * p.Cout + co0) * p.Cin + ci;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (co0 + j < p.Cout) dst[static_cast<long long>(j) * p.Cin] = __uint_as_float(v[j]);
                }
            }
        }
    } else if (lane == 0) {
        constexpr unsigned idesc = make_idesc(128, 32, false, false);
        bool ok = true;
        for (int it = 0; it < niter && ok; ++it) {
            const int sa = it % kNA, sb = it % NB;
            ok = mbar_wait(&pipe.a_full[sa], (it / kNA) & 1, p.err_flag);
            ok = ok && mbar_wait(&pipe.b_full[sb], (it / NB) & 1, p.err_flag);
            fence_async_proxy();
            tc_fence_after();
            const unsigned long long ad = make_desc(smem_u32(a_s + sa * A_TILE), 16, 1024);
            const unsigned b_addr = smem_u32(b_s + sb * B_STAGE);
            for (int tap = 0; tap < 9; ++tap) {
                const unsigned long long bd = make_desc(b_addr + tap * B_TAP, 16, 1024);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    mma_bf16(tmem_d + tap * 32, ad + 2 * k, bd + 2 * k, idesc, (it > 0 || k > 0) ? 1u : 0u);
            }
            mma_commit(&pipe.a_empty[sa]);
            mma_commit(&pipe.b_empty[sb]);
        }
        if (niter > 0) mma_commit(&pipe.acc);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kProdWarps) {
        __syncwarp();
        tmem_dealloc(tmem_d, 512);
    }
}

// dW[co][ci][tap] = Delta * sum over splits of partials[split][tap][co][ci]. A block spreads the
// splits over its eight warps (lanes = 32 consecutive float4 of [tap][co][ci]) and combines the
// eight partial sums in a fixed order.
__global__ void __launch_bounds__(256) tc3_dw_reduce_kernel(const float4 *__restrict__ partials, int nsplit,
                                                            long long Cout, long long Cin,
                                                            const float *__restrict__ delta_p, float *__restrict__ dW) {
    chain_wait();        // launched chained: earlier kernels' writes are visible from here on
    chain_release();
    __shared__ float4 sh[8][32];
    const long long n = Cout * Cin, tot4 = n * 9 / 4;            // Cin % 4 == 0
    const int e = threadIdx.x & 31, sg = threadIdx.x >> 5;
    const long long i4 = blockIdx.x * 32ll + e;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i4 < tot4) {
#pragma unroll 4
        for (int s = sg; s < nsplit; s += 8) {
            const float4 v = __ldcs(partials + s * tot4 + i4);
            a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        }
    }
    sh[sg][e] = a;
    __syncthreads();
    if (sg == 0 && i4 < tot4) {
#pragma unroll
        for (int g = 1; g < 8; ++g) {
            const float4 v = sh[g][e];
            a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        }
        const float delta = *delta_p;
        const long long i = i4 * 4, tap = i / n, rem = i - tap * n;      // rem = co * Cin + ci
        float *dst = dW + rem * 9 + tap;
        dst[0] = a.x * delta; dst[9] = a.y * delta; dst[18] = a.z * delta; dst[27] = a.w * delta;
    }
}

// The same sum for large weight tensors and few splits: a block owns 128 consecutive (co, ci)
// pairs, a warp one tap at a time (coalesced 512-byte reads of every split), and the block writes
// its 128 x 9 results as one contiguous run instead of stores nine floats apart.
__global__ void __launch_bounds__(256) tc3_dw_reduce_rows_kernel(const float4 *__restrict__ partials, int nsplit,
                                                                 long long Cout, long long Cin,
                                                                 const float *__restrict__ delta_p, float *__restrict__ dW) {
    chain_wait();        // launched chained: earlier kernels' writes are visible from here on
    chain_release();
    __shared__ float out[128 * 9];
    const long long n = Cout * Cin, n4 = n / 4, tot4 = n4 * 9;   // Cin % 4 == 0
    const int e = threadIdx.x & 31, sg = threadIdx.x >> 5;
    const long long r4 = blockIdx.x * 32ll + e;                  // float4 index inside a tap's plane
    const float delta = *delta_p;
    for (int tap = sg; tap < 9; tap += 8) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r4 < n4) {
            const float4 *src = partials + tap * n4 + r4;
#pragma unroll 4
            for (int s = 0; s < nsplit; ++s) {
                const float4 v = __ldcs(src + s * tot4);
                a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
            }
        }
        out[(4 * e + 0) * 9 + tap] = a.x * delta;
        out[(4 * e + 1) * 9 + tap] = a.y * delta;
        out[(4 * e + 2) * 9 + tap] = a.z * delta;
        out[(4 * e + 3) * 9 + tap] = a.w * delta;
    }
    __syncthreads();
    const long long base = blockIdx.x * 128ll;                   // first (co, ci) pair of the block
    const long long left = n - base;
    const int cnt = static_cast<int>(left < 128 ? left : 128) * 9;   // a multiple of 4
    float4 *dst = reinterpret_cast<float4 *>(dW + base * 9);
    for (int i = threadIdx.x; i < cnt / 4; i += 256) dst[i] = reinterpret_cast<const float4 *>(out)[i];
}

int raw_geometry(int W, int span, int &words, int &pitch) {
    // a staged row covers positions [floor4(start - (W+1)), start + span + (W+1)) plus slack for
    // the three-word reads of bytes8
    words = (span + 2 * (W + 1) + 3 + 3) / 4 + 2;
    pitch = words | 1;
    return words <= kRawMaxWords ? DBP_OK : DBP_EUNSUPPORTED;
}

template <typename K>
int set_smem3(K kern, size_t bytes) {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) == cudaSuccess
               ? DBP_OK : DBP_ECUDA;
}

}  // namespace

bool tc3_supported(const ConvShape &s, int io) {
    return io == DBP_BF16 && s.k == 3 && s.Cin % 8 == 0 && s.Cout % 8 == 0 && s.W <= 62 && s.H * s.W < (1 << 24);
}

int launch_tc3_dx(dbp_ctx *ctx, const int8_t *codes, const void *W, const float *delta_p,
                  const ConvShape &s, void *dX, bool dx_bf16, int *err_flag) {
    {
        const int rc_shift = launch_tc3_dx_shift(ctx, codes, W, delta_p, s, dX, dx_bf16, err_flag);
        if (rc_shift != DBP_EUNSUPPORTED) return rc_shift;
    }
    P3 p{};
    p.codes = codes; p.delta_p = delta_p; p.dX = dX; p.dx_f32 = dx_bf16 ? 0 : 1;
    p.B = static_cast<int>(s.B); p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.H = static_cast<int>(s.H); p.W = static_cast<int>(s.W); p.P = p.H * p.W;
    p.tiles_per_img = (p.P + 127) / 128;
    p.err_flag = err_flag;
    int rc = raw_geometry(p.W, 128, p.raw_words, p.raw_pitch);
    if (rc) return rc;
    if (64 * p.raw_words > 17 * kProd) return DBP_EUNSUPPORTED;
    const size_t wb = sizeof(__nv_bfloat16) * static_cast<size_t>(s.Cout) * s.Cin * 9;
    if ((rc = ws_reserve(ctx, ctx->w_taps, wb))) return rc;
    __nv_bfloat16 *wr = static_cast<__nv_bfloat16 *>(ctx->w_taps.ptr);
    {
        long long blocks = (static_cast<long long>(s.Cout) * s.Cin * 9 + 255) / 256;
        if (blocks > ctx->sm_count * 8) blocks = ctx->sm_count * 8;
        weight_rows_kernel<<<static_cast<unsigned>(blocks), 256, 0, ctx->stream>>>(
            static_cast<const __nv_bfloat16 *>(W), wr, s.Cout, s.Cin);
        if ((rc = cuda_ok(cudaGetLastError()))) return rc;
    }
    p.Wr = wr;
    const int mt = s.Cin > 256 ? 4 : s.Cin > 128 ? 2 : 1;
    dim3 grid(static_cast<unsigned>(s.B * p.tiles_per_img), static_cast<unsigned>((s.Cin + mt * 128 - 1) / (mt * 128)));
    const size_t smem = static_cast<size_t>(kNA + 3) * 16384 + 2 * 64 * static_cast<size_t>(p.raw_pitch) * 4 + 1024;
    if (mt == 4) { if ((rc = set_smem3(tc3_dx_kernel<4>, smem))) return rc; tc3_dx_kernel<4><<<grid, kThreads3, smem, ctx->stream>>>(p); }
    else if (mt == 2) { if ((rc = set_smem3(tc3_dx_kernel<2>, smem))) return rc; tc3_dx_kernel<2><<<grid, kThreads3, smem, ctx->stream>>>(p); }
    else { if ((rc = set_smem3(tc3_dx_kernel<1>, smem))) return rc; tc3_dx_kernel<1><<<grid, kThreads3, smem, ctx->stream>>>(p); }
    return cuda_ok(cudaGetLastError());
}

static int launch_tc3_dw_generic(dbp_ctx *ctx, const int8_t *codes, const void *X, const float *delta_p,
                                 const ConvShape &s, int *err_flag, long long *nsplit) {
    P3 p{};
    p.codes = codes; p.X = static_cast<const __nv_bfloat16 *>(X); p.delta_p = delta_p;
    p.B = static_cast<int>(s.B); p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.H = static_cast<int>(s.H); p.W = static_cast<int>(s.W); p.P = p.H * p.W;
    p.tiles_per_img = (p.P + 63) / 64;
    p.nstages = static_cast<long long>(s.B) * p.tiles_per_img;
    p.err_flag = err_flag;
    int rc = raw_geometry(p.W, 64, p.raw_words, p.raw_pitch);
    if (rc) return rc;
    if (32 * p.raw_words > 9 * kProd) return DBP_EUNSUPPORTED;
    const long long tiles = ((s.Cin + 127) / 128) * ((s.Cout + 31) / 32);
    const long long split = choose_split(tiles, p.nstages, ctx->sm_count, &p.per_split);
    const size_t nw = static_cast<size_t>(s.Cout) * s.Cin * 9;
    if ((rc = ws_reserve(ctx, ctx->tc_partials, sizeof(float) * nw * split))) return rc;
    p.partials = static_cast<float *>(ctx->tc_partials.ptr);
    dim3 grid(static_cast<unsigned>((s.Cin + 127) / 128), static_cast<unsigned>((s.Cout + 31) / 32),
              static_cast<unsigned>(split));
    const size_t smem = static_cast<size_t>(kNA) * 16384 + 2 * 9 * 4096 + 2 * 32 * static_cast<size_t>(p.raw_pitch) * 4 + 1024;
    if (p.P % 8 == 0) {
        if ((rc = set_smem3(tc3_dw_kernel<8>, smem))) return rc;
        tc3_dw_kernel<8><<<grid, kThreads3, smem, ctx->stream>>>(p);
    } else if (p.P % 4 == 0) {
        if ((rc = set_smem3(tc3_dw_kernel<4>, smem))) return rc;
        tc3_dw_kernel<4><<<grid, kThreads3, smem, ctx->stream>>>(p);
    } else {
        if ((rc = set_smem3(tc3_dw_kernel<1>, smem))) return rc;
        tc3_dw_kernel<1><<<grid, kThreads3, smem, ctx->stream>>>(p);
    }
    *nsplit = split;
    return cuda_ok(cudaGetLastError());
}

int launch_tc3_dw(dbp_ctx *ctx, const int8_t *codes, const void *X, const float *delta_p,
                  const ConvShape &s, float *dW, int *err_flag) {
    const size_t nw = static_cast<size_t>(s.Cout) * s.Cin * 9;
    long long split = 0;
    int rc = launch_tc3_dw_shift(ctx, codes, X, s, err_flag, &split);
    if (rc == DBP_EUNSUPPORTED) rc = launch_tc3_dw_generic(ctx, codes, X, delta_p, s, err_flag, &split);
    if (rc) return rc;
    const long long tot4 = static_cast<long long>(nw) / 4;
    const long long pairs = s.Cout * s.Cin;
    if (split <= 32 && pairs >= 128 * 128)
        return cuda_ok(launch_chained(tc3_dw_reduce_rows_kernel, dim3(static_cast<unsigned>((pairs + 127) / 128)), dim3(256), 0,
                                      ctx->stream, reinterpret_cast<const float4 *>(ctx->tc_partials.ptr),
                                      static_cast<int>(split), s.Cout, s.Cin, delta_p, dW));
    return cuda_ok(launch_chained(tc3_dw_reduce_kernel, dim3(static_cast<unsigned>((tot4 + 31) / 32)), dim3(256), 0, ctx->stream,
                                  reinterpret_cast<const float4 *>(ctx->tc_partials.ptr), static_cast<int>(split), s.Cout,
                                  s.Cin, delta_p, dW));
}

}  // namespace dbp
