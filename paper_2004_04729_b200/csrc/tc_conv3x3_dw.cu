// Dense tensor-core weight gradient of 3x3 convolutions (stride 1, pad 1), bf16 operands:
//   dW[co][ci][ky][kx] = Delta * sum_(b,u) X[b][ci][u] * q[b][co][u + (1-ky) W + (1-kx)]
// with u a position of the image and the code taken as zero outside it (and where the column
// would wrap around a row end).
//
// One GEMM per tap: M = 128 input channels (A = the activations as they lie in memory,
// K-major), N = 64 or 128 output channels, K = positions in stages of 64. A tcgen05 MMA with
// M = 128 occupies the tensor core for about 72 cycles whatever N <= 128 is, so N must be wide;
// nine accumulators of that width do not fit the tensor memory, hence a CTA computes the three
// taps of ONE kernel column kx (three accumulators) and the grid has three CTAs per tile.
//
// The codes of a segment of positions (plus a halo of W + 1 on either side) are expanded to
// bf16 once, transposed to rows of [position][co] (an MN-major operand), and a tap ky is then
// only a different start row of that operand: the swizzle is a function of the absolute
// shared-memory address, so a descriptor may start at any row. Left/right padding cannot be a
// row offset: the copy for kx = 0 has the rows of image column 0 zeroed, the copy for kx = 2
// those of column W-1.
//
// Sixteen warps stage and expand (cp.async into staging buffers, tracked by cp.async groups,
// one mbarrier arrival per warp), one thread issues the MMAs. K is split across CTAs by
// segments; partial blocks go to a workspace and a small kernel sums them. All waits are bounded.
#include "tc_common.cuh"

namespace dbp {

namespace {

using namespace tc;

constexpr int kXW = 16;                  // staging / expansion warps (also the epilogue)
constexpr int kX = kXW * 32;
constexpr int kThreadsW = kX + 32;       // + MMA warp
constexpr int kMaxNX = 6;                // ring of activation tiles
constexpr int kTileX = 16384;            // 128 ci x 64 positions bf16
constexpr int kMaxStages = 4;            // 64-position stages per segment

struct Sw3P {
    const int8_t *codes;           // [B][Cout][P]
    const __nv_bfloat16 *X;        // [B][Cin][P]
    float *partials;               // [split][tap][Cout][Cin]
    int B, Cin, Cout, W, P;
    int SEG;                       // positions per segment (multiple of 64)
    int segs_per_img;
    int RQ;                        // rows of one expanded copy (multiple of 8)
    int HQ;                        // expanded rows before the segment's first position (>= W + 1, multiple of 4)
    int raw_pitch;                 // bytes between two code rows of the staging buffer
    int raw_coff;                  // staging column of expanded row 0
    int raw_lead;                  // row mode: positions staged before the segment (multiple of 16); -1: slab mode
    int raw_bytes;                 // one staging buffer
    int nsplit;                    // K splits (grid.z = 3 * nsplit)
    int nx;                        // activation tiles in the ring
    long long nseg, per_split;
    int *err_flag;
};

struct PipeW {
    unsigned long long x_full[kMaxNX], x_empty[kMaxNX], qt_full[2], qt_empty[2], acc;
    unsigned tmem_base;
};

// XM: how the activation tile is filled: 8 = 16-byte copies (P % 8 == 0), 4 = 8-byte copies
// (P % 4 == 0), 0 = the image's [128 ci][P] block staged whole and re-laid from shared memory
// (any P <= 64). NP: 64-channel panels of the code operand (N = 64 NP output channels).
template <int XM, int NP>
__global__ void __launch_bounds__(kThreadsW) tc3_dw_shift_kernel(const Sw3P p) {
    chain_wait();        // launched chained: earlier kernels' writes are visible from here on
    chain_release();
    constexpr int N = 64 * NP;
    constexpr int TCOLS = NP == 2 ? 512 : 256;                         // three accumulators of N columns
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char *x_s = smem;                                         // nx activation tiles
    unsigned char *qt = x_s + p.nx * kTileX;                           // 2 buffers x NP panels x RQ rows x 128 B
    const unsigned panel_bytes = static_cast<unsigned>(p.RQ) * 128u;
    unsigned char *raw_s = qt + 2 * NP * panel_bytes;                        // 2 code staging buffers
    unsigned char *xraw = raw_s + 2 * p.raw_bytes;                     // XM == 0: staged activations (16 KB)
    __shared__ PipeW pipe;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ci0 = blockIdx.x * 128, co0 = blockIdx.y * N;
    const int kx = blockIdx.z % 3, zsplit = blockIdx.z / 3;
    const long long g0 = zsplit * p.per_split;
    long long g1 = g0 + p.per_split;
    if (g1 > p.nseg) g1 = p.nseg;
    const int nsegs = g1 > g0 ? static_cast<int>(g1 - g0) : 0;
    const int halo = p.HQ;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.nx; ++s) { mbar_init(&pipe.x_full[s], kXW); mbar_init(&pipe.x_empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&pipe.qt_full[s], kXW); mbar_init(&pipe.qt_empty[s], 1); }
        mbar_init(&pipe.acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kXW) tmem_alloc(&pipe.tmem_base, TCOLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_d = pipe.tmem_base;

    // segment g: image g / segs_per_img, first position (g % segs_per_img) * SEG, its 64-position stages
    auto seg_of = [&](long long g, int &b, int &u0, int &ns) {
        b = static_cast<int>(g / p.segs_per_img);
        u0 = static_cast<int>(g - static_cast<long long>(b) * p.segs_per_img) * p.SEG;
        const int left = p.P - u0;
        ns = ((left < p.SEG ? left : p.SEG) + 63) >> 6;
    };

    if (warp < kXW) {
        const int t = threadIdx.x;
        // ---- activation tile: my chunk column and my two rows
        const int xc = t & 7, xr = t >> 3;                     // rows xr, xr + 64
        const bool xv0 = ci0 + xr < p.Cin, xv1 = ci0 + xr + 64 < p.Cin;
        const unsigned xo0 = swz(xr, xc), xo1 = swz(xr + 64, xc);
        // ---- expansion: chunks of eight co (t >> 6) + 8 * panel, rows (t & 63) + 64 * pass
        const int ch = t >> 6, er = t & 63;
        const bool row_mode = p.raw_lead >= 0;
        bool ok = true;
        int xslot = 0, xphase = 0;                              // ring position of the next tile to fill
        int aslot = 0;                                          // ring position of the next tile to announce

        auto issue_raw = [&](long long g) {
            int b, u0, ns;
            seg_of(g, b, u0, ns);
            unsigned char *raw = raw_s + (g & 1) * p.raw_bytes;
            const int8_t *src = p.codes + (static_cast<long long>(b) * p.Cout + co0) * p.P;
            if (row_mode) {
                const int cpr = p.raw_pitch >> 4;                // 16-byte chunks per row
                for (int idx = t; idx < N * cpr; idx += kX) {
                    const int co = idx / cpr, j = idx - co * cpr;
                    const int pos = u0 - p.raw_lead + 16 * j;
                    const bool v = pos >= 0 && pos < p.P && co0 + co < p.Cout;       // P % 16 == 0: all or nothing
                    // rows are staged in the order (co % 8, co / 8): the eight rows of a chunk lie N/8 rows apart
                    const int rho = (co & 7) * (N / 8) + (co >> 3);
                    cp_async16(raw + rho * p.raw_pitch + 16 * j, v ? src + static_cast<long long>(co) * p.P + pos : p.codes, v);
                }
            } else {
                const int nb = N * p.P;                          // Cout % N == 0: all rows exist
                for (int idx = t; idx * 16 < nb; idx += kX) cp_async16(raw + idx * 16, src + idx * 16, true);
            }
        };

        if (nsegs > 0) issue_raw(g0);
        cp_async_commit();
        for (int sg = 0; sg < nsegs; ++sg) {
            const long long g = g0 + sg;
            int b, u0, ns;
            seg_of(g, b, u0, ns);
            const int buf = sg & 1;
            // ---- (1) activation tiles of this segment, one cp.async group per stage
            const __nv_bfloat16 *xb = p.X + (static_cast<long long>(b) * p.Cin + ci0) * p.P;
            if (XM == 0) {
                // whole [128 ci][P] block (one stage); nobody reads xraw any more: the re-layout of
                // the previous segment ended before that segment's last barrier
                const int nci = p.Cin - ci0 < 128 ? p.Cin - ci0 : 128;
                for (int idx = t; idx * 8 < nci * p.P; idx += kX) cp_async16(xraw + idx * 16, xb + idx * 8, true);
                cp_async_commit();
            } else {
                for (int k = 0; k < ns; ++k) {
                    ok = ok && mbar_wait(&pipe.x_empty[xslot], xphase ^ 1, p.err_flag);
                    unsigned char *xt = x_s + xslot * kTileX;
                    const int pos = u0 + 64 * k + 8 * xc;
                    const __nv_bfloat16 *s0 = xb + static_cast<long long>(xr) * p.P + pos;
                    const __nv_bfloat16 *s1 = s0 + 64ll * p.P;
                    if (XM == 8) {
                        const bool v = pos < p.P;
                        cp_async16(xt + xo0, (v && xv0) ? s0 : p.X, v && xv0);
                        cp_async16(xt + xo1, (v && xv1) ? s1 : p.X, v && xv1);
                    } else {
                        const bool va = pos < p.P, vb = pos + 4 < p.P;
                        cp_async_small<8>(xt + xo0, (va && xv0) ? s0 : p.X, va && xv0);
                        cp_async_small<8>(xt + xo0 + 8, (vb && xv0) ? s0 + 4 : p.X, vb && xv0);
                        cp_async_small<8>(xt + xo1, (va && xv1) ? s1 : p.X, va && xv1);
                        cp_async_small<8>(xt + xo1 + 8, (vb && xv1) ? s1 + 4 : p.X, vb && xv1);
                    }
                    cp_async_commit();
                    if (++xslot == p.nx) { xslot = 0; xphase ^= 1; }
                }
            }
            const int ngrp = XM == 0 ? 1 : ns;                   // groups committed in (1)
            // ---- (2) the codes of this segment have landed (they were requested a segment ago)
            cp_async_wait_pending(ngrp);
            asm volatile("bar.sync 1, %0;" ::"n"(kX) : "memory");
            // ---- (3) request the next segment's codes (the other staging buffer is free since the barrier)
            if (sg + 1 < nsegs) issue_raw(g + 1);
            cp_async_commit();
            // ---- (4) expand into the three copies of buffer `buf`
            ok = ok && mbar_wait(&pipe.qt_empty[buf], ((sg >> 1) & 1) ^ 1, p.err_flag);
            {
                unsigned char *q1 = qt + buf * NP * panel_bytes;
                const int nrows = ns * 64 + 2 * halo;
                const int zero_col = kx == 0 ? 0 : (kx == 2 ? p.W - 1 : -1);     // image column whose rows are zero in this copy
                if (row_mode) {
                    // Four rows x eight channels per task: eight 32-bit loads (four consecutive
                    // positions of one channel each), a byte transpose, four expansions. Lane bits:
                    // chunk (2), row-group parity (1), row group (2): conflict-free loads (the
                    // staging pitch is an odd multiple of 32 bytes) and stores.
                    const unsigned *raw32 = reinterpret_cast<const unsigned *>(raw_s + (g & 1) * p.raw_bytes);
                    const int pitchw = p.raw_pitch >> 2, c0w = p.raw_coff >> 2, estep = (N / 8) * pitchw;
                    const int ch = (warp & 1) * 4 + (t & 3);
                    const int ngroups = nrows >> 2;
#pragma unroll 1
                    for (int rg = ((t >> 2) & 7) + 8 * (warp >> 1); rg < ngroups; rg += 64) {
                        const int r0 = 4 * rg, us0 = u0 - halo + r0;
                        int x = (us0 + 2 * p.W) % p.W;
                        unsigned live = 0;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int us = us0 + i;
                            if (us >= 0 && us < p.P && x != zero_col) live |= 1u << i;
                            if (++x == p.W) x = 0;
                        }
#pragma unroll
                        for (int pn = 0; pn < NP; ++pn) {
                            unsigned lo[4] = {0u, 0u, 0u, 0u}, hi[4] = {0u, 0u, 0u, 0u};
                            if (live) {
                                const unsigned *sw = raw32 + (pn * 8 + ch) * pitchw + c0w + rg;
                                const unsigned w0 = sw[0], w1 = sw[estep], w2 = sw[2 * estep], w3 = sw[3 * estep];
                                const unsigned w4 = sw[4 * estep], w5 = sw[5 * estep], w6 = sw[6 * estep], w7 = sw[7 * estep];
                                const unsigned a0 = __byte_perm(w0, w1, 0x5140), a1 = __byte_perm(w2, w3, 0x5140);
                                const unsigned a2 = __byte_perm(w0, w1, 0x7362), a3 = __byte_perm(w2, w3, 0x7362);
                                const unsigned b0 = __byte_perm(w4, w5, 0x5140), b1 = __byte_perm(w6, w7, 0x5140);
                                const unsigned b2 = __byte_perm(w4, w5, 0x7362), b3 = __byte_perm(w6, w7, 0x7362);
                                lo[0] = __byte_perm(a0, a1, 0x5410); lo[1] = __byte_perm(a0, a1, 0x7632);
                                lo[2] = __byte_perm(a2, a3, 0x5410); lo[3] = __byte_perm(a2, a3, 0x7632);
                                hi[0] = __byte_perm(b0, b1, 0x5410); hi[1] = __byte_perm(b0, b1, 0x7632);
                                hi[2] = __byte_perm(b2, b3, 0x5410); hi[3] = __byte_perm(b2, b3, 0x7632);
                            }
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                uint4 e = make_uint4(0u, 0u, 0u, 0u);
                                if ((live >> i) & 1u) e = expand8(make_uint2(lo[i], hi[i]));
                                *reinterpret_cast<uint4 *>(q1 + pn * panel_bytes + swz(r0 + i, ch)) = e;
                            }
                        }
                    }
                } else {
                    // slab mode: the whole image is staged as [co][P]; bytes are gathered one by one
                    const unsigned char *raw = raw_s + (g & 1) * p.raw_bytes + ch * 8 * p.raw_pitch + p.raw_coff + u0;
                    const int pitch = p.raw_pitch;
#pragma unroll 1
                    for (int r = er; r < nrows; r += 64) {
                        const int us = u0 - halo + r;                // source position of this row
                        const bool live = us >= 0 && us < p.P && (us % p.W) != zero_col;
                        const unsigned o = swz(r, ch);
#pragma unroll
                        for (int pn = 0; pn < NP; ++pn) {
                            uint4 e = make_uint4(0u, 0u, 0u, 0u);
                            if (live) {
                                const unsigned char *s = raw + pn * 64 * pitch + r;
                                const unsigned w0 = s[0] | (s[pitch] << 8) | (s[2 * pitch] << 16) | (s[3 * pitch] << 24);
                                const unsigned w1 = s[4 * pitch] | (s[5 * pitch] << 8) | (s[6 * pitch] << 16) | (s[7 * pitch] << 24);
                                e = expand8(make_uint2(w0, w1));
                            }
                            *reinterpret_cast<uint4 *>(q1 + pn * panel_bytes + o) = e;
                        }
                    }
                }
            }
            fence_async_proxy();
            warp_arrive(&pipe.qt_full[buf]);
            // ---- (5) announce the activation tiles as their copies land
            if (XM == 0) {
                cp_async_wait_pending(1);                        // all but the code request of (3)
                asm volatile("bar.sync 1, %0;" ::"n"(kX) : "memory");
                ok = ok && mbar_wait(&pipe.x_empty[xslot], xphase ^ 1, p.err_flag);
                unsigned char *xt = x_s + xslot * kTileX;
                const int nci = p.Cin - ci0 < 128 ? p.Cin - ci0 : 128;
                const unsigned *xw = reinterpret_cast<const unsigned *>(xraw);
                const int nv = p.P - xc * 8 >= 8 ? 8 : (p.P - xc * 8 > 0 ? p.P - xc * 8 : 0);
                const unsigned m0 = nv >= 2 ? 0xffffffffu : (nv == 1 ? 0xffffu : 0u);
                const unsigned m1 = nv >= 4 ? 0xffffffffu : (nv == 3 ? 0xffffu : 0u);
                const unsigned m2 = nv >= 6 ? 0xffffffffu : (nv == 5 ? 0xffffu : 0u);
                const unsigned m3 = nv >= 8 ? 0xffffffffu : (nv == 7 ? 0xffffu : 0u);
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int row = xr + 64 * i;
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (row < nci && nv > 0) {
                        const int off = row * p.P + xc * 8, wi = off >> 1;
                        const unsigned sh = (off & 1) * 16;
                        const unsigned w0 = xw[wi], w1 = xw[wi + 1], w2 = xw[wi + 2], w3 = xw[wi + 3], w4 = xw[wi + 4];
                        v = make_uint4(__funnelshift_r(w0, w1, sh) & m0, __funnelshift_r(w1, w2, sh) & m1,
                                       __funnelshift_r(w2, w3, sh) & m2, __funnelshift_r(w3, w4, sh) & m3);
                    }
                    *reinterpret_cast<uint4 *>(xt + (i ? xo1 : xo0)) = v;
                }
                fence_async_proxy();
                warp_arrive(&pipe.x_full[xslot]);
                if (++xslot == p.nx) { xslot = 0; xphase ^= 1; }
                // the staged block may be overwritten once every thread is past this point
                asm volatile("bar.sync 1, %0;" ::"n"(kX) : "memory");
            } else {
                for (int k = 0; k < ns; ++k) {
                    cp_async_wait_pending(ns - k);               // later stages and the code request may be pending
                    fence_async_proxy();
                    warp_arrive(&pipe.x_full[aslot]);
                    if (++aslot == p.nx) aslot = 0;
                }
            }
        }
        cp_async_wait_pending(0);
        // ---------------- epilogue: lanes = ci, columns = (ky, co); partials [split][tap][Cout][Cin]
        if (nsegs > 0 && mbar_wait(&pipe.acc, 0, p.err_flag)) {
            tc_fence_after();
            const int q = warp & 3;
            const int ci = ci0 + q * 32 + lane;
            for (int c = warp >> 2; c < 3 * N / 32; c += kXW / 4) {       // 32-column chunks of the three accumulators
                unsigned v[32];
                tmem_ld32(tmem_d + (static_cast<unsigned>(q * 32) << 16) + c * 32, v);
                const int ky = c / (N / 32), cob = co0 + (c - ky * (N / 32)) * 32;
                if (ci < p.Cin) {
                    float *dst = p.partials + ((static_cast<long long>(zsplit) * 9 + ky * 3 + kx) * p.Cout + cob) * p.Cin + ci;
#pragma unroll
                    for (int j = 0; j < 32; ++j) dst[static_cast<long long>(j) * p.Cin] = __uint_as_float(v[j]);
                }
            }
        }
    } else if (lane == 0) {
        constexpr unsigned idesc = make_idesc(128, N, false, true);
        const unsigned x_addr = smem_u32(x_s), qt_addr = smem_u32(qt);
        // descriptors differ only in their address field (16-byte units, no carry out of it)
        unsigned tap_off[3];          // start row (1-ky) W + (1-kx) relative to the stage's first position
#pragma unroll
        for (int ky = 0; ky < 3; ++ky) tap_off[ky] = static_cast<unsigned>((halo + (1 - ky) * p.W + (1 - kx)) * 128) >> 4;
        const unsigned long long bd0 = make_desc(qt_addr, panel_bytes, 1024), ad0 = make_desc(x_addr, 16, 1024);
        bool ok = true;
        int slot = 0, phase = 0;
        unsigned acc_on = 0u;
        for (int sg = 0; sg < nsegs && ok; ++sg) {
            int b, u0, ns;
            seg_of(g0 + sg, b, u0, ns);
            const int buf = sg & 1;
            ok = mbar_wait(&pipe.qt_full[buf], (sg >> 1) & 1, p.err_flag);
            fence_async_proxy();
            tc_fence_after();
            const unsigned long long bd_buf = bd0 + ((static_cast<unsigned>(buf) * NP * panel_bytes) >> 4);
            for (int k = 0; k < ns && ok; ++k) {
                ok = mbar_wait(&pipe.x_full[slot], phase, p.err_flag);
                fence_async_proxy();
                tc_fence_after();
                const unsigned long long ad = ad0 + static_cast<unsigned>(slot * (kTileX >> 4));
                const unsigned long long bd_k = bd_buf + static_cast<unsigned>(k * (64 * 128 >> 4));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {          // 16 positions = 2048 bytes of rows per step
#pragma unroll
                    for (int ky = 0; ky < 3; ++ky)
                        mma_bf16(tmem_d + ky * N, ad + 2 * kk, bd_k + tap_off[ky] + 128 * kk, idesc, kk ? 1u : acc_on);
                }
                acc_on = 1u;
                mma_commit(&pipe.x_empty[slot]);
                if (++slot == p.nx) { slot = 0; phase ^= 1; }
            }
            mma_commit(&pipe.qt_empty[buf]);
        }
        if (nsegs > 0) mma_commit(&pipe.acc);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kXW) {
        __syncwarp();
        tmem_dealloc(tmem_d, TCOLS);
    }
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

template <int XM, int NP>
int run_w(dbp_ctx *ctx, const Sw3P &p, dim3 grid, size_t smem) {
    if (cudaFuncSetAttribute(tc3_dw_shift_kernel<XM, NP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem)) != cudaSuccess)
        return DBP_ECUDA;
    if (launch_chained(tc3_dw_shift_kernel<XM, NP>, grid, dim3(kThreadsW), smem, ctx->stream, p) != cudaSuccess) return DBP_ECUDA;
    return cuda_ok(cudaGetLastError());
}
template <int XM>
int run_np(dbp_ctx *ctx, const Sw3P &p, int np, dim3 grid, size_t smem) {
    return np == 2 ? run_w<XM, 2>(ctx, p, grid, smem) : run_w<XM, 1>(ctx, p, grid, smem);
}

}  // namespace

// Launches the product into ctx->tc_partials ([split][tap][Cout][Cin]) and reports the number of
// splits; DBP_EUNSUPPORTED when the shape does not fit this kernel (the caller uses the generic one).
int launch_tc3_dw_shift(dbp_ctx *ctx, const int8_t *codes, const void *X, const ConvShape &s,
                        int *err_flag, long long *nsplit) {
    const long long P = s.H * s.W;
    if (s.Cout % 64 != 0 || s.Cin % 8 != 0 || s.W > 63 || s.W < 2 || P > (1 << 20)) return DBP_EUNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(codes) & 15u) != 0 || (reinterpret_cast<uintptr_t>(X) & 15u) != 0) return DBP_EUNSUPPORTED;
    const int xm = P % 8 == 0 ? 8 : P % 4 == 0 ? 4 : 0;
    if (xm == 0 && P > 64) return DBP_EUNSUPPORTED;
    const bool row_mode = P % 16 == 0;
    if (!row_mode && P > 1024) return DBP_EUNSUPPORTED;       // slab mode stages the whole [co][P] block of an image
    const int np = s.Cout % 128 == 0 ? 2 : 1, n = 64 * np;
    Sw3P p{};
    p.codes = codes; p.X = static_cast<const __nv_bfloat16 *>(X);
    p.B = static_cast<int>(s.B); p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.W = static_cast<int>(s.W); p.P = static_cast<int>(P);
    p.err_flag = err_flag;
    const int halo = round_up(p.W + 1, 4);
    p.HQ = halo;
    // the longest segment whose buffers fit beside at least four activation tiles
    const int seg_max = p.P < 64 * kMaxStages ? round_up(p.P, 64) : 64 * kMaxStages;
    size_t smem = 0;
    for (int seg = seg_max; seg >= 64; seg -= 64) {
        p.SEG = seg;
        p.RQ = round_up(seg + 2 * halo, 8);
        if (row_mode) {
            p.raw_lead = round_up(halo, 16);
            p.raw_pitch = round_up(p.raw_lead + seg + halo, 32);
            if ((p.raw_pitch / 32) % 2 == 0) p.raw_pitch += 32;          // odd multiple of 32 bytes: see the expansion
            p.raw_coff = p.raw_lead - halo;
            p.raw_bytes = n * p.raw_pitch;
        } else {
            p.raw_lead = -1;
            p.raw_pitch = p.P;
            p.raw_coff = -halo;
            p.raw_bytes = round_up(n * p.P, 16);
        }
        const size_t fixed = 2 * np * static_cast<size_t>(p.RQ) * 128 + 2 * static_cast<size_t>(p.raw_bytes) + (xm == 0 ? kTileX : 0) + 1024 + 64;
        const size_t room = 227 * 1024 - 2048 - fixed;
        if (fixed + 4 * kTileX > 227 * 1024 - 2048) continue;
        p.nx = static_cast<int>(room / kTileX);
        if (p.nx > kMaxNX) p.nx = kMaxNX;
        smem = fixed + static_cast<size_t>(p.nx) * kTileX;
        break;
    }
    if (smem == 0) return DBP_EUNSUPPORTED;
    p.segs_per_img = (p.P + p.SEG - 1) / p.SEG;
    p.nseg = s.B * p.segs_per_img;
    const long long tiles = ((s.Cin + 127) / 128) * (s.Cout / n) * 3;
    const long long split = choose_split(tiles, p.nseg, ctx->sm_count, &p.per_split);
    const size_t nw = static_cast<size_t>(s.Cout) * s.Cin * 9;
    int rc = ws_reserve(ctx, ctx->tc_partials, sizeof(float) * nw * split);
    if (rc) return rc;
    p.partials = static_cast<float *>(ctx->tc_partials.ptr);
    p.nsplit = static_cast<int>(split);
    dim3 grid(static_cast<unsigned>((s.Cin + 127) / 128), static_cast<unsigned>(s.Cout / n), static_cast<unsigned>(3 * split));
    *nsplit = split;
    return xm == 8 ? run_np<8>(ctx, p, np, grid, smem) : xm == 4 ? run_np<4>(ctx, p, np, grid, smem) : run_np<0>(ctx, p, np, grid, smem);
}

}  // namespace dbp
