// Dense tensor-core weight gradient of 1x1 convolutions and linear layers, bf16 operands:
//   dW[co][ci] = Delta * sum_r q[r,co] X[r,ci],   r = (image, position) flattened
//   M = co (128), N = ci (NT), K = rows in stages of 64; both operands K-major.
//
// The kernel is bound by HBM (every byte of X and of the codes is read once), so its pipeline
// is built to keep many bytes in flight per SM: all global reads are cp.async copies issued
// several stages ahead -- X straight into its 128-byte-swizzled operand tile, the int8 codes
// into a raw staging tile -- and tracked by cp.async groups; the producer warps then expand
// the staged codes to bf16 from shared memory (no global latency on that path) while the next
// stages' copies are already under way. One more warp issues the MMAs. K is split across CTAs;
// partial blocks go to a workspace and a small kernel sums them and applies Delta.
#include "tc_common.cuh"

namespace dbp {

namespace {

using namespace tc;

constexpr int kPW = 8;
constexpr int kP = kPW * 32;
constexpr int kRS = kP / 8;              // rows between two chunks of one producer thread
constexpr int kThreadsDw = kP + 32;
constexpr int kMaxS = 5;
constexpr int kKT = 64;

struct DwP {
    const int8_t *codes;          // [B][Cout][P]
    const __nv_bfloat16 *X;       // [B][Cin][P]
    float *partials;              // [ksplit][Cout][Cin]
    int Cin, Cout;
    long long P, rows;
    int stages;
    long long kstages, per_split;
    int *err_flag;
};

struct PipeDw {
    unsigned long long full[kMaxS], empty[kMaxS], acc;
    unsigned tmem_base;
};

// G = rows per aligned, image-contained group: 8 (P % 8 == 0), 4 (P % 4 == 0) or 1 (any P).
// G = 0 is the slab mode for small planes (9 <= P <= 64) of any alignment: a K stage is one
// image (its P positions, zero-padded to 64); the [128 co][P] code block and the [NT ci][P]
// activation block of an image are contiguous in memory, so both are staged by 16-byte
// cp.async copies and re-laid into the operand tiles from shared memory.
template <int NT, int G>
__global__ void __launch_bounds__(kThreadsDw) tc_dw_async_kernel(const DwP p) {
    constexpr int A_BYTES = 128 * 128;
    constexpr int B_BYTES = NT * 128;
    constexpr int RAW_BYTES = 128 * 64;
    constexpr int XRAW_BYTES = G == 0 ? NT * 128 : 0;       // slab mode: staged activations
    constexpr int STAGE = A_BYTES + B_BYTES + RAW_BYTES + XRAW_BYTES;
    constexpr int NGRP = G == 0 ? 1 : 8 / G;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ PipeDw pipe;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int co0 = blockIdx.x * 128, ci0 = blockIdx.y * NT;
    const long long ks0 = blockIdx.z * p.per_split;
    long long ks1 = ks0 + p.per_split;
    if (ks1 > p.kstages) ks1 = p.kstages;
    const int niter = ks1 > ks0 ? static_cast<int>(ks1 - ks0) : 0;
    const int S = p.stages;
    // copies run LA stages ahead; with LA = S - 2 a slot is refilled two MMAs after it was
    // consumed, so producers never wait on the tensor core's latency
    const int LA = S > 2 ? S - 2 : S - 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&pipe.full[s], kPW);             // one arrival per producer warp
            mbar_init(&pipe.empty[s], 1);
        }
        mbar_init(&pipe.acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kPW) tmem_alloc(&pipe.tmem_base, NT);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_d = pipe.tmem_base;

    if (warp < kPW) {
        const int tid = threadIdx.x;
        const int c8 = tid & 7, rsub = tid >> 3;      // chunk column, first of my rows (stride kRS)
        bool ok = true;
        // Addresses are kept incremental: a thread's rows are kRS apart (constant pointer and
        // shared-memory steps) and a stage advances every group by 64 flattened rows.
        const long long xstep = kRS * p.P, cstep = kRS * p.P;
        const unsigned b_off0 = swz(rsub, c8), raw_off0 = rsub * 64 + c8 * 8;
        // Per group: flattened row, position inside its image and the source pointers of my first
        // row, all advanced by 64 rows per stage (a pointer jumps by (C - 1) P when the group
        // moves on to the next image). Row-exists masks and ring position are kept likewise, so a
        // stage costs no division and no 64-bit multiply.
        long long grow[NGRP > 2 ? 1 : NGRP], gp[NGRP > 2 ? 1 : NGRP];
        const __nv_bfloat16 *xptr[NGRP > 2 ? 1 : NGRP];
        const int8_t *cptr[NGRP > 2 ? 1 : NGRP];
        unsigned xmask = 0, cmask = 0;
        const long long xwrap = (p.Cin - 1) * p.P, cwrap = (p.Cout - 1) * p.P;
        if (G > 1) {
#pragma unroll
            for (int g = 0; g < NGRP; ++g) {
                grow[g] = ks0 * kKT + c8 * 8 + g * G;
                const long long gb = grow[g] / p.P;
                gp[g] = grow[g] - gb * p.P;
                xptr[g] = p.X + (gb * p.Cin + ci0 + rsub) * p.P + gp[g];
                cptr[g] = p.codes + (gb * p.Cout + co0 + rsub) * p.P + gp[g];
            }
#pragma unroll
            for (int i = 0; i < NT / kRS; ++i) xmask |= (ci0 + rsub + kRS * i < p.Cin ? 1u : 0u) << i;
#pragma unroll
            for (int i = 0; i < 128 / kRS; ++i) cmask |= (co0 + rsub + kRS * i < p.Cout ? 1u : 0u) << i;
        }
        int is = 0;                 // ring slot of the next stage to fill
        unsigned iparity = 1;       // parity to wait for on its empty barrier
        // copies of local stage j (called for j = 0, 1, 2, ... in order): X chunks into the
        // operand tile, code bytes into the raw tile
        auto issue = [&](int j) {
            const int s = is;
            ok = ok && mbar_wait(&pipe.empty[s], iparity, p.err_flag);
            if (++is == S) { is = 0; iparity ^= 1u; }
            unsigned char *st = smem + s * STAGE;
            unsigned char *b_s = st + A_BYTES, *raw = b_s + B_BYTES;
            const long long r0 = (ks0 + j) * kKT + c8 * 8;
            if (G == 0) {
                const long long b = ks0 + j;                 // this stage's image
                const int P = static_cast<int>(p.P);
                const int nco = p.Cout - co0 < 128 ? p.Cout - co0 : 128, nci = p.Cin - ci0 < NT ? p.Cin - ci0 : NT;
                const int8_t *cs = p.codes + (b * p.Cout + co0) * p.P;
                for (int idx = tid; idx * 16 < nco * P; idx += kP) cp_async16(raw + idx * 16, cs + idx * 16, true);
                const __nv_bfloat16 *xs = p.X + (b * p.Cin + ci0) * p.P;
                unsigned char *rawx = raw + RAW_BYTES;
                for (int idx = tid; idx * 8 < nci * P; idx += kP) cp_async16(rawx + idx * 16, xs + idx * 8, true);
            } else if (G > 1) {
#pragma unroll
                for (int g = 0; g < NGRP; ++g) {
                    const bool gv = grow[g] < p.rows;
                    const __nv_bfloat16 *xs = xptr[g];
                    unsigned char *xd = b_s + b_off0 + g * 8;
#pragma unroll
                    for (int i = 0; i < NT / kRS; ++i) {
                        const bool v = gv && ((xmask >> i) & 1u);
                        if (G == 8) cp_async16(xd, v ? xs : p.X, v);
                        else cp_async_small<8>(xd, v ? xs : p.X, v);
                        xs += xstep;
                        xd += kRS * 128;
                    }
                    const int8_t *cs = cptr[g];
                    unsigned char *cd = raw + raw_off0 + g * 4;
#pragma unroll
                    for (int i = 0; i < 128 / kRS; ++i) {
                        const bool v = gv && ((cmask >> i) & 1u);
                        if (G == 8) cp_async_small<8>(cd, v ? cs : p.codes, v);
                        else cp_async_small<4>(cd, v ? cs : p.codes, v);
                        cs += cstep;
                        cd += kRS * 64;
                    }
                    // next stage: 64 rows further
                    grow[g] += kKT;
                    gp[g] += kKT;
                    xptr[g] += kKT;
                    cptr[g] += kKT;
                    while (gp[g] >= p.P) { gp[g] -= p.P; xptr[g] += xwrap; cptr[g] += cwrap; }
                }
            } else {
                // element-wise: walk the eight rows from (b, p)
                const long long rr = r0 < p.rows ? r0 : 0;
                const long long b0 = rr / p.P, q0 = rr - b0 * p.P;
                const unsigned short *xs = reinterpret_cast<const unsigned short *>(p.X);
                for (int i = 0; i < NT / kRS; ++i) {
                    const int row = rsub + kRS * i, ci = ci0 + row;
                    unsigned short h[8];
                    long long b = b0, pp = q0;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        h[e] = (r0 + e < p.rows && ci < p.Cin) ? __ldg(xs + (b * p.Cin + ci) * p.P + pp) : 0;
                        if (++pp == p.P) { pp = 0; ++b; }
                    }
                    *reinterpret_cast<uint4 *>(b_s + swz(row, c8)) =
                        make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
                }
                for (int i = 0; i < 128 / kRS; ++i) {
                    const int row = rsub + kRS * i, co = co0 + row;
                    unsigned w[2] = {0u, 0u};
                    long long b = b0, pp = q0;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        if (r0 + e < p.rows && co < p.Cout)
                            w[e >> 2] |= (static_cast<unsigned>(__ldg(p.codes + (b * p.Cout + co) * p.P + pp)) & 0xffu) << (8 * (e & 3));
                        if (++pp == p.P) { pp = 0; ++b; }
                    }
                    *reinterpret_cast<uint2 *>(raw + row * 64 + c8 * 8) = make_uint2(w[0], w[1]);
                }
            }
        };
        // every thread closes one cp.async group per stage (empty once the copies run out), so
        // "at most LA groups pending" means the copies of stage `it` have landed
        int cslot = 0;              // ring slot of the stage being expanded
        for (int j = 0; j < LA; ++j) {
            if (j < niter) issue(j);
            cp_async_commit();
        }
        for (int it = 0; it < niter; ++it) {
            if (it + LA < niter) issue(it + LA);
            cp_async_commit();
            const int s = cslot;
            if (++cslot == S) cslot = 0;
            cp_async_wait_pending(LA);
            if (G == 0) asm volatile("bar.sync 1, %0;" ::"n"(kP) : "memory");   // slabs are read across threads
            unsigned char *a_s = smem + s * STAGE, *raw = a_s + A_BYTES + B_BYTES;
            if (G == 0) {
                // my chunk covers positions c8*8 .. c8*8+7 of the image; nv of them exist
                const int P = static_cast<int>(p.P);
                const int nv = P - c8 * 8 >= 8 ? 8 : (P - c8 * 8 > 0 ? P - c8 * 8 : 0);
                const int nco = p.Cout - co0 < 128 ? p.Cout - co0 : 128, nci = p.Cin - ci0 < NT ? p.Cin - ci0 : NT;
                // byte masks of the valid positions
                const unsigned m0 = nv >= 4 ? 0xffffffffu : (nv > 0 ? (1u << (8 * nv)) - 1u : 0u);
                const unsigned m1 = nv >= 8 ? 0xffffffffu : (nv > 4 ? (1u << (8 * (nv - 4))) - 1u : 0u);
                const unsigned *rawc_w = reinterpret_cast<const unsigned *>(raw);
#pragma unroll
                for (int i = 0; i < 128 / kRS; ++i) {
                    const int row = rsub + kRS * i;
                    uint4 e = make_uint4(0u, 0u, 0u, 0u);
                    if (row < nco && nv > 0) {
                        // eight bytes from byte offset row * P + c8 * 8 (any alignment)
                        const int off = row * P + c8 * 8, wi = off >> 2;
                        const unsigned sel = 0x3210u + 0x1111u * static_cast<unsigned>(off & 3);
                        const unsigned w0 = rawc_w[wi], w1 = rawc_w[wi + 1], w2 = rawc_w[wi + 2];
                        e = expand8(make_uint2(__byte_perm(w0, w1, sel) & m0, __byte_perm(w1, w2, sel) & m1));
                    }
                    *reinterpret_cast<uint4 *>(a_s + swz(row, c8)) = e;
                }
                const unsigned *rawx_w = reinterpret_cast<const unsigned *>(raw + RAW_BYTES);
                unsigned char *b_t = a_s + A_BYTES;
                // 16-bit element masks for the four words of a chunk
                const unsigned x0 = nv >= 2 ? 0xffffffffu : (nv == 1 ? 0xffffu : 0u);
                const unsigned x1 = nv >= 4 ? 0xffffffffu : (nv == 3 ? 0xffffu : 0u);
                const unsigned x2 = nv >= 6 ? 0xffffffffu : (nv == 5 ? 0xffffu : 0u);
                const unsigned x3 = nv >= 8 ? 0xffffffffu : (nv == 7 ? 0xffffu : 0u);
#pragma unroll
                for (int i = 0; i < NT / kRS; ++i) {
                    const int row = rsub + kRS * i;
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (row < nci && nv > 0) {
                        // eight bf16 from element offset row * P + c8 * 8 (2-byte aligned)
                        const int off = row * P + c8 * 8, wi = off >> 1;
                        const unsigned sh = (off & 1) * 16;
                        const unsigned w0 = rawx_w[wi], w1 = rawx_w[wi + 1], w2 = rawx_w[wi + 2], w3 = rawx_w[wi + 3],
                                       w4 = rawx_w[wi + 4];
                        v = make_uint4(__funnelshift_r(w0, w1, sh) & x0, __funnelshift_r(w1, w2, sh) & x1,
                                       __funnelshift_r(w2, w3, sh) & x2, __funnelshift_r(w3, w4, sh) & x3);
                    }
                    *reinterpret_cast<uint4 *>(b_t + swz(row, c8)) = v;
                }
            } else {
#pragma unroll
            for (int i = 0; i < 128 / kRS; ++i) {
                const int row = rsub + kRS * i;
                const uint2 c = *reinterpret_cast<const uint2 *>(raw + row * 64 + c8 * 8);
                *reinterpret_cast<uint4 *>(a_s + swz(row, c8)) = expand8(c);
            }
            }
            fence_async_proxy();
            warp_arrive(&pipe.full[s]);
        }
        // ---------------- epilogue: lanes = co rows, columns = ci -> partial block of this split
        if (niter > 0 && mbar_wait(&pipe.acc, 0, p.err_flag)) {
            tc_fence_after();
            const int q = warp & 3, part = warp >> 2;      // lane quarter, first 32-column chunk
            const int co = co0 + q * 32 + lane;
            float *dst_row = p.partials + (static_cast<long long>(blockIdx.z) * p.Cout + co) * p.Cin + ci0;
#pragma unroll 1
            for (int c0 = part * 32; c0 < NT; c0 += 32 * (kPW / 4)) {
                unsigned r[32];
                tmem_ld32(tmem_d + (static_cast<unsigned>(q * 32) << 16) + c0, r);
                if (co < p.Cout) {
                    if (ci0 + c0 + 32 <= p.Cin) {   // Cin % 8 == 0, ci0 % 64 == 0: 16-byte aligned
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<uint4 *>(dst_row + c0 + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (ci0 + c0 + j < p.Cin) dst_row[c0 + j] = __uint_as_float(r[j]);
                    }
                }
            }
        }
    } else if (lane == 0) {
        constexpr unsigned idesc = make_idesc(128, NT, false, false);
        bool ok = true;
        int s = 0;
        unsigned parity = 0;
        for (int it = 0; it < niter && ok; ++it) {
            ok = mbar_wait(&pipe.full[s], parity, p.err_flag);
            fence_async_proxy();
            tc_fence_after();
            const unsigned a_addr = smem_u32(smem + s * STAGE), b_addr = a_addr + A_BYTES;
            const unsigned long long ad = make_desc(a_addr, 16, 1024), bd = make_desc(b_addr, 16, 1024);
#pragma unroll
            for (int k = 0; k < kKT / 16; ++k)
                mma_bf16(tmem_d, ad + 2 * k, bd + 2 * k, idesc, (it > 0 || k > 0) ? 1u : 0u);
            mma_commit(&pipe.empty[s]);
            if (++s == S) { s = 0; parity ^= 1u; }
        }
        if (niter > 0) mma_commit(&pipe.acc);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kPW) {
        __syncwarp();
        tmem_dealloc(tmem_d, NT);
    }
}

// dW = Delta * sum over splits of the partial blocks. With few weights and many splits the sum
// is a latency chain, so a block spreads the splits over its eight warps (lanes = 32 consecutive
// float4 of the block) and combines the eight partial sums in a fixed order.
__global__ void __launch_bounds__(256) tc_dw_sum_kernel(const float4 *__restrict__ partials, int ksplit,
                                                        long long n4, const float *__restrict__ delta_p,
                                                        float4 *__restrict__ dW) {
    __shared__ float4 sh[8][32];
    const int e = threadIdx.x & 31, sg = threadIdx.x >> 5;
    const long long i4 = blockIdx.x * 32ll + e;
    chain_wait();
    chain_release();
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i4 < n4) {
#pragma unroll 4
        for (int s = sg; s < ksplit; s += 8) {
            const float4 v = __ldcs(partials + s * n4 + i4);
            a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        }
    }
    sh[sg][e] = a;
    __syncthreads();
    if (sg == 0 && i4 < n4) {
#pragma unroll
        for (int g = 1; g < 8; ++g) {
            const float4 v = sh[g][e];
            a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        }
        const float delta = *delta_p;
        dW[i4] = make_float4(a.x * delta, a.y * delta, a.z * delta, a.w * delta);
    }
}

template <int NT, int G>
int run(dbp_ctx *ctx, const DwP &p, dim3 grid, size_t smem) {
    if (cudaFuncSetAttribute(tc_dw_async_kernel<NT, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem)) != cudaSuccess)
        return DBP_ECUDA;
    note_launch();
    tc_dw_async_kernel<NT, G><<<grid, kThreadsDw, smem, ctx->stream>>>(p);
    return cuda_ok(cudaGetLastError());
}

template <int NT>
int run_g(dbp_ctx *ctx, const DwP &p, dim3 grid, size_t smem, bool slab) {
    if (slab) return run<(NT > 128 ? 128 : NT), 0>(ctx, p, grid, smem);
    if (p.P % 8 == 0) return run<NT, 8>(ctx, p, grid, smem);
    if (p.P % 4 == 0) return run<NT, 4>(ctx, p, grid, smem);
    return run<NT, 1>(ctx, p, grid, smem);
}

}  // namespace

int launch_tc_dw(dbp_ctx *ctx, const int8_t *codes, const void *X, const float *delta_p,
                 const ConvShape &s, float *dW, int *err_flag) {
    DwP p{};
    p.codes = codes; p.X = static_cast<const __nv_bfloat16 *>(X);
    p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.P = s.H * s.W; p.rows = s.B * p.P;
    p.err_flag = err_flag;
    // small planes of awkward size: one image per K stage, staged as contiguous slabs
    const bool slab = p.P % 4 != 0 && p.P >= 9 && p.P <= 64 && s.Cout % 16 == 0 && s.Cin % 8 == 0;
    p.kstages = slab ? s.B : (p.rows + kKT - 1) / kKT;
    const int nt = slab ? (s.Cin > 64 ? 128 : 64) : s.Cin >= 256 ? 256 : s.Cin > 64 ? 128 : 64;
    const long long tiles = ((s.Cout + 127) / 128) * ((s.Cin + nt - 1) / nt);
    const long long split = choose_split(tiles, p.kstages, ctx->sm_count, &p.per_split);
    const int max_s = (nt == 256 || slab) ? 4 : kMaxS;
    p.stages = p.per_split < max_s ? static_cast<int>(p.per_split) : max_s;
    const size_t nw = static_cast<size_t>(s.Cout) * s.Cin;
    int rc = ws_reserve(ctx, ctx->tc_partials, sizeof(float) * nw * split);
    if (rc) return rc;
    p.partials = static_cast<float *>(ctx->tc_partials.ptr);
    dim3 grid(static_cast<unsigned>((s.Cout + 127) / 128), static_cast<unsigned>((s.Cin + nt - 1) / nt),
              static_cast<unsigned>(split));
    const size_t smem = static_cast<size_t>(p.stages) * (128 * 128 + nt * 128 + 128 * 64 + (slab ? nt * 128 : 0)) + 1024 + 64;
    rc = nt == 256 ? run_g<256>(ctx, p, grid, smem, slab) : nt == 128 ? run_g<128>(ctx, p, grid, smem, slab)
                                                                      : run_g<64>(ctx, p, grid, smem, slab);
    if (rc) return rc;
    const long long n4 = static_cast<long long>(nw) / 4;          // Cout * Cin % 4 == 0
    { note_launch(); tc_dw_sum_kernel<<<static_cast<unsigned>((n4 + 31) / 32), 256, 0, ctx->stream>>>(
        reinterpret_cast<const float4 *>(p.partials), static_cast<int>(split), n4, delta_p, reinterpret_cast<float4 *>(dW)); }
    return cuda_ok(cudaGetLastError());
}

int launch_dw_sum(dbp_ctx *ctx, const float *partials, int nsplit, long long nw, const float *delta_p, float *dW) {
    const long long n4 = nw / 4;
    return cuda_ok(launch_chained(tc_dw_sum_kernel, dim3(static_cast<unsigned>((n4 + 31) / 32)), dim3(256), 0, ctx->stream,
                                  reinterpret_cast<const float4 *>(partials), nsplit, n4, delta_p,
                                  reinterpret_cast<float4 *>(dW)));
}

}  // namespace dbp
