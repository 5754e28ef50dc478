// Dense tensor-core input gradient of 1x1 convolutions and linear layers, bf16 operands:
//   dX[r][ci] = Delta * sum_co q[r,co] W[co,ci],   r = (image, position) flattened
//   M = 128 input channels, N = 128 rows r, K = co in stages of 64; both operands MN-major
//   (a k-row holds 64 consecutive input channels / 64 consecutive rows r). With channels on
//   the accumulator's lanes, a thread of the epilogue holds consecutive positions of one
//   channel, which is how dX lies in memory.
//
// Bound by HBM: the codes are read once and dX is written once. All global reads are cp.async
// copies issued ahead of use (weights straight into their swizzled operand tile, code bytes
// into a raw staging tile); the producer warps expand the staged codes to bf16 from shared
// memory; one more warp issues the MMAs.
#include "tc_common.cuh"

namespace dbp {

namespace {

using namespace tc;

constexpr int kPW = 8;
constexpr int kP = kPW * 32;
constexpr int kKS = kP / 16;             // k-rows between two chunks of one producer thread
constexpr int kThreadsDx = kP + 32;
constexpr int kMaxS = 5;
constexpr int kKT = 64;

struct DxP {
    const int8_t *codes;          // [B][Cout][P]
    const __nv_bfloat16 *W;       // [Cout][Cin]
    const float *delta_p;
    void *dX;                     // [B][Cin][P], bf16 or fp32
    int dx_f32;
    int Cin, Cout;
    long long P, rows;
    int stages;
    int *err_flag;
};

struct PipeDx {
    unsigned long long full[kMaxS], empty[kMaxS], acc;
    unsigned tmem_base;
};

// 32-byte store (one full sector); dst 32-byte aligned
__device__ __forceinline__ void st_global_v8(void *dst, const unsigned (&w)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                 "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
}

// G = rows per aligned, image-contained group: 8 (P % 8 == 0), 4 (P % 4 == 0) or 1 (any P).
// G = 0 is the slab mode for small planes (9 <= P <= 64) of any alignment: the [64 co][P] code
// blocks of the images a row tile touches are contiguous in memory and are staged whole by
// 16-byte cp.async copies; the expansion gathers its eight rows from them (a chunk of eight
// rows crosses at most one image boundary).
template <int NT, int G>
__global__ void __launch_bounds__(kThreadsDx) tc_dx_async_kernel(const DxP p) {
    constexpr int A_BYTES = 2 * kKT * 128;          // codes: two 64-row groups x 64 k-rows
    constexpr int B_BYTES = (NT / 64) * kKT * 128;
    constexpr int RAW_BYTES = G == 0 ? 2 * kKT * 128 : kKT * 128;   // 64 co x 128 rows, one byte each (slabs: up to twice that)
    constexpr int STAGE = A_BYTES + B_BYTES + RAW_BYTES;
    constexpr unsigned PANEL = kKT * 128;
    constexpr int NGRP = G == 0 ? 1 : 8 / G;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ PipeDx pipe;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long row0 = static_cast<long long>(blockIdx.x) * 128;
    const int ci0 = blockIdx.y * NT;
    const int niter = (p.Cout + kKT - 1) / kKT;
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
    if (warp == kPW) tmem_alloc(&pipe.tmem_base, 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_d = pipe.tmem_base;

    if (warp < kPW) {
        const int tid = threadIdx.x;
        const int c16 = tid & 15, ksub = tid >> 4;     // my 8-row chunk of the tile, first k-row (stride kKS)
        // where my chunk's groups live: the same for every stage
        const long long r0 = row0 + c16 * 8;
        long long gbase[NGRP > 2 ? 1 : NGRP];          // offset of (image, position) in channel 0, or -1
        if (G > 1) {
#pragma unroll
            for (int g = 0; g < NGRP; ++g) {
                const long long r = r0 + g * G;
                const long long b = r / p.P;
                gbase[g] = r < p.rows ? b * p.Cout * p.P + (r - b * p.P) : -1;
            }
        }
        const int8_t *cptr[NGRP > 2 ? 1 : NGRP];
        if (G > 1) {
#pragma unroll
            for (int g = 0; g < NGRP; ++g) cptr[g] = p.codes + (gbase[g] >= 0 ? gbase[g] : 0) + static_cast<long long>(ksub) * p.P;
        }
        const long long rr0 = r0 < p.rows ? r0 : 0;
        const long long b0 = rr0 / p.P, q0 = rr0 - b0 * p.P;
        // slab mode: staged images img_lo .. img_lo + nimg - 1 as [image][64 co][P]; my copies are
        // the 16-byte chunks tid + kP i; my chunk of eight rows starts at slab byte s_base (k-row 0)
        // and continues in the next image after `split` rows
        const int Pi = static_cast<int>(p.P);
        const long long img_lo = row0 / p.P;
        int s_dst[4], s_base = 0, split = 8, nvr = 0;
        long long s_src[4];
        if (G == 0) {
            const long long last_row = (row0 + 127 < p.rows ? row0 + 127 : p.rows - 1);
            const int nimg = static_cast<int>(last_row / p.P - img_lo) + 1;
            const int per_img = 4 * Pi;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int idx = tid + kP * i;
                s_dst[i] = -1;
                s_src[i] = -1;
                if (idx < nimg * per_img) {
                    const int img = idx / per_img, k16 = idx - img * per_img;
                    s_dst[i] = img * 64 * Pi + 16 * k16;
                    s_src[i] = (img_lo + img) * p.Cout * p.P + 16 * k16;      // image exists: it holds a row of the tile
                }
            }
            nvr = r0 < p.rows ? static_cast<int>(p.rows - r0 < 8 ? p.rows - r0 : 8) : 0;
            s_base = static_cast<int>(b0 - img_lo) * 64 * Pi + static_cast<int>(q0);
            split = Pi - static_cast<int>(q0) < 8 ? Pi - static_cast<int>(q0) : 8;
        }
        bool ok = true;
        // ring position, weight pointer and first k-row of the next stage to fill: advanced per
        // stage, so a stage costs no division and no 64-bit multiply
        int is = 0, co_next = ksub;
        unsigned iparity = 1;
        const __nv_bfloat16 *wptr = p.W + static_cast<long long>(ksub) * p.Cin + ci0 + c16 * 8;
        const bool wcol = ci0 + c16 * 8 < p.Cin;                 // Cin % 8 == 0
        const long long wstep = kKS * static_cast<long long>(p.Cin), cstep = kKS * p.P;
        auto issue = [&](int j) {
            const int s = is;
            ok = ok && mbar_wait(&pipe.empty[s], iparity, p.err_flag);
            if (++is == S) { is = 0; iparity ^= 1u; }
            unsigned char *st = smem + s * STAGE;
            unsigned char *b_s = st + A_BYTES, *raw = b_s + B_BYTES;
            // weights: k-row = co; my chunk column is c16 (8 channels), my k-rows ksub + kKS i.
            // Pointers step by constants: kKS k-rows per i, 64 per stage.
            {
                const __nv_bfloat16 *ws = wptr;
                unsigned char *wd = b_s + (c16 >> 3) * PANEL + swz(ksub, c16 & 7);
#pragma unroll
                for (int i = 0; i < kKT / kKS; ++i) {
                    const bool v = wcol && (co_next + kKS * i < p.Cout);
                    cp_async16(wd, v ? ws : p.W, v);
                    ws += wstep;
                    wd += kKS * 128;
                }
                wptr += static_cast<long long>(kKT) * p.Cin;
            }
            // code bytes: k-row = co, my chunk of 8 rows
            if (G == 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (s_dst[i] >= 0)
                        cp_async16(raw + s_dst[i], p.codes + s_src[i] + static_cast<long long>(j) * kKT * p.P, true);
            } else if (G > 1) {
#pragma unroll
                for (int g = 0; g < NGRP; ++g) {
                    const int8_t *cs = cptr[g];
                    unsigned char *cd = raw + ksub * 128 + c16 * 8 + g * 4;
#pragma unroll
                    for (int i = 0; i < kKT / kKS; ++i) {
                        const bool v = gbase[g] >= 0 && (co_next + kKS * i < p.Cout);
                        if (G == 8) cp_async_small<8>(cd, v ? cs : p.codes, v);
                        else cp_async_small<4>(cd, v ? cs : p.codes, v);
                        cs += cstep;
                        cd += kKS * 128;
                    }
                    cptr[g] += static_cast<long long>(kKT) * p.P;
                }
            } else {
                for (int i = 0; i < kKT / kKS; ++i) {
                    const int k = ksub + kKS * i, co = j * kKT + k;
                    unsigned w[2] = {0u, 0u};
                    long long b = b0, pp = q0;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        if (r0 + e < p.rows && co < p.Cout)
                            w[e >> 2] |= (static_cast<unsigned>(__ldg(p.codes + (b * p.Cout + co) * p.P + pp)) & 0xffu) << (8 * (e & 3));
                        if (++pp == p.P) { pp = 0; ++b; }
                    }
                    *reinterpret_cast<uint2 *>(raw + k * 128 + c16 * 8) = make_uint2(w[0], w[1]);
                }
            }
            co_next += kKT;
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
                // byte e of my chunk is row r0 + e: before `split` it lies in image b0, after it in
                // the next image, 63 P bytes further in the slab layout; rows beyond the end are zero
                const unsigned long long keep = nvr >= 8 ? ~0ull : ((1ull << (8 * nvr)) - 1ull);
                const unsigned long long first = split >= 8 ? ~0ull : ((1ull << (8 * split)) - 1ull);
                const unsigned *raw_w = reinterpret_cast<const unsigned *>(raw);
#pragma unroll
                for (int i = 0; i < kKT / kKS; ++i) {
                    const int k = ksub + kKS * i;
                    uint4 e = make_uint4(0u, 0u, 0u, 0u);
                    if (nvr > 0) {
                        const int off = s_base + k * Pi, wi = off >> 2;
                        const unsigned sel = 0x3210u + 0x1111u * static_cast<unsigned>(off & 3);
                        const unsigned w0 = raw_w[wi], w1 = raw_w[wi + 1], w2 = raw_w[wi + 2];
                        unsigned long long c = __byte_perm(w0, w1, sel) |
                                               (static_cast<unsigned long long>(__byte_perm(w1, w2, sel)) << 32);
                        if (split < nvr) {      // a row of the next image exists (and that image is staged)
                            const int off2 = off + 63 * Pi, wj = off2 >> 2;
                            const unsigned sel2 = 0x3210u + 0x1111u * static_cast<unsigned>(off2 & 3);
                            const unsigned v0 = raw_w[wj], v1 = raw_w[wj + 1], v2 = raw_w[wj + 2];
                            const unsigned long long c2 = __byte_perm(v0, v1, sel2) |
                                                          (static_cast<unsigned long long>(__byte_perm(v1, v2, sel2)) << 32);
                            c = (c & first) | (c2 & ~first);
                        }
                        c &= keep;
                        e = expand8(make_uint2(static_cast<unsigned>(c), static_cast<unsigned>(c >> 32)));
                    }
                    *reinterpret_cast<uint4 *>(a_s + (c16 >> 3) * PANEL + swz(k, c16 & 7)) = e;
                }
            } else {
#pragma unroll
            for (int i = 0; i < kKT / kKS; ++i) {
                const int k = ksub + kKS * i;
                const uint2 c = *reinterpret_cast<const uint2 *>(raw + k * 128 + c16 * 8);
                *reinterpret_cast<uint4 *>(a_s + (c16 >> 3) * PANEL + swz(k, c16 & 7)) = expand8(c);
            }
            }
            fence_async_proxy();
            warp_arrive(&pipe.full[s]);
        }
        // ---------------- epilogue: TMEM lanes = input channels, columns = rows. Warp w takes lane
        // quarter w % 4 and the 32 columns w / 4; a lane stores runs of consecutive positions.
        if (mbar_wait(&pipe.acc, 0, p.err_flag)) {
            tc_fence_after();
            const float delta = *p.delta_p;
            const int q = warp & 3, part = warp >> 2;
            const int ci = ci0 + q * 32 + lane;
            constexpr int RL = G >= 8 ? 8 : (G == 0 ? 1 : G);          // rows per store group
#pragma unroll 1
            for (int c0 = part * 32; c0 < 128; c0 += 32 * (kPW / 4)) {
                unsigned v[32];
                tmem_ld32(tmem_d + (static_cast<unsigned>(q * 32) << 16) + c0, v);
                const long long rfirst = row0 + c0;
                if (ci < p.Cin && rfirst < p.rows) {
                    long long b = rfirst / p.P, pp = rfirst - b * p.P;
                    if (G == 8 && (p.dx_f32 || (p.P & 15) == 0)) {
                        // 32-byte stores: one full sector per lane and instruction
                        constexpr int kStep32 = 0;
                        (void)kStep32;
                        const int step = p.dx_f32 ? 8 : 16;
#pragma unroll
                        for (int j0 = 0; j0 < 32; j0 += 8) {
                            if (!p.dx_f32 && (j0 & 8)) continue;        // bf16: 16 rows per store
                            if (rfirst + j0 < p.rows) {
                                const long long o = (b * p.Cin + ci) * p.P + pp;
                                unsigned w[8];
                                if (p.dx_f32) {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) w[e] = __float_as_uint(__uint_as_float(v[j0 + e]) * delta);
                                    st_global_v8(static_cast<float *>(p.dX) + o, w);
                                } else {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) {
                                        const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[j0 + 2 * e]) * delta,
                                                                                       __uint_as_float(v[(j0 + 2 * e + 1) & 31]) * delta);
                                        w[e] = *reinterpret_cast<const unsigned *>(&h);
                                    }
                                    st_global_v8(static_cast<__nv_bfloat16 *>(p.dX) + o, w);
                                }
                            }
                            pp += step;
                            if (pp >= p.P) { pp -= p.P; ++b; }
                        }
                    } else {
#pragma unroll
                    for (int j0 = 0; j0 < 32; j0 += RL) {
                        if (rfirst + j0 < p.rows) {
                            const long long o = (b * p.Cin + ci) * p.P + pp;
                            if (p.dx_f32) {
                                float *dst = static_cast<float *>(p.dX) + o;
                                if (RL >= 4) {
#pragma unroll
                                    for (int e = 0; e < RL; e += 4)
                                        *reinterpret_cast<float4 *>(dst + e) =
                                            make_float4(__uint_as_float(v[j0 + e]) * delta, __uint_as_float(v[j0 + e + 1]) * delta,
                                                        __uint_as_float(v[j0 + e + 2]) * delta, __uint_as_float(v[j0 + e + 3]) * delta);
                                } else {
                                    dst[0] = __uint_as_float(v[j0]) * delta;
                                }
                            } else {
                                __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.dX) + o;
                                if (RL >= 4) {
                                    unsigned w[RL / 2 > 0 ? RL / 2 : 1];
#pragma unroll
                                    for (int e = 0; e < RL / 2; ++e) {
                                        const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[j0 + 2 * e]) * delta,
                                                                                       __uint_as_float(v[j0 + 2 * e + 1]) * delta);
                                        w[e] = *reinterpret_cast<const unsigned *>(&h);
                                    }
                                    if (RL == 8) *reinterpret_cast<uint4 *>(dst) = make_uint4(w[0], w[1], w[RL / 2 > 2 ? 2 : 0], w[RL / 2 > 3 ? 3 : 0]);
                                    else *reinterpret_cast<uint2 *>(dst) = make_uint2(w[0], w[1]);
                                } else {
                                    dst[0] = __float2bfloat16_rn(__uint_as_float(v[j0]) * delta);
                                }
                            }
                        }
                        pp += RL;
                        if (pp >= p.P) { pp -= p.P; ++b; }      // groups never straddle two images
                    }
                    }
                }
            }
        }
    } else if (lane == 0) {
        constexpr unsigned idesc = make_idesc(128, 128, true, true);
        bool ok = true;
        int s = 0;
        unsigned parity = 0;
        for (int it = 0; it < niter && ok; ++it) {
            ok = mbar_wait(&pipe.full[s], parity, p.err_flag);
            fence_async_proxy();
            tc_fence_after();
            const unsigned q_addr = smem_u32(smem + s * STAGE), w_addr = q_addr + A_BYTES;
            // A = weights (M = channels), B = codes (N = rows)
            const unsigned long long ad = make_desc(w_addr, PANEL, 1024), bd = make_desc(q_addr, PANEL, 1024);
#pragma unroll
            for (int k = 0; k < kKT / 16; ++k)     // 16 k-rows = two 1024-byte groups further per MMA
                mma_bf16(tmem_d, ad + 128 * k, bd + 128 * k, idesc, (it > 0 || k > 0) ? 1u : 0u);
            mma_commit(&pipe.empty[s]);
            if (++s == S) { s = 0; parity ^= 1u; }
        }
        mma_commit(&pipe.acc);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kPW) {
        __syncwarp();
        tmem_dealloc(tmem_d, 128);
    }
}

template <int NT, int G>
int run(dbp_ctx *ctx, const DxP &p, dim3 grid, size_t smem) {
    if (cudaFuncSetAttribute(tc_dx_async_kernel<NT, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem)) != cudaSuccess)
        return DBP_ECUDA;
    note_launch();
    tc_dx_async_kernel<NT, G><<<grid, kThreadsDx, smem, ctx->stream>>>(p);
    return cuda_ok(cudaGetLastError());
}

template <int NT>
int run_g(dbp_ctx *ctx, const DxP &p, dim3 grid, size_t smem, bool slab) {
    if (slab) return run<NT, 0>(ctx, p, grid, smem);
    if (p.P % 8 == 0) return run<NT, 8>(ctx, p, grid, smem);
    if (p.P % 4 == 0) return run<NT, 4>(ctx, p, grid, smem);
    return run<NT, 1>(ctx, p, grid, smem);
}

}  // namespace

bool tc_supported(const ConvShape &s, int io) {
    return io == DBP_BF16 && s.k == 1 && s.Cin % 8 == 0;
}

int launch_tc_dx(dbp_ctx *ctx, const int8_t *codes, const void *W, const float *delta_p,
                 const ConvShape &s, void *dX, bool dx_bf16, int *err_flag) {
    DxP p{};
    p.codes = codes; p.W = static_cast<const __nv_bfloat16 *>(W); p.delta_p = delta_p; p.dX = dX;
    p.dx_f32 = dx_bf16 ? 0 : 1;
    p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.P = s.H * s.W; p.rows = s.B * p.P;
    p.err_flag = err_flag;
    const int niter = static_cast<int>((s.Cout + kKT - 1) / kKT);
    // small planes of awkward size: stage whole [64 co][P] blocks of the touched images
    const bool slab = p.P % 4 != 0 && p.P >= 9 && p.P <= 64 && s.Cout % 64 == 0;
    const int max_s = slab ? 4 : kMaxS;
    p.stages = niter < max_s ? niter : max_s;
    // one CTA: 128 rows x 128 channels; few stages leave room for several CTAs per SM, which
    // overlaps the load, MMA and store phases of different tiles
    dim3 grid(static_cast<unsigned>((p.rows + 127) / 128), static_cast<unsigned>((s.Cin + 127) / 128));
    const size_t smem = static_cast<size_t>(p.stages) * (2 * kKT * 128 + 2 * kKT * 128 + (slab ? 2 : 1) * kKT * 128) + 1024 + 64;
    return run_g<128>(ctx, p, grid, smem, slab);
}

}  // namespace dbp
