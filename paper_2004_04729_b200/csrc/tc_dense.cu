// Dense tensor-core path for 1x1 convolutions and linear layers: the input-gradient product
// (the weight-gradient product lives in tc_dw1x1.cu).
// with bf16 operands (the fallback above the density crossover): the int8 codes are expanded
// to bf16 on the fly (exact: |q| <= 127) and the products run on the 5th-generation tensor
// cores (tcgen05.mma, fp32 accumulators in tensor memory).
//
//   dW[co][ci] = Delta * sum_r q[r,co] X[r,ci]      M = co, N = ci, K = rows r = (image, position)
//   dX[r][ci]  = Delta * sum_co q[r,co] W[co,ci]    M = rows r,  N = ci, K = co
//
// Operands live in NCHW memory (positions contiguous) whose row pitch is in general not a
// multiple of 16 bytes and whose codes need conversion, so tiles are not fetched by TMA:
// four producer warps load 8-element groups (cp.async where no conversion is needed), convert,
// and store 16-byte chunks directly in the 128-byte-swizzled canonical shared-memory layout
// that the MMA descriptors name. A fifth warp issues the MMAs; mbarriers order producers,
// tensor core and epilogue. Every wait is bounded: on expiry the kernel raises a flag in
// global memory and runs to its end.
#include "tc_common.cuh"

namespace dbp {

namespace {

constexpr int kProducerWarps = 4;
constexpr int kProducers = kProducerWarps * 32;
constexpr int kThreads = kProducers + 32;
constexpr int kMaxStages = 4;
constexpr int kKT = 64;                             // K elements per stage (one 128-byte swizzled row)

using namespace tc;

// Row r of the flattened (image, position) index of a [B][C][P] tensor: walks eight consecutive
// rows from (b, p) without divisions, for any P (P = 1 is a linear layer's [B][C] matrix).
struct RowCursor {
    long long b, p;
    __device__ RowCursor(long long r, long long P) : b(r / P), p(r - (r / P) * P) {}
};

template <bool FAST>
__device__ __forceinline__ uint4 load8_codes(const int8_t *codes, long long C, long long P, long long rows,
                                             long long ch, long long r0, const RowCursor &cur) {
    if (r0 >= rows) return make_uint4(0u, 0u, 0u, 0u);
    if (FAST) {   // P % 8 == 0: the eight rows sit in one image, 8-byte aligned
        const uint2 v = __ldg(reinterpret_cast<const uint2 *>(codes + (cur.b * C + ch) * P + cur.p));
        uint4 o;
        codes4_to_bf16(v.x, o.x, o.y);
        codes4_to_bf16(v.y, o.z, o.w);
        return o;
    }
    unsigned short h[8];
    long long b = cur.b, pp = cur.p;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        h[j] = (r0 + j < rows) ? code_to_bf16(__ldg(codes + (b * C + ch) * P + pp)) : 0;
        if (++pp == P) { pp = 0; ++b; }
    }
    return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
}

struct TcParams {
    const int8_t *codes;          // [B][Cout][P]
    const __nv_bfloat16 *X;       // [B][Cin][P]      (dW)
    const __nv_bfloat16 *W;       // [Cout][Cin]      (dX)
    const float *delta_p;
    float *partials;              // dW: [ksplit][Cout][Cin] partial sums (not yet scaled by Delta)
    void *dX;                     // [B][Cin][P], bf16 or fp32
    int dx_f32;
    int Cin, Cout;
    long long P, rows;
    int stages;
    int ksplit;                   // dW: CTAs sharing one output tile
    long long kstages;            // dW: 64-row stages in total
    long long per_split;          // dW: stages per CTA
    int *err_flag;
};

struct Pipe {
    unsigned long long full[kMaxStages], empty[kMaxStages], acc;
    unsigned tmem_base;
};

__device__ __forceinline__ void pipe_setup(Pipe &pipe, int stages, int full_count, int warp, int ncols) {
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&pipe.full[s], full_count); mbar_init(&pipe.empty[s], 1); }
        mbar_init(&pipe.acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducerWarps) tmem_alloc(&pipe.tmem_base, ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
}

// ---------------------------------------------------------------- dX: M = rows, N = ci, K = co
// Both operands MN-major: k-rows (co) of 64 consecutive flattened rows r (A) / 64 ci (B).
template <int NT, bool FAST>
__global__ void __launch_bounds__(kThreads) tc_dx_kernel(const TcParams p) {
    constexpr int A_BYTES = 2 * kKT * 128;
    constexpr int B_BYTES = (NT / 64) * kKT * 128;
    constexpr int STAGE = A_BYTES + B_BYTES;
    constexpr unsigned PANEL = kKT * 128;       // bytes between 64-element MN groups
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ Pipe pipe;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long row0 = static_cast<long long>(blockIdx.x) * 128;
    const int ci0 = blockIdx.y * NT;
    const int niter = (p.Cout + kKT - 1) / kKT;
    const int stages = p.stages;

    pipe_setup(pipe, stages, 2 * kProducers, warp, NT);
    const unsigned tmem_d = pipe.tmem_base;

    if (warp < kProducerWarps) {
        const int tid = threadIdx.x;
        const int c8 = tid & 7, ksub = tid >> 3;    // 16 k-rows per pass
        // my two 8-row groups of the tile never change
        const long long ra = row0 + c8 * 8, rb = ra + 64;
        const RowCursor cura(ra < p.rows ? ra : 0, p.P), curb(rb < p.rows ? rb : 0, p.P);
        bool ok = true;
        for (int it = 0; it < niter && ok; ++it) {
            const int s = it % stages;
            ok = mbar_wait(&pipe.empty[s], ((it / stages) & 1) ^ 1, p.err_flag);
            unsigned char *a_s = smem + s * STAGE, *b_s = a_s + A_BYTES;
            // B = W[co][ci]: k-row = co, 64-element groups of ci; no conversion: cp.async
#pragma unroll
            for (int i = 0; i < kKT / 16; ++i) {
                const int k = ksub + 16 * i;
                const int co = it * kKT + k;
#pragma unroll
                for (int grp = 0; grp < NT / 64; ++grp) {
                    const int ci = ci0 + grp * 64 + c8 * 8;
                    const bool v = co < p.Cout && ci < p.Cin;     // Cin % 8 == 0
                    cp_async16(b_s + grp * PANEL + swz(k, c8), v ? p.W + static_cast<long long>(co) * p.Cin + ci : p.W, v);
                }
            }
            mbar_arrive_on_cp_async(&pipe.full[s]);
            // A = codes: k-row = co, two 64-element groups of flattened rows
            uint4 va[kKT / 16], vb[kKT / 16];
#pragma unroll
            for (int i = 0; i < kKT / 16; ++i) {
                const int co = it * kKT + ksub + 16 * i;
                va[i] = vb[i] = make_uint4(0u, 0u, 0u, 0u);
                if (co < p.Cout) {
                    va[i] = load8_codes<FAST>(p.codes, p.Cout, p.P, p.rows, co, ra, cura);
                    vb[i] = load8_codes<FAST>(p.codes, p.Cout, p.P, p.rows, co, rb, curb);
                }
            }
#pragma unroll
            for (int i = 0; i < kKT / 16; ++i) {
                const int k = ksub + 16 * i;
                *reinterpret_cast<uint4 *>(a_s + swz(k, c8)) = va[i];
                *reinterpret_cast<uint4 *>(a_s + PANEL + swz(k, c8)) = vb[i];
            }
            fence_async_proxy();
            mbar_arrive(&pipe.full[s]);
        }
        // ---------------- epilogue: lanes = rows (image, position), columns = ci.
        // Each warp turns its 32 rows x 32 columns block through a private shared-memory patch so
        // that a lane stores 16 contiguous bytes of one channel row.
        if (mbar_wait(&pipe.acc, 0, p.err_flag)) {
            tc_fence_after();
            const float delta = *p.delta_p;
            // all MMAs are complete: the stage buffers are free
            constexpr int CS = 192;                          // bytes per column of the patch
            unsigned char *patch = smem + warp * (32 * CS);
            const int es = p.dx_f32 ? 4 : 2;
            const int rows_per_lane = 16 / es;               // rows in one 16-byte store
            const int lanes_per_col = 32 / rows_per_lane;
            const int cols_per_pass = 32 / lanes_per_col;
            const int rr = (lane % lanes_per_col) * rows_per_lane;
            const long long r = row0 + warp * 32 + rr;       // first of my rows when storing
            const long long rb_ = r < p.rows ? r / p.P : 0, rp_ = r < p.rows ? r - rb_ * p.P : 0;
#pragma unroll 1
            for (int c0 = 0; c0 < NT; c0 += 32) {
                unsigned v[32];
                tmem_ld32(tmem_d + (static_cast<unsigned>(warp * 32) << 16) + c0, v);
                if (ci0 + c0 >= p.Cin) break;               // warp-uniform
                if (p.dx_f32) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        *reinterpret_cast<float *>(patch + j * CS + lane * 4) = __uint_as_float(v[j]) * delta;
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        *reinterpret_cast<unsigned short *>(patch + j * CS + lane * 2) =
                            __bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float(v[j]) * delta));
                }
                __syncwarp();
                for (int cb = 0; cb < 32; cb += cols_per_pass) {
                    const int j = cb + lane / lanes_per_col;
                    const int ci = ci0 + c0 + j;
                    if (ci < p.Cin && r < p.rows) {
                        const uint4 val = *reinterpret_cast<const uint4 *>(patch + j * CS + rr * es);
                        if (FAST) {      // the group sits in one image, 16-byte aligned
                            unsigned char *dst = static_cast<unsigned char *>(p.dX) + ((rb_ * p.Cin + ci) * p.P + rp_) * es;
                            *reinterpret_cast<uint4 *>(dst) = val;
                        } else {
                            long long b = rb_, pp = rp_;
                            const unsigned w4[4] = {val.x, val.y, val.z, val.w};
                            for (int e = 0; e < rows_per_lane && r + e < p.rows; ++e) {
                                const long long o = (b * p.Cin + ci) * p.P + pp;
                                if (p.dx_f32) static_cast<float *>(p.dX)[o] = __uint_as_float(w4[e]);
                                else static_cast<unsigned short *>(p.dX)[o] =
                                    static_cast<unsigned short>((w4[e >> 1] >> (16 * (e & 1))) & 0xffff);
                                if (++pp == p.P) { pp = 0; ++b; }
                            }
                        }
                    }
                }
                __syncwarp();
            }
        }
    } else if (lane == 0) {
        constexpr unsigned idesc = make_idesc(128, NT, true, true);
        bool ok = true;
        for (int it = 0; it < niter && ok; ++it) {
            const int s = it % stages;
            ok = mbar_wait(&pipe.full[s], (it / stages) & 1, p.err_flag);
            fence_async_proxy();
            tc_fence_after();
            const unsigned a_addr = smem_u32(smem + s * STAGE), b_addr = a_addr + A_BYTES;
            const unsigned long long ad = make_desc(a_addr, PANEL, 1024), bd = make_desc(b_addr, PANEL, 1024);
#pragma unroll
            for (int k = 0; k < kKT / 16; ++k)     // 16 k-rows = two 1024-byte groups further per MMA
                mma_bf16(tmem_d, ad + 128 * k, bd + 128 * k, idesc, (it > 0 || k > 0) ? 1u : 0u);
            mma_commit(&pipe.empty[s]);
        }
        mma_commit(&pipe.acc);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kProducerWarps) {
        __syncwarp();
        tmem_dealloc(tmem_d, NT);
    }
}

template <typename K>
int set_smem(K kern, size_t bytes) {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) == cudaSuccess
               ? DBP_OK : DBP_ECUDA;
}

template <int NT, bool FAST>
int run_dx(dbp_ctx *ctx, const TcParams &p, dim3 grid, size_t smem) {
    int rc = set_smem(tc_dx_kernel<NT, FAST>, smem);
    if (rc) return rc;
    tc_dx_kernel<NT, FAST><<<grid, kThreads, smem, ctx->stream>>>(p);
    return cuda_ok(cudaGetLastError());
}

}  // namespace

bool tc_supported(const ConvShape &s, int io) {
    return io == DBP_BF16 && s.k == 1 && s.Cin % 8 == 0;
}

int launch_tc_dx(dbp_ctx *ctx, const int8_t *codes, const void *W, const float *delta_p,
                 const ConvShape &s, void *dX, bool dx_bf16, int *err_flag) {
    TcParams p{};
    p.codes = codes; p.W = static_cast<const __nv_bfloat16 *>(W); p.delta_p = delta_p; p.dX = dX;
    p.dx_f32 = dx_bf16 ? 0 : 1;
    p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.P = s.H * s.W; p.rows = s.B * p.P;
    p.err_flag = err_flag;
    const int niter = static_cast<int>((s.Cout + kKT - 1) / kKT);
    p.stages = niter < kMaxStages ? niter : kMaxStages;
    // narrower N tiles leave room for several CTAs per SM, which is what overlaps the load,
    // MMA and store phases of different tiles
    const int nt = s.Cin > 64 ? 128 : 64;
    dim3 grid(static_cast<unsigned>((p.rows + 127) / 128), static_cast<unsigned>((s.Cin + nt - 1) / nt));
    size_t smem = static_cast<size_t>(p.stages) * (2 * kKT * 128 + (nt / 64) * kKT * 128);
    if (smem < 4 * 32 * 192) smem = 4 * 32 * 192;
    smem += 1024;
    const bool fast = p.P % 8 == 0;
    if (nt == 128) return fast ? run_dx<128, true>(ctx, p, grid, smem) : run_dx<128, false>(ctx, p, grid, smem);
    return fast ? run_dx<64, true>(ctx, p, grid, smem) : run_dx<64, false>(ctx, p, grid, smem);
}

}  // namespace dbp
