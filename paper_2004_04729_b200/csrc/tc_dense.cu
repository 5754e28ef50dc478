// Dense tensor-core path for the two backward products of 1x1 convolutions and linear layers
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
#include "dbp_internal.cuh"

namespace dbp {

namespace {

constexpr int kProducerWarps = 4;
constexpr int kProducers = kProducerWarps * 32;
constexpr int kThreads = kProducers + 32;
constexpr int kMaxStages = 4;
constexpr int kKT = 64;                             // K elements per stage (one 128-byte swizzled row)
constexpr long long kWaitCycles = 1000000000ll;     // a wait gives up after this many SM clocks

__device__ __forceinline__ unsigned smem_u32(const void *p) {
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(unsigned long long *bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// arrival that fires when this thread's earlier cp.async copies have landed
__device__ __forceinline__ void mbar_arrive_on_cp_async(unsigned long long *bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Returns false when the phase did not complete within about half a second.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, unsigned parity, int *err_flag) {
    const unsigned addr = smem_u32(bar);
    const long long t0 = clock64();
    for (;;) {
        unsigned done;
        asm volatile(
            "{\n\t.reg .pred P1;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 P1, [%1], %2;\n\t"
            "selp.b32 %0, 1, 0, P1;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (clock64() - t0 > kWaitCycles) break;
        __nanosleep(20);
    }
    atomicExch(err_flag, 1);
    return false;
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(unsigned *dst_smem, int ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
}
__device__ __forceinline__ void tmem_dealloc(unsigned taddr, int ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols));
}
__device__ __forceinline__ void mma_bf16(unsigned tmem_d, unsigned long long adesc, unsigned long long bdesc,
                                         unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(unsigned long long *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(unsigned taddr, unsigned (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc, bool valid) {
    const int n = valid ? 16 : 0;   // src-size 0: the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(n) : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1; lbo/sbo in bytes.
// K-major operand: rows of 64 K-elements, 8-row groups sbo apart (lbo unused).
// MN-major operand: rows (one per k) of 64 MN-elements, 8-row groups sbo apart, 64-element
// MN groups lbo apart.
__device__ __forceinline__ unsigned long long make_desc(unsigned smem_addr, unsigned lbo, unsigned sbo) {
    unsigned long long d = 0;
    d |= static_cast<unsigned long long>((smem_addr & 0x3ffffu) >> 4);
    d |= static_cast<unsigned long long>((lbo >> 4) & 0x3fffu) << 16;
    d |= static_cast<unsigned long long>((sbo >> 4) & 0x3fffu) << 32;
    d |= 1ull << 46;     // version
    d |= 2ull << 61;     // SWIZZLE_128B
    return d;
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16.
__host__ __device__ constexpr unsigned make_idesc(int M, int N, bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (a_mn_major ? (1u << 15) : 0u) | (b_mn_major ? (1u << 16) : 0u) |
           (static_cast<unsigned>(N >> 3) << 17) | (static_cast<unsigned>(M >> 4) << 24);
}

// byte offset of 16-byte chunk `chunk` (0..7) of row `row` inside a 128-byte-swizzled panel
__device__ __forceinline__ unsigned swz(unsigned row, unsigned chunk) { return row * 128u + ((chunk ^ (row & 7u)) << 4); }

// four int8 codes packed in a word -> two words of packed bf16 (exact).
// byte ^ 0x80 = code + 128 as an unsigned byte; 0x4B0000xx read as a float is 2^23 + xx, so
// subtracting 2^23 + 128 leaves the code as a float whose top 16 bits are its bf16 pattern.
__device__ __forceinline__ void codes4_to_bf16(unsigned w, unsigned &lo, unsigned &hi) {
    const unsigned x = w ^ 0x80808080u;
    const float f0 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7650)) - 8388736.0f;
    const float f1 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7651)) - 8388736.0f;
    const float f2 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7652)) - 8388736.0f;
    const float f3 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7653)) - 8388736.0f;
    lo = __byte_perm(__float_as_uint(f0), __float_as_uint(f1), 0x7632);
    hi = __byte_perm(__float_as_uint(f2), __float_as_uint(f3), 0x7632);
}
__device__ __forceinline__ unsigned short code_to_bf16(int c) {
    return static_cast<unsigned short>(__float_as_uint(static_cast<float>(c)) >> 16);
}

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

__device__ __forceinline__ uint4 load8_bf16_slow(const __nv_bfloat16 *x, long long C, long long P, long long rows,
                                                 long long ch, long long r0, const RowCursor &cur) {
    if (r0 >= rows) return make_uint4(0u, 0u, 0u, 0u);
    const unsigned short *src = reinterpret_cast<const unsigned short *>(x);
    unsigned short h[8];
    long long b = cur.b, pp = cur.p;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        h[j] = (r0 + j < rows) ? __ldg(src + (b * C + ch) * P + pp) : 0;
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

// ---------------------------------------------------------------- dW: M = co, N = ci, K = rows
// Both operands K-major: 128 (co) and NT (ci) rows of 64 consecutive flattened rows r.
template <int NT, bool FAST>
__global__ void __launch_bounds__(kThreads) tc_dw_kernel(const TcParams p) {
    constexpr int A_BYTES = 128 * 128;
    constexpr int B_BYTES = NT * 128;
    constexpr int STAGE = A_BYTES + B_BYTES;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ Pipe pipe;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int co0 = blockIdx.x * 128, ci0 = blockIdx.y * NT;
    const long long ks0 = blockIdx.z * p.per_split;
    long long ks1 = ks0 + p.per_split;
    if (ks1 > p.kstages) ks1 = p.kstages;
    const int niter = ks1 > ks0 ? static_cast<int>(ks1 - ks0) : 0;
    const int stages = p.stages;

    pipe_setup(pipe, stages, FAST ? 2 * kProducers : kProducers, warp, NT);
    const unsigned tmem_d = pipe.tmem_base;

    if (warp < kProducerWarps) {
        // ---------------- producers: chunk (row, c8); c8 = tid % 8 is fixed for the thread
        const int tid = threadIdx.x;
        const int c8 = tid & 7, rsub = tid >> 3;
        bool ok = true;
        for (int it = 0; it < niter && ok; ++it) {
            const int s = it % stages;
            ok = mbar_wait(&pipe.empty[s], ((it / stages) & 1) ^ 1, p.err_flag);
            unsigned char *a_s = smem + s * STAGE, *b_s = a_s + A_BYTES;
            const long long r0 = (ks0 + it) * kKT + c8 * 8;
            const RowCursor cur(r0 < p.rows ? r0 : 0, p.P);
            if (FAST) {   // X needs no conversion: asynchronous 16-byte copies
                const bool row_ok = r0 < p.rows;
                const __nv_bfloat16 *src = p.X + (cur.b * p.Cin + ci0) * p.P + cur.p;
#pragma unroll 4
                for (int row = rsub; row < NT; row += 16) {
                    const bool v = row_ok && (ci0 + row < p.Cin);
                    cp_async16(b_s + swz(row, c8), v ? src + row * p.P : p.X, v);
                }
                mbar_arrive_on_cp_async(&pipe.full[s]);
            }
#pragma unroll
            for (int half = 0; half < 2; ++half) {     // 4 loads in flight, then 4 stores
                uint4 v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = rsub + 16 * (half * 4 + i);
                    const int co = co0 + row;
                    v[i] = (co < p.Cout) ? load8_codes<FAST>(p.codes, p.Cout, p.P, p.rows, co, r0, cur)
                                         : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    *reinterpret_cast<uint4 *>(a_s + swz(rsub + 16 * (half * 4 + i), c8)) = v[i];
            }
            if (!FAST) {
#pragma unroll 2
                for (int row = rsub; row < NT; row += 16) {
                    const int ci = ci0 + row;
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (ci < p.Cin) v = load8_bf16_slow(p.X, p.Cin, p.P, p.rows, ci, r0, cur);
                    *reinterpret_cast<uint4 *>(b_s + swz(row, c8)) = v;
                }
            }
            fence_async_proxy();
            mbar_arrive(&pipe.full[s]);
        }
        // ---------------- epilogue: lanes = co rows, columns = ci -> partial block of this split
        if (niter > 0 && mbar_wait(&pipe.acc, 0, p.err_flag)) {
            tc_fence_after();
            const int co = co0 + warp * 32 + lane;
            float *dst_row = p.partials + (static_cast<long long>(blockIdx.z) * p.Cout + co) * p.Cin + ci0;
#pragma unroll 1
            for (int c0 = 0; c0 < NT; c0 += 32) {
                unsigned r[32];
                tmem_ld32(tmem_d + (static_cast<unsigned>(warp * 32) << 16) + c0, r);
                if (co < p.Cout) {
                    if (ci0 + c0 + 32 <= p.Cin) {   // Cin % 8 == 0 and ci0 % 64 == 0: 16-byte aligned
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
        // ---------------- MMA issuer
        constexpr unsigned idesc = make_idesc(128, NT, false, false);
        bool ok = true;
        for (int it = 0; it < niter && ok; ++it) {
            const int s = it % stages;
            ok = mbar_wait(&pipe.full[s], (it / stages) & 1, p.err_flag);
            fence_async_proxy();
            tc_fence_after();
            const unsigned a_addr = smem_u32(smem + s * STAGE), b_addr = a_addr + A_BYTES;
            const unsigned long long ad = make_desc(a_addr, 16, 1024), bd = make_desc(b_addr, 16, 1024);
#pragma unroll
            for (int k = 0; k < kKT / 16; ++k)     // 32 bytes further along K per MMA
                mma_bf16(tmem_d, ad + 2 * k, bd + 2 * k, idesc, (it > 0 || k > 0) ? 1u : 0u);
            mma_commit(&pipe.empty[s]);
        }
        if (niter > 0) mma_commit(&pipe.acc);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kProducerWarps) {
        __syncwarp();
        tmem_dealloc(tmem_d, NT);
    }
}

// dW = Delta * sum over splits of the partial blocks
__global__ void __launch_bounds__(256) tc_dw_reduce_kernel(const float *__restrict__ partials, int ksplit,
                                                           long long n, const float *__restrict__ delta_p,
                                                           float *__restrict__ dW) {
    const float delta = *delta_p;
    for (long long i = (blockIdx.x * 256ll + threadIdx.x) * 4; i < n; i += gridDim.x * 1024ll) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < ksplit; ++s) {
            const float4 v = __ldcs(reinterpret_cast<const float4 *>(partials + s * n + i));
            a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        }
        *reinterpret_cast<float4 *>(dW + i) = make_float4(a.x * delta, a.y * delta, a.z * delta, a.w * delta);
    }
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
int run_dw(dbp_ctx *ctx, const TcParams &p, dim3 grid, size_t smem) {
    int rc = set_smem(tc_dw_kernel<NT, FAST>, smem);
    if (rc) return rc;
    tc_dw_kernel<NT, FAST><<<grid, kThreads, smem, ctx->stream>>>(p);
    return cuda_ok(cudaGetLastError());
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

int launch_tc_dw(dbp_ctx *ctx, const int8_t *codes, const void *X, const float *delta_p,
                 const ConvShape &s, float *dW, int *err_flag) {
    TcParams p{};
    p.codes = codes; p.X = static_cast<const __nv_bfloat16 *>(X); p.delta_p = delta_p;
    p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.P = s.H * s.W; p.rows = s.B * p.P;
    p.kstages = (p.rows + kKT - 1) / kKT;
    p.err_flag = err_flag;
    const int nt = s.Cin >= 256 ? 256 : s.Cin > 64 ? 128 : 64;
    const long long tiles = ((s.Cout + 127) / 128) * ((s.Cin + nt - 1) / nt);
    // split K so that every SM has a CTA, without empty splits
    long long split = (ctx->sm_count + tiles - 1) / tiles;
    if (split > p.kstages) split = p.kstages;
    if (split < 1) split = 1;
    p.per_split = (p.kstages + split - 1) / split;
    split = (p.kstages + p.per_split - 1) / p.per_split;
    p.ksplit = static_cast<int>(split);
    p.stages = p.per_split < kMaxStages ? static_cast<int>(p.per_split) : kMaxStages;
    const size_t nw = static_cast<size_t>(s.Cout) * s.Cin;
    int rc = ws_reserve(ctx, ctx->tc_partials, sizeof(float) * nw * split);
    if (rc) return rc;
    p.partials = static_cast<float *>(ctx->tc_partials.ptr);
    dim3 grid(static_cast<unsigned>((s.Cout + 127) / 128), static_cast<unsigned>((s.Cin + nt - 1) / nt),
              static_cast<unsigned>(split));
    const size_t smem = static_cast<size_t>(p.stages) * (128 * 128 + nt * 128) + 1024;
    const bool fast = p.P % 8 == 0;
    if (nt == 256) rc = fast ? run_dw<256, true>(ctx, p, grid, smem) : run_dw<256, false>(ctx, p, grid, smem);
    else if (nt == 128) rc = fast ? run_dw<128, true>(ctx, p, grid, smem) : run_dw<128, false>(ctx, p, grid, smem);
    else rc = fast ? run_dw<64, true>(ctx, p, grid, smem) : run_dw<64, false>(ctx, p, grid, smem);
    if (rc) return rc;
    long long blocks = (static_cast<long long>(nw) / 4 + 255) / 256;
    if (blocks > ctx->sm_count * 8) blocks = ctx->sm_count * 8;
    if (blocks < 1) blocks = 1;
    tc_dw_reduce_kernel<<<static_cast<unsigned>(blocks), 256, 0, ctx->stream>>>(
        p.partials, p.ksplit, static_cast<long long>(nw), delta_p, dW);   // Cout*Cin % 4 == 0 since Cin % 8 == 0
    return cuda_ok(cudaGetLastError());
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
