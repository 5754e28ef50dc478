// Dense tensor-core path for the two backward products of 1x1 convolutions and linear layers
// with bf16 operands (the fallback above the density crossover): the int8 codes are expanded
// to bf16 on the fly (exact: |q| <= 127) and the products run on the 5th-generation tensor
// cores (tcgen05.mma, fp32 accumulators in tensor memory).
//
//   dW[co][ci] = Delta * sum_r q[r,co] X[r,ci]      M = co, N = ci, K = rows r = (image, position)
//   dX[r][ci]  = Delta * sum_co q[r,co] W[co,ci]    M = rows r,  N = ci, K = co
//
// Operands live in NCHW memory (positions contiguous), whose row pitch is in general not a
// multiple of 16 bytes and whose codes need conversion, so tiles are not fetched by TMA:
// four producer warps load 8-element groups, convert, and store 16-byte chunks directly in
// the 128-byte-swizzled canonical shared-memory layout that the MMA descriptors name. A fifth
// warp issues the MMAs; mbarriers order producers, tensor core and epilogue. Every wait is
// bounded: on expiry the kernel raises a flag in global memory and runs to its end.
#include "dbp_internal.cuh"

namespace dbp {

namespace {

constexpr int kProducerWarps = 4;
constexpr int kThreads = (kProducerWarps + 1) * 32;
constexpr int kStages = 4;
constexpr int kKT = 64;                     // K elements per stage (one 128-byte swizzled row)
constexpr long long kWaitCycles = 1000000000ll;   // a wait gives up after this many SM clocks

__device__ __forceinline__ unsigned smem_u32(const void *p) {
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(unsigned long long *bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1.
// lbo/sbo in bytes. K-major operand: rows of 64 K-elements, 8-row groups sbo apart (lbo unused).
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

// ---- 8-element groups of a [image][channel][position] tensor along the flattened row index
// r = image * P + position, for a fixed channel. `g` (1, 2, 4 or 8) divides P and the row
// index of every group start, so a group never straddles two images and is g-element aligned.
struct RowMap {
    long long P;       // positions per image
    long long C;       // channels of the tensor
    long long rows;    // B * P
    int g;
};

__device__ __forceinline__ uint4 load8_codes_as_bf16(const int8_t *codes, const RowMap &m, long long ch, long long r0) {
    // eight consecutive rows r0..r0+7 of channel ch, int8 -> bf16 (exact)
    unsigned short h[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) h[j] = 0;
    if (m.g == 8) {
        if (r0 < m.rows) {
            const long long b = r0 / m.P, p = r0 - b * m.P;
            const uint2 v = __ldg(reinterpret_cast<const uint2 *>(codes + (b * m.C + ch) * m.P + p));
            const unsigned w[2] = {v.x, v.y};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int c = static_cast<int8_t>((w[j >> 2] >> (8 * (j & 3))) & 0xff);
                h[j] = __bfloat16_as_ushort(__int2bfloat16_rn(c));
            }
        }
    } else {
        for (int j0 = 0; j0 < 8; j0 += m.g) {
            const long long r = r0 + j0;
            if (r >= m.rows) break;
            const long long b = r / m.P, p = r - b * m.P;
            const int8_t *src = codes + (b * m.C + ch) * m.P + p;
            for (int j = 0; j < m.g; ++j) h[j0 + j] = __bfloat16_as_ushort(__int2bfloat16_rn(static_cast<int>(__ldg(src + j))));
        }
    }
    return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
}

__device__ __forceinline__ uint4 load8_bf16(const __nv_bfloat16 *x, const RowMap &m, long long ch, long long r0) {
    if (m.g == 8) {
        if (r0 >= m.rows) return make_uint4(0u, 0u, 0u, 0u);
        const long long b = r0 / m.P, p = r0 - b * m.P;
        return __ldg(reinterpret_cast<const uint4 *>(x + (b * m.C + ch) * m.P + p));
    }
    unsigned short h[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) h[j] = 0;
    for (int j0 = 0; j0 < 8; j0 += m.g) {
        const long long r = r0 + j0;
        if (r >= m.rows) break;
        const long long b = r / m.P, p = r - b * m.P;
        const unsigned short *src = reinterpret_cast<const unsigned short *>(x + (b * m.C + ch) * m.P + p);
        for (int j = 0; j < m.g; ++j) h[j0 + j] = __ldg(src + j);
    }
    return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
}

// byte offset of 16-byte chunk `chunk` (0..7) of row `row` inside a 128-byte-swizzled panel
__device__ __forceinline__ unsigned swz(unsigned row, unsigned chunk) { return row * 128u + ((chunk ^ (row & 7u)) << 4); }

struct TcParams {
    const int8_t *codes;          // [B][Cout][P]
    const __nv_bfloat16 *X;       // [B][Cin][P]      (dW)
    const __nv_bfloat16 *W;       // [Cout][Cin]      (dX)
    const float *delta_p;
    float *dW;                    // [Cout][Cin]
    void *dX;                     // [B][Cin][P], bf16 or fp32
    int dx_f32;
    int Cin, Cout;
    long long P, rows;
    int g;                        // group size for row-wise loads
    int ksplit;                   // dW: CTAs sharing one output tile
    long long kstages;            // dW: 64-row stages in total
    int *err_flag;
};

struct Pipe {
    unsigned long long full[kStages], empty[kStages], acc;
    unsigned tmem_base;
};

// ---------------------------------------------------------------- dW: M = co, N = ci, K = rows
template <int NT>
__global__ void __launch_bounds__(kThreads) tc_dw_kernel(const TcParams p) {
    constexpr int A_BYTES = 128 * 128;          // 128 co rows x 64 k
    constexpr int B_BYTES = NT * 128;           // NT ci rows x 64 k
    constexpr int STAGE = A_BYTES + B_BYTES;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ Pipe pipe;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int co0 = blockIdx.x * 128, ci0 = blockIdx.y * NT;
    // my share of the K stages
    const long long per = (p.kstages + p.ksplit - 1) / p.ksplit;
    const long long ks0 = blockIdx.z * per;
    long long ks1 = ks0 + per;
    if (ks1 > p.kstages) ks1 = p.kstages;
    const int niter = ks1 > ks0 ? static_cast<int>(ks1 - ks0) : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&pipe.full[s], kProducerWarps); mbar_init(&pipe.empty[s], 1); }
        mbar_init(&pipe.acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducerWarps) tmem_alloc(&pipe.tmem_base, NT);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_d = pipe.tmem_base;

    if (warp < kProducerWarps) {
        // ---------------- producers: chunk (row, c8) with c8 = tid % 8 fixed for the thread
        const RowMap mq{p.P, p.Cout, p.rows, p.g}, mx{p.P, p.Cin, p.rows, p.g};
        const int tid = threadIdx.x;           // 0..127
        const int c8 = tid & 7, rsub = tid >> 3;   // 16 rows per pass
        bool ok = true;
        for (int it = 0; it < niter && ok; ++it) {
            const int s = it % kStages;
            ok = mbar_wait(&pipe.empty[s], ((it / kStages) & 1) ^ 1, p.err_flag);
            unsigned char *a_s = smem + s * STAGE, *b_s = a_s + A_BYTES;
            const long long r0 = (ks0 + it) * kKT + c8 * 8;
#pragma unroll 4
            for (int row = rsub; row < 128; row += 16) {
                const int co = co0 + row;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (co < p.Cout) v = load8_codes_as_bf16(p.codes, mq, co, r0);
                *reinterpret_cast<uint4 *>(a_s + swz(row, c8)) = v;
            }
#pragma unroll 4
            for (int row = rsub; row < NT; row += 16) {
                const int ci = ci0 + row;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (ci < p.Cin) v = load8_bf16(p.X, mx, ci, r0);
                *reinterpret_cast<uint4 *>(b_s + swz(row, c8)) = v;
            }
            fence_async_proxy();
            __syncwarp();
            if (lane == 0) mbar_arrive(&pipe.full[s]);
        }
        // ---------------- epilogue: lanes = co rows, columns = ci
        if (niter > 0 && mbar_wait(&pipe.acc, 0, p.err_flag)) {
            tc_fence_after();
            const float delta = *p.delta_p;
            const int co = co0 + warp * 32 + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < NT; c0 += 32) {
                unsigned r[32];
                tmem_ld32(tmem_d + (static_cast<unsigned>(warp * 32) << 16) + c0, r);
                if (co < p.Cout) {
                    float *dst = p.dW + static_cast<long long>(co) * p.Cin + ci0 + c0;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float v = __uint_as_float(r[j]) * delta;
                        if (ci0 + c0 + j < p.Cin && v != 0.f) atomicAdd(dst + j, v);
                    }
                }
            }
        }
    } else if (lane == 0) {
        // ---------------- MMA issuer
        constexpr unsigned idesc = make_idesc(128, NT, false, false);
        bool ok = true;
        for (int it = 0; it < niter && ok; ++it) {
            const int s = it % kStages;
            ok = mbar_wait(&pipe.full[s], (it / kStages) & 1, p.err_flag);
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

// ---------------------------------------------------------------- dX: M = rows, N = ci, K = co
template <int NT>
__global__ void __launch_bounds__(kThreads) tc_dx_kernel(const TcParams p) {
    constexpr int A_BYTES = 2 * kKT * 128;      // two 64-row MN groups x 64 k-rows of 128 bytes
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

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&pipe.full[s], kProducerWarps); mbar_init(&pipe.empty[s], 1); }
        mbar_init(&pipe.acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducerWarps) tmem_alloc(&pipe.tmem_base, NT);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_d = pipe.tmem_base;

    if (warp < kProducerWarps) {
        const RowMap mq{p.P, p.Cout, p.rows, p.g};
        const int tid = threadIdx.x;
        const int c8 = tid & 7, ksub = tid >> 3;    // 16 k-rows per pass
        bool ok = true;
        for (int it = 0; it < niter && ok; ++it) {
            const int s = it % kStages;
            ok = mbar_wait(&pipe.empty[s], ((it / kStages) & 1) ^ 1, p.err_flag);
            unsigned char *a_s = smem + s * STAGE, *b_s = a_s + A_BYTES;
            // A = codes: k-row = co, 64-element MN groups of flattened rows
#pragma unroll 2
            for (int k = ksub; k < kKT; k += 16) {
                const int co = it * kKT + k;
#pragma unroll
                for (int grp = 0; grp < 2; ++grp) {
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (co < p.Cout) v = load8_codes_as_bf16(p.codes, mq, co, row0 + grp * 64 + c8 * 8);
                    *reinterpret_cast<uint4 *>(a_s + grp * PANEL + swz(k, c8)) = v;
                }
            }
            // B = W[co][ci]: k-row = co, 64-element groups of ci
#pragma unroll 2
            for (int k = ksub; k < kKT; k += 16) {
                const int co = it * kKT + k;
#pragma unroll
                for (int grp = 0; grp < NT / 64; ++grp) {
                    const int ci = ci0 + grp * 64 + c8 * 8;
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (co < p.Cout && ci < p.Cin)     // Cin % 8 == 0 is required by the launcher
                        v = __ldg(reinterpret_cast<const uint4 *>(p.W + static_cast<long long>(co) * p.Cin + ci));
                    *reinterpret_cast<uint4 *>(b_s + grp * PANEL + swz(k, c8)) = v;
                }
            }
            fence_async_proxy();
            __syncwarp();
            if (lane == 0) mbar_arrive(&pipe.full[s]);
        }
        // ---------------- epilogue: lanes = rows (image, position), columns = ci
        if (mbar_wait(&pipe.acc, 0, p.err_flag)) {
            tc_fence_after();
            const float delta = *p.delta_p;
            const long long r = row0 + warp * 32 + lane;
            const bool row_ok = r < p.rows;
            const long long b = row_ok ? r / p.P : 0, pp = row_ok ? r - b * p.P : 0;
            const long long base = b * p.Cin * p.P + pp;
#pragma unroll 1
            for (int c0 = 0; c0 < NT; c0 += 32) {
                unsigned v[32];
                tmem_ld32(tmem_d + (static_cast<unsigned>(warp * 32) << 16) + c0, v);
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int ci = ci0 + c0 + j;
                        if (ci >= p.Cin) break;
                        const float f = __uint_as_float(v[j]) * delta;
                        if (p.dx_f32) static_cast<float *>(p.dX)[base + ci * p.P] = f;
                        else static_cast<__nv_bfloat16 *>(p.dX)[base + ci * p.P] = __float2bfloat16_rn(f);
                    }
                }
            }
        }
    } else if (lane == 0) {
        constexpr unsigned idesc = make_idesc(128, NT, true, true);
        bool ok = true;
        for (int it = 0; it < niter && ok; ++it) {
            const int s = it % kStages;
            ok = mbar_wait(&pipe.full[s], (it / kStages) & 1, p.err_flag);
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

int pick_group(long long P) { return P % 8 == 0 ? 8 : P % 4 == 0 ? 4 : P % 2 == 0 ? 2 : 1; }

template <typename K>
int set_smem(K kern, size_t bytes) {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) == cudaSuccess
               ? DBP_OK : DBP_ECUDA;
}

}  // namespace

bool tc_supported(const ConvShape &s, int io) {
    return io == DBP_BF16 && s.k == 1 && s.Cin % 8 == 0;
}

int launch_tc_dw(dbp_ctx *ctx, const int8_t *codes, const void *X, const float *delta_p,
                 const ConvShape &s, float *dW, int *err_flag) {
    TcParams p{};
    p.codes = codes; p.X = static_cast<const __nv_bfloat16 *>(X); p.delta_p = delta_p; p.dW = dW;
    p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.P = s.H * s.W; p.rows = s.B * p.P; p.g = pick_group(p.P);
    p.kstages = (p.rows + kKT - 1) / kKT;
    p.err_flag = err_flag;
    if (cudaMemsetAsync(dW, 0, sizeof(float) * s.Cout * s.Cin, ctx->stream) != cudaSuccess) return DBP_ECUDA;
    const int nt = s.Cin >= 256 ? 256 : s.Cin > 64 ? 128 : 64;
    const long long tiles = ((s.Cout + 127) / 128) * ((s.Cin + nt - 1) / nt);
    long long split = (2LL * ctx->sm_count + tiles - 1) / tiles;
    if (split > p.kstages) split = p.kstages;
    if (split < 1) split = 1;
    p.ksplit = static_cast<int>(split);
    dim3 grid(static_cast<unsigned>((s.Cout + 127) / 128), static_cast<unsigned>((s.Cin + nt - 1) / nt),
              static_cast<unsigned>(split));
    const size_t smem = static_cast<size_t>(kStages) * (128 * 128 + nt * 128) + 1024;
    int rc;
    if (nt == 256) { if ((rc = set_smem(tc_dw_kernel<256>, smem))) return rc; tc_dw_kernel<256><<<grid, kThreads, smem, ctx->stream>>>(p); }
    else if (nt == 128) { if ((rc = set_smem(tc_dw_kernel<128>, smem))) return rc; tc_dw_kernel<128><<<grid, kThreads, smem, ctx->stream>>>(p); }
    else { if ((rc = set_smem(tc_dw_kernel<64>, smem))) return rc; tc_dw_kernel<64><<<grid, kThreads, smem, ctx->stream>>>(p); }
    return cuda_ok(cudaGetLastError());
}

int launch_tc_dx(dbp_ctx *ctx, const int8_t *codes, const void *W, const float *delta_p,
                 const ConvShape &s, void *dX, bool dx_bf16, int *err_flag) {
    TcParams p{};
    p.codes = codes; p.W = static_cast<const __nv_bfloat16 *>(W); p.delta_p = delta_p; p.dX = dX;
    p.dx_f32 = dx_bf16 ? 0 : 1;
    p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.P = s.H * s.W; p.rows = s.B * p.P; p.g = pick_group(p.P);
    p.err_flag = err_flag;
    const int nt = s.Cin >= 256 ? 256 : s.Cin > 64 ? 128 : 64;
    dim3 grid(static_cast<unsigned>((p.rows + 127) / 128), static_cast<unsigned>((s.Cin + nt - 1) / nt));
    const size_t smem = static_cast<size_t>(kStages) * (2 * kKT * 128 + (nt / 64) * kKT * 128) + 1024;
    int rc;
    if (nt == 256) { if ((rc = set_smem(tc_dx_kernel<256>, smem))) return rc; tc_dx_kernel<256><<<grid, kThreads, smem, ctx->stream>>>(p); }
    else if (nt == 128) { if ((rc = set_smem(tc_dx_kernel<128>, smem))) return rc; tc_dx_kernel<128><<<grid, kThreads, smem, ctx->stream>>>(p); }
    else { if ((rc = set_smem(tc_dx_kernel<64>, smem))) return rc; tc_dx_kernel<64><<<grid, kThreads, smem, ctx->stream>>>(p); }
    return cuda_ok(cudaGetLastError());
}

}  // namespace dbp
