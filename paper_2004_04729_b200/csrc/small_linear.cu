// Backward pass of a small fp32 linear layer in two chained launches (Algorithm 1 with Eqs. (nsd), (qda),
// (qdw)) instead of five: step size + quantization, then both products.
//
// For gradients of a few tens of thousands of elements every separate kernel (statistics, quantizer,
// weight re-layout, dX, dW) is a handful of microseconds of work behind a launch and a dependent wait,
// and the layer is bound by those.
//   1. small_linear_quantize_kernel: every CTA computes sigma and Delta = s * sigma over the whole
//      tensor by itself (the tensor sits in L2; every CTA adds in the same order, so all of them hold the
//      same Delta and no grid-wide step separates statistics from quantization), then quantizes its own
//      4096 elements into bf16 codes [B][N rounded up to 8] and counts the non-zero and clipped ones.
//      The first CTA publishes Delta; the second kernel adds up the counts.
//   2. small_linear_products_kernel: every CTA owns one 64 x 64 tile of dW or of dX and accumulates it
//      on the tensor cores: the codes are exact in bf16, the fp32 operand (X or W) is split into two
//      bf16 pieces (the value rounded to bf16 and what that left over, rounded again: the pair is within
//      2^-18 of the value), so a k-step is two warp-level MMAs with fp32 accumulation; Delta is applied
//      once at the end. Warp-level MMAs (not the CTA-wide ones with accumulators in tensor memory)
//      because a whole tile is a few hundred of them and nothing here can hide a tensor-memory
//      allocation, a commit and a read-back. The dW tiles of column 0 add up the bias gradient.
// The second kernel is launched with programmatic stream serialization: it becomes resident while the first
// runs, loads its first tiles of X and W, and reads the codes as soon as the first one has finished.
#include "dbp_internal.cuh"

namespace dbp {

namespace {

constexpr int kThreads = 512;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kRows = 64, kCols = 64, kRed = 64;      // output tile and reduction chunk
constexpr int kPitch = 72;                            // halfwords per shared-memory row: a 16-byte multiple whose eight
                                                      // consecutive rows fall into different 16-byte bank groups
constexpr int kQuantPerCta = kThreads * 8;            // elements a CTA of the first kernel quantizes
constexpr unsigned long long kGamma = 0x9E3779B97F4A7C15ull;
constexpr float kMagic = 12582912.0f;                 // 1.5 * 2^23: floats in [2^23, 2^24) have unit spacing

__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
// u = (2k+1) 2^-24, k = top 23 bits of h
__device__ __forceinline__ float dither(unsigned h) {
    return __uint_as_float(__funnelshift_r(h, 0x7fu, 9)) - 0.99999994f;
}

__device__ __forceinline__ unsigned smem_addr(const void *p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }
// four 8x8 matrices of 16-bit elements from shared memory: lane l gives the address of row l % 8 of matrix l / 8;
// register m of lane (g, tig) receives elements (g, 2 tig) and (g, 2 tig + 1) of matrix m, or, transposed,
// elements (2 tig, g) and (2 tig + 1, g)
__device__ __forceinline__ void ldmatrix_x4(unsigned (&r)[4], unsigned addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(unsigned (&r)[4], unsigned addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D += A (16 x 16, row-major fragments) * B (16 x 8, column-major fragments), bf16 in, fp32 accumulate
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

struct SmallLinP {
    const float *delta, *X, *W;   // [B][N], [B][K], [N][K]
    const uint8_t *mask;          // not null: delta is delta_a and the gradient is delta_a where mask != 0, else 0
    const float *delta_in;        // used when scale <= 0
    float scale;
    long long B, N, K, Np;        // Np: N rounded up to 8, the row pitch of the codes
    unsigned long long seed;
    float *dW, *dX, *db;          // any may be null (not both products)
    DeviceState *st;
    float *delta_set;             // second place the step size goes to (may be null)
    unsigned short *codes;        // bf16 [B][Np]
    unsigned *slots;              // one non-zero count per CTA of the first kernel
    int tiles_k, n_dw, n_dx, n_qctas;
    int vec4;                     // K % 4 == 0: 16-byte accesses along K
};

// ---------------------------------------------------------------- step size and codes
__global__ void __launch_bounds__(kThreads)
small_linear_quantize_kernel(const SmallLinP p) {
    __shared__ double red1[kThreads / 32], red2[kThreads / 32];
    __shared__ unsigned cnt_s[2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    chain_wait();
    chain_release();
    const long long n = p.B * p.N;
    if (tid < 2) cnt_s[tid] = 0u;

    // step size: shifted moments about the first element, fp32 inside a 16-byte load, fp64 across
    float delta;
    bool nonfinite = false;
    if (p.scale > 0.f) {
        const bool masked = p.mask != nullptr;
        const float pivot = (!masked || __ldg(p.mask)) ? __ldg(p.delta) : 0.f;
        const uchar4 *m4 = reinterpret_cast<const uchar4 *>(p.mask);
        double d1 = 0.0, d2 = 0.0;
        const long long nvec = n / 4;
        const float4 *v4 = reinterpret_cast<const float4 *>(p.delta);
        constexpr int kU = 20;                          // loads in flight per thread: one round trip for 10 K vectors
        for (long long i0 = 0; i0 < nvec; i0 += kThreads * kU) {
            float4 v[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const long long i = i0 + u * kThreads + tid;
                v[u] = i < nvec ? __ldg(v4 + i) : make_float4(pivot, pivot, pivot, pivot);
                if (masked && i < nvec) {
                    const uchar4 m = __ldg(m4 + i);
                    v[u].x = m.x ? v[u].x : 0.f; v[u].y = m.y ? v[u].y : 0.f;
                    v[u].z = m.z ? v[u].z : 0.f; v[u].w = m.w ? v[u].w : 0.f;
                }
            }
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const float c0 = v[u].x - pivot, c1 = v[u].y - pivot, c2 = v[u].z - pivot, c3 = v[u].w - pivot;
                const float s1 = (c0 + c1) + (c2 + c3);
                const float s2 = fmaf(c0, c0, fmaf(c1, c1, fmaf(c2, c2, c3 * c3)));
                d1 += static_cast<double>(s1);
                d2 += static_cast<double>(s2);
            }
        }
        if (tid == 0)
            for (long long i = nvec * 4; i < n; ++i) {
                const float xi = (!masked || __ldg(p.mask + i)) ? __ldg(p.delta + i) : 0.f;
                const double c = static_cast<double>(xi) - static_cast<double>(pivot);
                d1 += c;
                d2 += c * c;
            }
        d1 = warp_sum(d1);
        d2 = warp_sum(d2);
        if (lane == 0) { red1[warp] = d1; red2[warp] = d2; }
        __syncthreads();
        double a = 0.0, b = 0.0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) { a += red1[w]; b += red2[w]; }
        if (!isfinite(a) || !isfinite(b)) {
            nonfinite = true;
            delta = 0.f;
        } else {
            const double mean = a / static_cast<double>(n);
            double var = b / static_cast<double>(n) - mean * mean;
            if (var < 0.0) var = 0.0;
            delta = static_cast<float>(static_cast<double>(p.scale) * sqrt(var));
        }
    } else {
        delta = __ldg(p.delta_in);
    }
    const bool live = (delta > 0.f) && (delta < __int_as_float(0x7f800000));
    const float inv = live ? __fdiv_rn(1.0f, delta) : 0.f;

    // codes of this thread's eight consecutive elements (the first index is even: a pair shares a draw)
    const long long e0 = static_cast<long long>(blockIdx.x) * kQuantPerCta + static_cast<long long>(tid) * 8;
    unsigned nnz = 0, sat = 0;
    if (e0 < n) {
        float f[8];
        unsigned long long z = p.seed + (static_cast<unsigned long long>(e0 >> 1) + 1ull) * kGamma;
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            const unsigned long long r = mix64(z);
            z += kGamma;
            const float u[2] = {dither(static_cast<unsigned>(r)), dither(static_cast<unsigned>(r >> 32))};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float q = 0.f;
                if (live && e0 + j + h < n) {
                    const float xe = (p.mask == nullptr || __ldg(p.mask + e0 + j + h)) ? __ldg(p.delta + e0 + j + h) : 0.f;
                    const float t = __fmaf_rn(xe, inv, u[h]);
                    const float tc = fminf(fmaxf(t, -127.f), 127.99999f);      // clipped codes are counted, NaN gives 0
                    const bool num = (t == t);
                    sat += (num && tc != t) ? 1u : 0u;
                    q = num ? __fadd_rd(tc, kMagic) - kMagic : 0.f;
                }
                f[j + h] = q;
                nnz += q != 0.f;
            }
        }
        // to [b][Np]: one division for the first element, then step and wrap; small integers are exact in
        // bf16 (the float's upper half)
        long long b = e0 / p.N;
        long long j = e0 - b * p.N;
        unsigned short *dst = p.codes + b * p.Np + j;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (e0 + i < n) *dst = static_cast<unsigned short>(__float_as_uint(f[i]) >> 16);
            ++dst;
            if (++j == p.N) { j = 0; dst += p.Np - p.N; }
        }
    }
    nnz = __reduce_add_sync(kFull, nnz);
    sat = __reduce_add_sync(kFull, sat);
    __syncthreads();                                     // cnt_s is initialised (and red1 / red2 have been read)
    if (lane == 0) {
        if (nnz) atomicAdd(&cnt_s[0], nnz);
        if (sat) atomicAdd(&cnt_s[1], sat);
    }
    __syncthreads();
    // Every CTA holds the same Delta, so the first one publishes it; the counts of the CTAs are added up by the
    // products kernel, which runs when all of them are done (no election of a last CTA, no extra round trips here).
    if (tid == 0) {
        p.slots[blockIdx.x] = cnt_s[0];
        if (cnt_s[1]) atomicAdd(&p.st->saturated, static_cast<unsigned long long>(cnt_s[1]));
        if (blockIdx.x == 0) {
            p.st->delta = delta;
            if (nonfinite) p.st->nonfinite = 1;
            if (p.delta_set) *p.delta_set = delta;
        }
    }
}

// ---------------------------------------------------------------- both products
__global__ void __launch_bounds__(kThreads)
small_linear_products_kernel(const SmallLinP p) {
    // codes: dX tiles [row][reduction index], dW tiles [reduction index][row] (the order they are stored in either way)
    __shared__ __align__(16) unsigned short As[64 * kPitch];
    // rows of X (dW) or W (dX), [reduction index][column], as two bf16 pieces
    __shared__ __align__(16) unsigned short Bh[kRed * kPitch], Bl[kRed * kPitch];
    __shared__ float db_s[kRows];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const int t = blockIdx.x;
    const bool is_dw = t < p.n_dw;
    const int tt = is_dw ? t : t - p.n_dw;
    const int rt = tt / p.tiles_k, kt = tt - rt * p.tiles_k;
    const long long row0 = static_cast<long long>(rt) * kRows;      // first output row: j (dW) or b (dX)
    const long long k0 = static_cast<long long>(kt) * kCols;
    const long long nrows = is_dw ? p.N : p.B;                       // output rows in all
    const long long nred = is_dw ? p.B : p.N;                        // reduction length
    const float *Bsrc = is_dw ? p.X : p.W;                           // [nred][K]
    const bool do_db = is_dw && kt == 0 && p.db != nullptr;
    if (tid < kRows) db_s[tid] = 0.f;

    // Loads of a chunk: eight consecutive codes per thread, one 16-byte load (dX: row hi, reduction indices
    // lo..lo+7; dW: reduction index hi, rows lo..lo+7), and eight consecutive columns of row hi of X or W.
    const int hi = tid >> 3, lo = (tid & 7) * 8;
    // warp tiling of the 64 x 64 tile: 16 rows x 16 columns per warp (two 16 x 8 accumulators)
    const int wr = (warp >> 2) * 16, wc = (warp & 3) * 16;
    const int g = lane >> 2, tig = lane & 3;
    float acc[2][4] = {};
    float dbacc[8] = {};

    auto load_b = [&](long long r0, float4 (&b_reg)[2]) {
        const long long r = r0 + hi;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            const long long c = k0 + lo + 4 * h;
            if (r < nred) {
                const float *src = Bsrc + r * p.K + c;
                if (p.vec4) {
                    if (c < p.K) v = __ldg(reinterpret_cast<const float4 *>(src));
                } else {
                    if (c + 0 < p.K) v.x = __ldg(src + 0);
                    if (c + 1 < p.K) v.y = __ldg(src + 1);
                    if (c + 2 < p.K) v.z = __ldg(src + 2);
                    if (c + 3 < p.K) v.w = __ldg(src + 3);
                }
            }
            b_reg[h] = v;
        }
    };
    // codes outside the tensor (and the padding of a row) read as zero
    auto load_a = [&](long long r0, uint4 &a_reg) {
        const long long bb = is_dw ? r0 + hi : row0 + hi;            // image (row of delta_z)
        const long long jj = is_dw ? row0 + lo : r0 + lo;            // first of eight output channels
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (bb < p.B && jj < p.N) {
            v = __ldcg(reinterpret_cast<const uint4 *>(p.codes + bb * p.Np + jj));
            const long long left = p.N - jj;                         // valid codes from jj on
            if (left < 8) {
                unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (2 * i >= left) w[i] = 0u;
                    else if (2 * i + 1 >= left) w[i] &= 0xffffu;
                }
                v = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
        a_reg = v;
    };
    // the addresses this lane hands to the 8x8-matrix loads (lane l: row l % 8 of matrix l / 8)
    const int lm = lane >> 3, lr = lane & 7;
    // A, four matrices: (rows 0-7, k 0-7), (rows 8-15, k 0-7), (rows 0-7, k 8-15), (rows 8-15, k 8-15);
    // dW tiles hold them [k][row] and load them transposed
    const unsigned a_base = smem_addr(As) + 2u * (is_dw ? static_cast<unsigned>(((lm >> 1) * 8 + lr) * kPitch + wr + (lm & 1) * 8)
                                                        : static_cast<unsigned>((wr + (lm & 1) * 8 + lr) * kPitch + (lm >> 1) * 8));
    const unsigned a_kstep = 2u * (is_dw ? 16u * kPitch : 16u);
    // B, four matrices: (k 0-7, n 0-7), (k 8-15, n 0-7), (k 0-7, n 8-15), (k 8-15, n 8-15), stored [k][n]: transposed loads
    const unsigned b_off = 2u * static_cast<unsigned>(((lm & 1) * 8 + lr) * kPitch + wc + (lm >> 1) * 8);
    const unsigned bh_base = smem_addr(Bh) + b_off, bl_base = smem_addr(Bl) + b_off;

    // one chunk: registers -> shared memory, the loads of the chunk after next, then the MMAs
    auto step = [&](long long r0, uint4 &a_reg, float4 (&b_reg)[2]) {
        __syncthreads();                                 // the previous chunk has been used
        {
            *reinterpret_cast<uint4 *>(As + hi * kPitch + lo) = a_reg;
            if (do_db) {
                const unsigned w[4] = {a_reg.x, a_reg.y, a_reg.z, a_reg.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    dbacc[2 * i] += __uint_as_float(w[i] << 16);
                    dbacc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
                }
            }
            const float v[8] = {b_reg[0].x, b_reg[0].y, b_reg[0].z, b_reg[0].w, b_reg[1].x, b_reg[1].y, b_reg[1].z, b_reg[1].w};
            unsigned h2[4], l2[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const __nv_bfloat162 hh = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
                const float2 hf = __bfloat1622float2(hh);
                const __nv_bfloat162 ll = __floats2bfloat162_rn(v[2 * i] - hf.x, v[2 * i + 1] - hf.y);
                h2[i] = *reinterpret_cast<const unsigned *>(&hh);
                l2[i] = *reinterpret_cast<const unsigned *>(&ll);
            }
            *reinterpret_cast<uint4 *>(Bh + hi * kPitch + lo) = make_uint4(h2[0], h2[1], h2[2], h2[3]);
            *reinterpret_cast<uint4 *>(Bl + hi * kPitch + lo) = make_uint4(l2[0], l2[1], l2[2], l2[3]);
        }
        __syncthreads();
        if (r0 + 2 * kRed < nred) {                      // in flight during this chunk's and the next one's MMAs
            load_a(r0 + 2 * kRed, a_reg);
            load_b(r0 + 2 * kRed, b_reg);
        }
#pragma unroll
        for (int ks = 0; ks < kRed / 16; ++ks) {
            unsigned a[4], bh[4], bl[4];
            if (is_dw) ldmatrix_x4_trans(a, a_base + ks * a_kstep);
            else ldmatrix_x4(a, a_base + ks * a_kstep);
            ldmatrix_x4_trans(bh, bh_base + ks * 2u * 16u * kPitch);
            ldmatrix_x4_trans(bl, bl_base + ks * 2u * 16u * kPitch);
            mma_bf16_16816(acc[0], a, bh[0], bh[1]);
            mma_bf16_16816(acc[0], a, bl[0], bl[1]);
            mma_bf16_16816(acc[1], a, bh[2], bh[3]);
            mma_bf16_16816(acc[1], a, bl[2], bl[3]);
        }
    };

    uint4 a0, a1 = make_uint4(0u, 0u, 0u, 0u);
    float4 b0[2], b1[2];
    // X and W are inputs of the call: their first chunks are on their way before the first kernel is done
    load_b(0, b0);
    if (kRed < nred) load_b(kRed, b1);
    chain_wait();
    chain_release();
    const float delta = __ldcg(&p.st->delta);
    const float dscale = (delta > 0.f && delta < __int_as_float(0x7f800000)) ? delta : 0.f;
    if (blockIdx.x == 0 && warp == 0) {                  // nnz of the step: the first kernel's per-CTA counts
        unsigned long long total = 0;
        for (int i = lane; i < p.n_qctas; i += 32) total += __ldcg(p.slots + i);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(kFull, total, o);
        if (lane == 0) p.st->nnz = total;
    }
    load_a(0, a0);
    if (kRed < nred) load_a(kRed, a1);
    for (long long r0 = 0; r0 < nred; r0 += 2 * kRed) {
        step(r0, a0, b0);
        if (r0 + kRed < nred) step(r0 + kRed, a1, b1);
    }

    // the tile, scaled by Delta once: accumulator t holds rows g and g + 8, columns 2 tig, 2 tig + 1 of n-tile t
    float *out = is_dw ? p.dW : p.dX;
#pragma unroll
    for (int tn = 0; tn < 2; ++tn) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const long long row = row0 + wr + g + 8 * h;
            const long long col = k0 + wc + 8 * tn + 2 * tig;
            if (row >= nrows || col >= p.K) continue;
            float *dst = out + row * p.K + col;
            const float v0 = acc[tn][2 * h] * dscale, v1 = acc[tn][2 * h + 1] * dscale;
            if ((p.K & 1) == 0) {
                *reinterpret_cast<float2 *>(dst) = make_float2(v0, v1);
            } else {
                dst[0] = v0;
                if (col + 1 < p.K) dst[1] = v1;
            }
        }
    }
    if (do_db) {                                         // threads that share lo hold the same eight rows
#pragma unroll
        for (int i = 0; i < 8; ++i) atomicAdd(&db_s[lo + i], dbacc[i]);     // small integers: exact in any order
        __syncthreads();
        if (tid < kRows && row0 + tid < p.N) p.db[row0 + tid] = db_s[tid] * dscale;
    }
}

}  // namespace

// Shapes the two-launch path takes: small enough that every CTA of the first kernel can read the whole
// gradient for its statistics (gradient size times CTA count is the L2 traffic of that: at most 32 x 2^17 elements).
bool small_linear_fits(const dbp_ctx *ctx, long long B, long long N, long long K, bool want_dw, bool want_dx) {
    const long long n = B * N;
    if (n <= 0 || n > (1ll << 17) || K <= 0 || K > (1ll << 24)) return false;
    const long long tiles_k = (K + kCols - 1) / kCols;
    const long long n_dw = want_dw ? ((N + kRows - 1) / kRows) * tiles_k : 0;
    const long long n_dx = want_dx ? ((B + kRows - 1) / kRows) * tiles_k : 0;
    const long long ctas = n_dw + n_dx;
    if (ctas <= 0 || ctas > 65535) return false;
    const long long qctas = (n + kQuantPerCta - 1) / kQuantPerCta;
    return qctas * static_cast<long long>(sizeof(unsigned)) <= static_cast<long long>(sizeof(double)) * 2 * ctx->partial_blocks;
}

int launch_small_linear(dbp_ctx *ctx, const float *delta, const float *X, const float *W, long long B, long long N,
                        long long K, unsigned long long seed, float scale, const float *delta_in, float *dW, float *dX,
                        float *db, float *delta_set, const uint8_t *mask) {
    SmallLinP p{};
    p.delta = delta; p.X = X; p.W = W; p.delta_in = delta_in; p.scale = scale; p.mask = mask;
    p.B = B; p.N = N; p.K = K; p.Np = (N + 7) / 8 * 8; p.seed = seed;
    p.dW = dW; p.dX = dX; p.db = dW ? db : nullptr;
    p.st = ctx->state; p.delta_set = delta_set;
    const int k = ctx->code_set;
    if (int rc = ws_reserve(ctx, ctx->codes16[k], static_cast<size_t>(B) * p.Np * 2 + 64)) return rc;
    p.codes = static_cast<unsigned short *>(ctx->codes16[k].ptr);
    p.slots = reinterpret_cast<unsigned *>(ctx->partials);
    p.tiles_k = static_cast<int>((K + kCols - 1) / kCols);
    p.n_dw = dW ? static_cast<int>((N + kRows - 1) / kRows) * p.tiles_k : 0;
    p.n_dx = dX ? static_cast<int>((B + kRows - 1) / kRows) * p.tiles_k : 0;
    p.vec4 = (K % 4 == 0) ? 1 : 0;
    const long long n = B * N;
    const unsigned qctas = static_cast<unsigned>((n + kQuantPerCta - 1) / kQuantPerCta);
    p.n_qctas = static_cast<int>(qctas);
    if (int rc = cuda_ok(launch_chained(small_linear_quantize_kernel, dim3(qctas), dim3(kThreads), 0, ctx->stream, p))) return rc;
    return cuda_ok(launch_chained(small_linear_products_kernel, dim3(static_cast<unsigned>(p.n_dw + p.n_dx)), dim3(kThreads), 0,
                                  ctx->stream, p));
}

}  // namespace dbp
