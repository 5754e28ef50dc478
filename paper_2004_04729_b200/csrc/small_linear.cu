// Backward pass of a small fp32 linear layer in one launch (Algorithm 1 with Eqs. (nsd), (qda), (qdw)):
// step size, dither, quantization and both products.
//
// For gradients of a few tens of thousands of elements every separate kernel (statistics,
// quantizer, dX, dW) is a handful of microseconds of work behind a launch and a dependent wait, and
// the layer is bound by those. Here every CTA owns one 64 x 64 tile of dW or of dX and
//   1. computes sigma and Delta = s * sigma over the whole tensor by itself (the tensor sits in L2;
//      every CTA adds in the same order, so all of them hold the same Delta without a grid barrier),
//   2. quantizes the codes its tile needs as it loads them (the dither is a function of the seed and
//      the element's index, so any CTA can produce any code),
//   3. accumulates its tile with fp32 FMAs over the reduction index and scales by Delta once.
// The tiles whose column index is 0 see every element of delta_z exactly once: they count the
// non-zero and the clipped codes, and the dW ones among them add up the bias gradient. The last CTA
// to finish publishes Delta and nnz to the context.
#include "dbp_internal.cuh"

namespace dbp {

namespace {

constexpr int kThreads = 512;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kRows = 64, kCols = 64, kRed = 32;      // output tile and reduction chunk
constexpr unsigned long long kGamma = 0x9E3779B97F4A7C15ull;

__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// code of element e (Eq. (nsd)): q = floor(fma(x, 1 / Delta, u)), u = (2k+1) 2^-24 from the draw the
// element shares with its neighbour; clipped to [-127, 127] (counted), NaN gives 0
__device__ __forceinline__ float code_of(float x, long long e, unsigned long long seed, float inv, unsigned &sat) {
    const unsigned long long r = mix64(seed + (static_cast<unsigned long long>(e >> 1) + 1ull) * kGamma);
    const unsigned h = (e & 1) ? static_cast<unsigned>(r >> 32) : static_cast<unsigned>(r);
    const float u = __uint_as_float(__funnelshift_r(h, 0x7fu, 9)) - 0.99999994f;
    const float t = __fmaf_rn(x, inv, u);
    const float tc = fminf(fmaxf(t, -127.f), 127.99999f);
    const bool num = (t == t);
    sat += (num && tc != t) ? 1u : 0u;
    return num ? floorf(tc) : 0.f;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

struct SmallLinP {
    const float *delta, *X, *W;   // [B][N], [B][K], [N][K]
    const float *delta_in;        // used when scale <= 0
    float scale;
    long long B, N, K;
    unsigned long long seed;
    float *dW, *dX, *db;          // any may be null (not both products)
    DeviceState *st;
    float *delta_set;             // second place the step size goes to (may be null)
    unsigned *slots;              // one count per counting CTA
    int tiles_k, n_dw, n_dx, count_in_dx, n_count;
    int vec4;                     // K % 4 == 0: 16-byte accesses along K
};

__global__ void __launch_bounds__(kThreads)
small_linear_backward_kernel(const SmallLinP p) {
    __shared__ float As[kRed][kRows + 1];     // codes, reduction index first
    __shared__ float Bs[kRed][kCols];         // rows of X (dW) or W (dX)
    __shared__ double red1[kThreads / 32], red2[kThreads / 32];
    __shared__ float db_s[kRows];
    __shared__ unsigned cnt_s[2];
    __shared__ bool is_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    chain_wait();
    chain_release();
    const long long n = p.B * p.N;

    // ---- 1. step size: shifted moments about the first element, fp32 inside a 16-byte load, fp64 across
    float delta;
    bool nonfinite = false;
    if (p.scale > 0.f) {
        const float pivot = __ldg(p.delta);
        double d1 = 0.0, d2 = 0.0;
        const long long nvec = n / 4;
        const float4 *v4 = reinterpret_cast<const float4 *>(p.delta);
        for (long long i0 = 0; i0 < nvec; i0 += kThreads * 8) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const long long i = i0 + u * kThreads + tid;
                v[u] = i < nvec ? __ldg(v4 + i) : make_float4(pivot, pivot, pivot, pivot);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float c0 = v[u].x - pivot, c1 = v[u].y - pivot, c2 = v[u].z - pivot, c3 = v[u].w - pivot;
                const float s1 = (c0 + c1) + (c2 + c3);
                const float s2 = fmaf(c0, c0, fmaf(c1, c1, fmaf(c2, c2, c3 * c3)));
                d1 += static_cast<double>(s1);
                d2 += static_cast<double>(s2);
            }
        }
        if (tid == 0)
            for (long long i = nvec * 4; i < n; ++i) {
                const double c = static_cast<double>(__ldg(p.delta + i)) - static_cast<double>(pivot);
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
    const float dscale = live ? delta : 0.f;             // what the outputs are scaled by

    // ---- 2. this CTA's tile
    const int t = blockIdx.x;
    const bool is_dw = t < p.n_dw;
    const int tt = is_dw ? t : t - p.n_dw;
    const int rt = tt / p.tiles_k, kt = tt - rt * p.tiles_k;
    const long long row0 = static_cast<long long>(rt) * kRows;      // first output row: j (dW) or b (dX)
    const long long k0 = static_cast<long long>(kt) * kCols;
    const long long nrows = is_dw ? p.N : p.B;                       // output rows in all
    const long long nred = is_dw ? p.B : p.N;                        // reduction length
    const float *Bsrc = is_dw ? p.X : p.W;                           // [nred][K]
    const bool counting = kt == 0 && (is_dw != (p.count_in_dx != 0));
    const bool do_db = is_dw && kt == 0 && p.db != nullptr;
    if (tid < kRows) db_s[tid] = 0.f;
    if (tid < 2) cnt_s[tid] = 0u;

    // element of delta_z for (reduction index r, output row): dW: delta[r][row] - consecutive threads along the
    // rows; dX: delta[row][r] - consecutive threads along r. Either way four consecutive addresses per thread.
    const int a_hi = is_dw ? tid >> 4 : tid >> 3;          // dW: r (0..31); dX: row (0..63)
    const int a_lo = is_dw ? (tid & 15) * 4 : (tid & 7) * 4;   // dW: rows a_lo..+3; dX: r = a_lo..+3
    const int b_r = tid >> 4, b_c = (tid & 15) * 4;        // row b_r of the chunk, columns b_c..+3
    const int ty = tid >> 4, tx = tid & 15;                // outputs: rows 2ty, 2ty+1; columns 4tx..+3
    float acc[2][4] = {};
    float dbacc[4] = {};
    unsigned nnz = 0, sat = 0;

    float a_reg[4];
    float4 b_reg;
    auto load_chunk = [&](long long r0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const long long r = r0 + (is_dw ? a_hi : a_lo + i);
            const long long row = row0 + (is_dw ? a_lo + i : a_hi);
            float q = 0.f;
            if (r < nred && row < nrows) {
                const long long e = is_dw ? r * p.N + row : row * p.N + r;
                const float x = __ldg(p.delta + e);
                if (live) q = code_of(x, e, p.seed, inv, sat);
            }
            a_reg[i] = q;
        }
        {
            const long long r = r0 + b_r;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < nred) {
                const float *src = Bsrc + r * p.K + k0 + b_c;
                if (p.vec4) {
                    if (k0 + b_c < p.K) v = __ldg(reinterpret_cast<const float4 *>(src));
                } else {
                    if (k0 + b_c + 0 < p.K) v.x = __ldg(src + 0);
                    if (k0 + b_c + 1 < p.K) v.y = __ldg(src + 1);
                    if (k0 + b_c + 2 < p.K) v.z = __ldg(src + 2);
                    if (k0 + b_c + 3 < p.K) v.w = __ldg(src + 3);
                }
            }
            b_reg = v;
        }
    };

    load_chunk(0);
    for (long long r0 = 0; r0 < nred; r0 += kRed) {
        __syncthreads();                                 // the previous chunk has been used
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (is_dw) As[a_hi][a_lo + i] = a_reg[i];
            else As[a_lo + i][a_hi] = a_reg[i];
            nnz += a_reg[i] != 0.f;
            dbacc[i] += a_reg[i];
        }
        *reinterpret_cast<float4 *>(&Bs[b_r][b_c]) = b_reg;
        __syncthreads();
        if (r0 + kRed < nred) load_chunk(r0 + kRed);     // in flight during the FMAs
#pragma unroll
        for (int r = 0; r < kRed; ++r) {
            const float a0 = As[r][2 * ty], a1 = As[r][2 * ty + 1];
            const float4 b = *reinterpret_cast<const float4 *>(&Bs[r][4 * tx]);
            acc[0][0] = fmaf(a0, b.x, acc[0][0]); acc[0][1] = fmaf(a0, b.y, acc[0][1]);
            acc[0][2] = fmaf(a0, b.z, acc[0][2]); acc[0][3] = fmaf(a0, b.w, acc[0][3]);
            acc[1][0] = fmaf(a1, b.x, acc[1][0]); acc[1][1] = fmaf(a1, b.y, acc[1][1]);
            acc[1][2] = fmaf(a1, b.z, acc[1][2]); acc[1][3] = fmaf(a1, b.w, acc[1][3]);
        }
    }

    // ---- 3. the tile, scaled by Delta once
    float *out = is_dw ? p.dW : p.dX;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const long long row = row0 + 2 * ty + i;
        const long long col = k0 + 4 * tx;
        if (row >= nrows || col >= p.K) continue;
        float *dst = out + row * p.K + col;
        if (p.vec4) {
            *reinterpret_cast<float4 *>(dst) = make_float4(acc[i][0] * dscale, acc[i][1] * dscale, acc[i][2] * dscale, acc[i][3] * dscale);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (col + c < p.K) dst[c] = acc[i][c] * dscale;
        }
    }

    // ---- 4. counts, bias gradient, and the step's scalars
    if (do_db) {                                         // threads that share a_lo hold the same four rows
#pragma unroll
        for (int i = 0; i < 4; ++i) atomicAdd(&db_s[a_lo + i], dbacc[i]);   // small integers: exact in any order
    }
    nnz = __reduce_add_sync(kFull, nnz);
    sat = __reduce_add_sync(kFull, sat);
    if (lane == 0 && counting) {
        atomicAdd(&cnt_s[0], nnz);
        atomicAdd(&cnt_s[1], sat);
    }
    __syncthreads();
    if (do_db && tid < kRows && row0 + tid < p.N) p.db[row0 + tid] = db_s[tid] * dscale;
    if (tid == 0) {
        if (counting) {
            p.slots[rt] = cnt_s[0];
            if (cnt_s[1]) atomicAdd(&p.st->saturated, static_cast<unsigned long long>(cnt_s[1]));
        }
        __threadfence();
        const unsigned ticket = atomicAdd(&p.st->ticket, 1u);
        is_last = (ticket == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    unsigned long long total = 0;
    for (int i = tid; i < p.n_count; i += kThreads) total += __ldcg(p.slots + i);
    double tsum = warp_sum(static_cast<double>(total));   // counts below 2^53: exact
    __syncthreads();
    if (lane == 0) red1[warp] = tsum;
    __syncthreads();
    if (tid == 0) {
        double all = 0.0;
        for (int w = 0; w < kThreads / 32; ++w) all += red1[w];
        p.st->nnz = static_cast<unsigned long long>(all);
        p.st->delta = delta;
        if (nonfinite) p.st->nonfinite = 1;
        if (p.delta_set) *p.delta_set = delta;
        p.st->ticket = 0u;
    }
}

}  // namespace

// Shapes the one-launch kernel takes: small enough that every CTA can read the whole gradient for its
// statistics (the product of gradient size and CTA count bounds the L2 traffic of that), and few enough
// counting CTAs for the context's scratch.
bool small_linear_fits(const dbp_ctx *ctx, long long B, long long N, long long K, bool want_dw, bool want_dx) {
    const long long n = B * N;
    if (n <= 0 || n > (1ll << 17) || K <= 0 || K > (1ll << 24)) return false;
    const long long tiles_k = (K + kCols - 1) / kCols;
    const long long n_dw = want_dw ? ((N + kRows - 1) / kRows) * tiles_k : 0;
    const long long n_dx = want_dx ? ((B + kRows - 1) / kRows) * tiles_k : 0;
    const long long ctas = n_dw + n_dx;
    if (ctas <= 0 || ctas > 65535 || n * ctas > (1ll << 25)) return false;
    const long long n_count = want_dx ? (B + kRows - 1) / kRows : (N + kRows - 1) / kRows;
    return n_count * static_cast<long long>(sizeof(unsigned)) <= static_cast<long long>(sizeof(double)) * 2 * ctx->partial_blocks;
}

int launch_small_linear(dbp_ctx *ctx, const float *delta, const float *X, const float *W, long long B, long long N,
                        long long K, unsigned long long seed, float scale, const float *delta_in, float *dW, float *dX,
                        float *db, float *delta_set) {
    SmallLinP p{};
    p.delta = delta; p.X = X; p.W = W; p.delta_in = delta_in; p.scale = scale;
    p.B = B; p.N = N; p.K = K; p.seed = seed;
    p.dW = dW; p.dX = dX; p.db = dW ? db : nullptr;
    p.st = ctx->state; p.delta_set = delta_set;
    p.slots = reinterpret_cast<unsigned *>(ctx->partials);
    p.tiles_k = static_cast<int>((K + kCols - 1) / kCols);
    p.n_dw = dW ? static_cast<int>((N + kRows - 1) / kRows) * p.tiles_k : 0;
    p.n_dx = dX ? static_cast<int>((B + kRows - 1) / kRows) * p.tiles_k : 0;
    p.count_in_dx = dX ? 1 : 0;
    p.n_count = static_cast<int>(dX ? (B + kRows - 1) / kRows : (N + kRows - 1) / kRows);
    p.vec4 = (K % 4 == 0) ? 1 : 0;
    return cuda_ok(launch_chained(small_linear_backward_kernel, dim3(static_cast<unsigned>(p.n_dw + p.n_dx)), dim3(kThreads), 0,
                                  ctx->stream, p));
}

}  // namespace dbp
