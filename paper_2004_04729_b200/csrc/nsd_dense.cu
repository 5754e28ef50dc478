// NSD quantization for the product kernels (Section 3.1, Eq. (nsd)): the same codes as
// quantize_kernel, written only as the dense array the dX / dW kernels read, without the
// bitmap / offsets / packed-values structure. Used when the caller did not ask for the sparse
// structure, so the pass costs one read of delta_z and one write of the codes.
//
// The common case (every |x / Delta + u| <= 127, no NaN) runs without clamping: the code's
// two's-complement byte is the low byte of the round-down sum with 1.5 * 2^23. A vector that
// holds a NaN or a value outside that range is redone element by element with the clipped,
// counted decision.
#include "dbp_internal.cuh"

namespace dbp {

namespace {

constexpr int kThreads = 256;
constexpr unsigned kFull = 0xffffffffu;
constexpr unsigned long long kGamma = 0x9E3779B97F4A7C15ull;

__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
// u = (2k+1) 2^-24, k = top 23 bits of h: the funnel shift builds 1 + k 2^-23 in one step
__device__ __forceinline__ float dither(unsigned h) {
    return __uint_as_float(__funnelshift_r(h, 0x7fu, 9)) - 0.99999994f;
}
// careful decision: clipped to [-127, 127], clipped codes counted, NaN gives 0
__device__ __forceinline__ unsigned careful_byte(float x, float inv, float u, unsigned &sat) {
    const float t = __fmaf_rn(x, inv, u);
    const float tc = fminf(fmaxf(t, -127.f), 127.99999f);
    const bool num = (t == t);
    sat += (num && tc != t) ? 1u : 0u;
    const unsigned q = __float_as_uint(__fadd_rd(tc, 12582912.0f)) & 0xffu;
    return num ? q : 0u;
}
// number of non-zero bytes of a word
__device__ __forceinline__ unsigned nonzero_bytes(unsigned w) {
    return __popc((((w & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w) & 0x80808080u);
}

// Codes of the V elements x[0..V) whose first element has the (even) linear index e0; packed
// four to a word in element order. V is 4 or 8.
template <int V>
__device__ __forceinline__ void codes_of(const float (&x)[V], long long e0, unsigned long long seed,
                                         float inv, unsigned (&pk)[V / 4], unsigned &sat) {
    unsigned long long z = seed + (static_cast<unsigned long long>(e0 >> 1) + 1ull) * kGamma;
    float u[V];
#pragma unroll
    for (int j = 0; j < V; j += 2) {
        const unsigned long long r = mix64(z);
        z += kGamma;
        u[j] = dither(static_cast<unsigned>(r));
        u[j + 1] = dither(static_cast<unsigned>(r >> 32));
    }
    unsigned b[V];
    float amax = 0.f, sum = 0.f;
#pragma unroll
    for (int j = 0; j < V; ++j) {
        const float t = __fmaf_rn(x[j], inv, u[j]);
        amax = fmaxf(amax, fabsf(t));
        sum += t;                                   // NaN iff some t is NaN (or +inf meets -inf)
        b[j] = __float_as_uint(__fadd_rd(t, 12582912.0f));
    }
    if (!(amax <= 127.f) || sum != sum) {           // rare: clip, count, NaN
#pragma unroll
        for (int j = 0; j < V; ++j) b[j] = careful_byte(x[j], inv, u[j], sat);
    }
#pragma unroll
    for (int w = 0; w < V / 4; ++w)
        pk[w] = __byte_perm(__byte_perm(b[4 * w], b[4 * w + 1], 0x0040), __byte_perm(b[4 * w + 2], b[4 * w + 3], 0x0040), 0x5410);
}


// four packed code bytes -> four bf16 (exact): byte ^ 0x80 is code + 128; 0x4B0000xx read as a
// float is 2^23 + xx, so subtracting 2^23 + 128 leaves the code, whose top half is its bf16
__device__ __forceinline__ void bytes4_to_bf16(unsigned w, unsigned &lo, unsigned &hi) {
    const unsigned x = w ^ 0x80808080u;
    const float f0 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7650)) - 8388736.0f;
    const float f1 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7651)) - 8388736.0f;
    const float f2 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7652)) - 8388736.0f;
    const float f3 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7653)) - 8388736.0f;
    lo = __byte_perm(__float_as_uint(f0), __float_as_uint(f1), 0x7632);
    hi = __byte_perm(__float_as_uint(f2), __float_as_uint(f3), 0x7632);
}

// Where the codes go. dense8: one byte per element, same order as delta_z (may be null).
// planes16: bf16 codes as [plane][pitch] with plane = e / hw (may be null); the pitch is a
// multiple of 8 so that every plane starts on a 16-byte boundary.
struct CodeSinks {
    int8_t *dense8;
    unsigned short *planes16;
    long long hw, pitch;
    int count;                    // add nnz / clipped counts to the context's counters
};

// plane = e / hw and the offset inside it; a 32-bit division when the index allows it (a 64-bit
// one costs several times as many instructions)
__device__ __forceinline__ void split_index(long long e, long long hw, long long &plane, long long &pp) {
    if (((e | hw) >> 32) == 0) {
        const unsigned q = static_cast<unsigned>(e) / static_cast<unsigned>(hw);
        plane = q;
        pp = static_cast<unsigned>(e) - q * static_cast<unsigned>(hw);
    } else {
        plane = e / hw;
        pp = e - plane * hw;
    }
}

template <int V>
__device__ __forceinline__ void store_codes(const CodeSinks &o, long long e0, const unsigned (&pk)[V / 4]) {
    if (o.dense8 != nullptr) {
        if (V == 4) *reinterpret_cast<unsigned *>(o.dense8 + e0) = pk[0];
        else *reinterpret_cast<uint2 *>(o.dense8 + e0) = make_uint2(pk[0], pk[V / 4 - 1]);
    }
    if (o.planes16 != nullptr) {
        unsigned h[V / 2];
#pragma unroll
        for (int w = 0; w < V / 4; ++w) bytes4_to_bf16(pk[w], h[2 * w], h[2 * w + 1]);
        if (o.pitch == o.hw) {                      // planes are back to back: same order as delta_z
            if (V == 4) *reinterpret_cast<uint2 *>(o.planes16 + e0) = make_uint2(h[0], h[1]);
            else *reinterpret_cast<uint4 *>(o.planes16 + e0) = make_uint4(h[0], h[1], h[V / 2 - 2], h[V / 2 - 1]);
        } else if ((o.hw & 3) == 0) {
            // e0 and the plane size are multiples of 4: each group of four codes lies in one plane
            // and starts on an 8-byte boundary there
            long long plane, pp;
            split_index(e0, o.hw, plane, pp);
#pragma unroll
            for (int g = 0; g < V / 4; ++g) {
                *reinterpret_cast<uint2 *>(o.planes16 + plane * o.pitch + pp) = make_uint2(h[2 * g], h[2 * g + 1]);
                pp += 4;
                if (pp == o.hw) { pp = 0; ++plane; }
            }
        } else {
            long long plane, pp;
            split_index(e0, o.hw, plane, pp);
#pragma unroll
            for (int j = 0; j < V; ++j) {
                o.planes16[plane * o.pitch + pp] = static_cast<unsigned short>(h[j >> 1] >> (16 * (j & 1)));
                if (++pp == o.hw) { pp = 0; ++plane; }
            }
        }
    }
}
__device__ __forceinline__ void store_code(const CodeSinks &o, long long e, unsigned byte) {
    if (o.dense8 != nullptr) o.dense8[e] = static_cast<int8_t>(byte);
    if (o.planes16 != nullptr) {
        const long long plane = e / o.hw;
        const float f = static_cast<float>(static_cast<int>(static_cast<signed char>(byte)));
        o.planes16[plane * o.pitch + (e - plane * o.hw)] = static_cast<unsigned short>(__float_as_uint(f) >> 16);
    }
}

template <typename T>
struct Vec;
template <>
struct Vec<float> {
    static constexpr int V = 4;
    __device__ static void load(const float *p, float (&v)[4]) {
        const float4 q = __ldg(reinterpret_cast<const float4 *>(p));
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    }
    __device__ static float one(const float *p) { return __ldg(p); }
};
template <>
struct Vec<__nv_bfloat16> {
    static constexpr int V = 8;
    __device__ static void load(const __nv_bfloat16 *p, float (&v)[8]) {
        const uint4 q = __ldg(reinterpret_cast<const uint4 *>(p));
        const unsigned w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    __device__ static float one(const __nv_bfloat16 *p) {
        return __uint_as_float(static_cast<unsigned>(__ldg(reinterpret_cast<const unsigned short *>(p))) << 16);
    }
};

template <typename T>
__global__ void __launch_bounds__(kThreads)
quantize_dense_kernel(const T *__restrict__ x, long long n, unsigned long long seed,
                      const float *__restrict__ delta_p, const CodeSinks out,
                      DeviceState *__restrict__ st) {
    constexpr int V = Vec<T>::V;
    const long long nvec = n / V;
    const long long stride = static_cast<long long>(gridDim.x) * kThreads;
    long long i = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x;
    chain_wait();
    chain_release();
    const float delta = *delta_p;
    const bool live = (delta > 0.f) && (delta < __int_as_float(0x7f800000));
    if (!live) {                                    // sigma = 0 or non-finite input: every code is 0
        for (; i < nvec; i += stride) {
            const unsigned zero[V / 4] = {};
            store_codes<V>(out, i * V, zero);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0)
            for (long long e = nvec * V; e < n; ++e) store_code(out, e, 0u);
        return;
    }
    const float inv = __fdiv_rn(1.0f, delta);
    unsigned nnz = 0, sat = 0;
    // two vectors in flight per thread
    for (; i + stride < nvec; i += 2 * stride) {
        float a[V], b[V];
        Vec<T>::load(x + i * V, a);
        Vec<T>::load(x + (i + stride) * V, b);
        unsigned pa[V / 4], pb[V / 4];
        codes_of<V>(a, i * V, seed, inv, pa, sat);
        codes_of<V>(b, (i + stride) * V, seed, inv, pb, sat);
        store_codes<V>(out, i * V, pa);
        store_codes<V>(out, (i + stride) * V, pb);
#pragma unroll
        for (int w = 0; w < V / 4; ++w) nnz += nonzero_bytes(pa[w]) + nonzero_bytes(pb[w]);
    }
    if (i < nvec) {
        float a[V];
        Vec<T>::load(x + i * V, a);
        unsigned pa[V / 4];
        codes_of<V>(a, i * V, seed, inv, pa, sat);
        store_codes<V>(out, i * V, pa);
#pragma unroll
        for (int w = 0; w < V / 4; ++w) nnz += nonzero_bytes(pa[w]);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {      // the n % V last elements, one by one
        for (long long e = nvec * V; e < n; ++e) {
            const unsigned long long r = mix64(seed + (static_cast<unsigned long long>(e >> 1) + 1ull) * kGamma);
            const float u = dither((e & 1) ? static_cast<unsigned>(r >> 32) : static_cast<unsigned>(r));
            const unsigned q = careful_byte(Vec<T>::one(x + e), inv, u, sat);
            store_code(out, e, q);
            nnz += q != 0u;
        }
    }
    nnz = __reduce_add_sync(kFull, nnz);
    sat = __reduce_add_sync(kFull, sat);
    __shared__ unsigned s_nnz, s_sat;
    if (threadIdx.x == 0) { s_nnz = 0; s_sat = 0; }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) {
        if (nnz) atomicAdd(&s_nnz, nnz);
        if (sat) atomicAdd(&s_sat, sat);
    }
    __syncthreads();
    if (threadIdx.x == 0 && out.count) {
        if (s_nnz) atomicAdd(&st->nnz, static_cast<unsigned long long>(s_nnz));
        if (s_sat) atomicAdd(&st->saturated, static_cast<unsigned long long>(s_sat));
    }
}


// ---------------------------------------------------------------- position-major bf16 codes
// The same codes, written as bf16 in the order [image][position][channel] (the 3x3 tensor-core
// kernels read this form: a row of 64 channels of one position is 128 contiguous bytes, so a
// rectangular patch of positions with its halo is one tiled copy and a tap of the filter is a row
// offset inside it). delta_z itself is [image][channel][position], so a block transposes tiles of
// 64 channels x 64 positions through shared memory: rows of the input are read along the
// positions, rows of the output are written along the channels. The dither of an element is
// still keyed on its index in delta_z's own order.
constexpr int kTC = 64, kTP = 64;                 // channels x positions per tile
constexpr int kTileBytes = kTP * kTC * 2;

// shared-memory byte offset of (position p, channel c) inside a tile: 128-byte rows, the
// 16-byte pieces of a row permuted by the row's group of eight
__device__ __forceinline__ unsigned tile_off(int p, int c) {
    return static_cast<unsigned>(p) * 128u + (((static_cast<unsigned>(c) >> 3) ^ ((static_cast<unsigned>(p) >> 3) & 7u)) << 4) +
           ((static_cast<unsigned>(c) & 7u) << 1);
}

// one element by itself (planes whose size is odd: the pair that shares a draw may straddle two
// vectors); same decision as codes_of
__device__ __forceinline__ unsigned code_single(float x, long long e, unsigned long long seed, float inv, unsigned &sat) {
    const unsigned long long r = mix64(seed + (static_cast<unsigned long long>(e >> 1) + 1ull) * kGamma);
    const float u = dither((e & 1) ? static_cast<unsigned>(r >> 32) : static_cast<unsigned>(r));
    const float t = __fmaf_rn(x, inv, u);
    if (fabsf(t) <= 127.f) return __float_as_uint(__fadd_rd(t, 12582912.0f)) & 0xffu;
    return careful_byte(x, inv, u, sat);
}
__device__ __forceinline__ unsigned short byte_to_bf16(unsigned b) {
    const float f = static_cast<float>(static_cast<int>(static_cast<signed char>(b)));
    return static_cast<unsigned short>(__float_as_uint(f) >> 16);
}

template <typename T, int V>
struct TileLoad;
template <>
struct TileLoad<__nv_bfloat16, 8> {
    __device__ static void ld(const __nv_bfloat16 *p, float (&v)[8]) { Vec<__nv_bfloat16>::load(p, v); }
};
template <>
struct TileLoad<__nv_bfloat16, 4> {
    __device__ static void ld(const __nv_bfloat16 *p, float (&v)[4]) {
        const uint2 q = __ldg(reinterpret_cast<const uint2 *>(p));
        v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xffff0000u);
        v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xffff0000u);
    }
};
template <>
struct TileLoad<float, 4> {
    __device__ static void ld(const float *p, float (&v)[4]) { Vec<float>::load(p, v); }
};

// V: elements per load (plane size % V == 0), or 1 for element-wise loads (any plane size)
template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
quantize_nhwc_kernel(const T *__restrict__ x, int B, int C, int HW, unsigned long long seed,
                     const float *__restrict__ delta_p, unsigned short *__restrict__ out,
                     int8_t *__restrict__ dense8, DeviceState *__restrict__ st, int count) {
    __shared__ __align__(16) unsigned char tile[2][kTileBytes];
    constexpr int VV = (V > 1) ? V : 4;               // vector length of the vector path
    chain_wait();
    chain_release();
    const float delta = *delta_p;
    const bool live = (delta > 0.f) && (delta < __int_as_float(0x7f800000));
    const float inv = live ? __fdiv_rn(1.0f, delta) : 0.f;
    const int ct = (C + kTC - 1) / kTC, pt = (HW + kTP - 1) / kTP;
    const long long ntiles = static_cast<long long>(B) * ct * pt;
    unsigned nnz = 0, sat = 0;
    int buf = 0;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x, buf ^= 1) {
        const int b = static_cast<int>(t / (ct * pt));
        const int rem = static_cast<int>(t - static_cast<long long>(b) * ct * pt);
        const int c0 = (rem / pt) * kTC, p0 = (rem % pt) * kTP;
        unsigned char *tl = tile[buf];
        if (V > 1) {
            constexpr int VPR = kTP / VV;            // vectors per channel row of the tile
#pragma unroll
            for (int i = 0; i < (kTC * VPR) / kThreads; ++i) {
                const int v = threadIdx.x + kThreads * i;
                const int c = v / VPR, pv = (v % VPR) * VV;
                unsigned pk[VV / 4] = {};
                const bool in = c0 + c < C && p0 + pv < HW;       // HW % V == 0: whole vectors
                const long long e0 = (static_cast<long long>(b) * C + c0 + c) * HW + p0 + pv;
                if (in && live) {
                    float a[VV];
                    TileLoad<T, VV>::ld(x + e0, a);
                    codes_of<VV>(a, e0, seed, inv, pk, sat);
                }
                if (in && dense8 != nullptr) {
                    if (VV == 4) *reinterpret_cast<unsigned *>(dense8 + e0) = pk[0];
                    else *reinterpret_cast<uint2 *>(dense8 + e0) = make_uint2(pk[0], pk[VV / 4 - 1]);
                }
#pragma unroll
                for (int w = 0; w < VV / 4; ++w) {
                    nnz += nonzero_bytes(pk[w]);
                    unsigned lo, hi;
                    bytes4_to_bf16(pk[w], lo, hi);
                    const int pp = pv + 4 * w;
                    *reinterpret_cast<unsigned short *>(tl + tile_off(pp, c)) = static_cast<unsigned short>(lo);
                    *reinterpret_cast<unsigned short *>(tl + tile_off(pp + 1, c)) = static_cast<unsigned short>(lo >> 16);
                    *reinterpret_cast<unsigned short *>(tl + tile_off(pp + 2, c)) = static_cast<unsigned short>(hi);
                    *reinterpret_cast<unsigned short *>(tl + tile_off(pp + 3, c)) = static_cast<unsigned short>(hi >> 16);
                }
            }
        } else {
#pragma unroll 4
            for (int i = 0; i < (kTC * kTP) / kThreads; ++i) {
                const int id = threadIdx.x + kThreads * i;
                const int c = id / kTP, pp = id % kTP;
                unsigned q = 0;
                const bool in = c0 + c < C && p0 + pp < HW;
                const long long e = (static_cast<long long>(b) * C + c0 + c) * HW + p0 + pp;
                if (in && live) q = code_single(Vec<T>::one(x + e), e, seed, inv, sat);
                if (in && dense8 != nullptr) dense8[e] = static_cast<int8_t>(q);
                nnz += q != 0u;
                *reinterpret_cast<unsigned short *>(tl + tile_off(pp, c)) = byte_to_bf16(q);
            }
        }
        __syncthreads();
        // rows of 64 channels (128 bytes) of one position each; eight lanes per row
#pragma unroll
        for (int i = 0; i < (kTP * 8) / kThreads; ++i) {
            const int v = threadIdx.x + kThreads * i;
            const int pp = v >> 3, ch = v & 7;
            if (p0 + pp < HW && c0 + ch * 8 < C)
                *reinterpret_cast<uint4 *>(out + (static_cast<long long>(b) * HW + p0 + pp) * C + c0 + ch * 8) =
                    *reinterpret_cast<const uint4 *>(tl + tile_off(pp, ch * 8));
        }
        // the other buffer is written next; this one again only after the next barrier
    }
    nnz = __reduce_add_sync(kFull, nnz);
    sat = __reduce_add_sync(kFull, sat);
    if ((threadIdx.x & 31) == 0 && count) {
        if (nnz) atomicAdd(&st->nnz, static_cast<unsigned long long>(nnz));
        if (sat) atomicAdd(&st->saturated, static_cast<unsigned long long>(sat));
    }
}

template <typename T, int V>
cudaError_t run_nhwc(dbp_ctx *ctx, const void *delta, int B, int C, int HW, unsigned long long seed, const float *delta_p,
                     void *out, int8_t *dense8, bool count) {
    const long long ntiles = static_cast<long long>(B) * ((C + kTC - 1) / kTC) * ((HW + kTP - 1) / kTP);
    long long blocks = ntiles < static_cast<long long>(ctx->sm_count) * 6 ? ntiles : static_cast<long long>(ctx->sm_count) * 6;
    if (blocks < 1) blocks = 1;
    return launch_chained(quantize_nhwc_kernel<T, V>, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, ctx->stream,
                          static_cast<const T *>(delta), B, C, HW, seed, delta_p, static_cast<unsigned short *>(out), dense8,
                          ctx->state, count ? 1 : 0);
}

}  // namespace

int launch_quantize_dense(dbp_ctx *ctx, const void *delta, int dtype, long long numel,
                          unsigned long long seed, const float *delta_p, int8_t *dense,
                          void *planes_bf16, long long hw, long long pitch, bool count) {
    const int v = dtype == DBP_F32 ? 4 : 8;
    long long blocks = (numel / v + 2 * kThreads - 1) / (2 * kThreads);
    if (blocks < 1) blocks = 1;
    const long long cap = static_cast<long long>(ctx->sm_count) * 8;
    if (blocks > cap) blocks = cap;
    CodeSinks out{dense, static_cast<unsigned short *>(planes_bf16), hw > 0 ? hw : 1, pitch > 0 ? pitch : 1, count ? 1 : 0};
    cudaError_t e;
    if (dtype == DBP_F32)
        e = launch_chained(quantize_dense_kernel<float>, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, ctx->stream,
                           static_cast<const float *>(delta), numel, seed, delta_p, out, ctx->state);
    else
        e = launch_chained(quantize_dense_kernel<__nv_bfloat16>, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0,
                           ctx->stream, static_cast<const __nv_bfloat16 *>(delta), numel, seed, delta_p, out, ctx->state);
    return cuda_ok(e);
}

// delta_z [B][C][HW] -> bf16 codes [B][HW][C] (C % 8 == 0) and, when dense8 is not null, int8 codes
// in delta_z's order
int launch_quantize_nhwc(dbp_ctx *ctx, const void *delta, int dtype, long long B, long long C, long long HW,
                         unsigned long long seed, const float *delta_p, void *codes_nhwc, int8_t *dense8, bool count) {
    if (C % 8 != 0 || B * C * HW >= (1ll << 40) || HW >= (1ll << 30)) return DBP_EUNSUPPORTED;
    const int b = static_cast<int>(B), c = static_cast<int>(C), hw = static_cast<int>(HW);
    cudaError_t e;
    if (dtype == DBP_F32)
        e = hw % 4 == 0 ? run_nhwc<float, 4>(ctx, delta, b, c, hw, seed, delta_p, codes_nhwc, dense8, count)
                        : run_nhwc<float, 1>(ctx, delta, b, c, hw, seed, delta_p, codes_nhwc, dense8, count);
    else
        e = hw % 8 == 0   ? run_nhwc<__nv_bfloat16, 8>(ctx, delta, b, c, hw, seed, delta_p, codes_nhwc, dense8, count)
            : hw % 4 == 0 ? run_nhwc<__nv_bfloat16, 4>(ctx, delta, b, c, hw, seed, delta_p, codes_nhwc, dense8, count)
                          : run_nhwc<__nv_bfloat16, 1>(ctx, delta, b, c, hw, seed, delta_p, codes_nhwc, dense8, count);
    return cuda_ok(e);
}

}  // namespace dbp
