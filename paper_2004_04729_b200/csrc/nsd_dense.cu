// NSD quantization for the product kernels (Section 3.1, Eq. (nsd)): the same codes as
// quantize_kernel, written only as the dense array the dX / dW kernels read, without the
// bitmap / offsets / packed-values structure. Used when the caller did not ask for the sparse
// structure, so the pass costs one read of delta_z and one write of the codes.
//
// The common case (every |x / Delta + u| <= 127, no NaN) runs without clamping or conversions:
// the code is the round-down sum with 1.5 * 2^23, less that constant (a float holding a small
// integer, whose upper half is its bf16). A vector that holds a NaN or a value outside that range
// is redone element by element with the clipped, counted decision.
#include "dbp_internal.cuh"

namespace dbp {

namespace {

constexpr int kThreads = 256;
#ifndef DBP_Q_BLOCKS_PER_SM
#define DBP_Q_BLOCKS_PER_SM 4
#endif
constexpr int kBlocksPerSM = DBP_Q_BLOCKS_PER_SM;   // resident blocks the dense quantizer is compiled for
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
constexpr float kMagic = 12582912.0f;             // 1.5 * 2^23: a float in [2^23, 2^24) has unit spacing
// careful decision: clipped to [-127, 127], clipped codes counted, NaN gives 0. Returns the bits of
// kMagic + code (the low byte is the code's two's-complement byte).
__device__ __forceinline__ unsigned careful_bits(float x, float inv, float u, unsigned &sat) {
    const float t = __fmaf_rn(x, inv, u);
    const float tc = fminf(fmaxf(t, -127.f), 127.99999f);
    const bool num = (t == t);
    sat += (num && tc != t) ? 1u : 0u;
    return num ? __float_as_uint(__fadd_rd(tc, kMagic)) : __float_as_uint(kMagic);
}
__device__ __forceinline__ unsigned careful_byte(float x, float inv, float u, unsigned &sat) {
    return careful_bits(x, inv, u, sat) & 0xffu;
}
// Codes of the V elements x[0..V) whose first element has the (even) linear index e0, as floats
// (exact small integers). V is 4 or 8. The common case (every |t| <= 127, no NaN) is recognised by
// the sum of the squares of t = x / Delta + u and needs no clamp: floor(t) is the round-down sum
// with kMagic, less kMagic. The number of non-zero codes is added to nz (a float: exact below 2^24).
template <int V>
__device__ __forceinline__ void codes_of(const float (&x)[V], long long e0, unsigned long long seed,
                                         float inv, float (&f)[V], float &nz, unsigned &sat) {
    unsigned long long z = seed + (static_cast<unsigned long long>(e0 >> 1) + 1ull) * kGamma;
    float u[V];
#pragma unroll
    for (int j = 0; j < V; j += 2) {
        const unsigned long long r = mix64(z);
        z += kGamma;
        u[j] = dither(static_cast<unsigned>(r));
        u[j + 1] = dither(static_cast<unsigned>(r >> 32));
    }
    float s2 = 0.f;
#pragma unroll
    for (int j = 0; j < V; ++j) {
        const float t = __fmaf_rn(x[j], inv, u[j]);
        s2 = __fmaf_rn(t, t, s2);                   // NaN or inf if some t is; > 127^2 if some |t| > 127
        f[j] = __fadd_rd(t, kMagic) - kMagic;
    }
    if (!(s2 <= 16128.f)) {                         // rare: clip, count, NaN
#pragma unroll
        for (int j = 0; j < V; ++j) f[j] = __uint_as_float(careful_bits(x[j], inv, u[j], sat)) - kMagic;
    }
#pragma unroll
    for (int j = 0; j < V; ++j) nz += __saturatef(f[j] * f[j]);
}
// the codes' bytes, four to a word in element order
template <int V>
__device__ __forceinline__ void pack_bytes(const float (&f)[V], unsigned (&pk)[V / 4]) {
    unsigned b[V];
#pragma unroll
    for (int j = 0; j < V; ++j) b[j] = __float_as_uint(f[j] + kMagic);     // low byte: the code
#pragma unroll
    for (int w = 0; w < V / 4; ++w)
        pk[w] = __byte_perm(__byte_perm(b[4 * w], b[4 * w + 1], 0x0040), __byte_perm(b[4 * w + 2], b[4 * w + 3], 0x0040), 0x5410);
}
// the codes as bf16, two to a word: an integer of at most 8 bits is exact in bf16, which is the
// float's upper half
template <int V>
__device__ __forceinline__ void pack_bf16(const float (&f)[V], unsigned (&h)[V / 2]) {
#pragma unroll
    for (int j = 0; j < V / 2; ++j) h[j] = __byte_perm(__float_as_uint(f[2 * j]), __float_as_uint(f[2 * j + 1]), 0x7632);
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
__device__ __forceinline__ void store_codes(const CodeSinks &o, long long e0, const float (&f)[V]) {
    if (o.dense8 != nullptr) {
        unsigned pk[V / 4];
        pack_bytes<V>(f, pk);
        if (V == 4) *reinterpret_cast<unsigned *>(o.dense8 + e0) = pk[0];
        else *reinterpret_cast<uint2 *>(o.dense8 + e0) = make_uint2(pk[0], pk[V / 4 - 1]);
    }
    if (o.planes16 != nullptr) {
        unsigned h[V / 2];
        pack_bf16<V>(f, h);
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
            // odd plane sizes: code by code, or two at a time where the pair starts on an even offset
            // of its plane and does not run over the plane's end
            long long plane, pp;
            split_index(e0, o.hw, plane, pp);
            unsigned short *dst = o.planes16 + plane * o.pitch + pp;
            long long left = o.hw - pp;                           // codes until the plane ends
            const long long gap = o.pitch - o.hw;
#pragma unroll
            for (int j = 0; j < V; j += 2) {
                if (left >= 2 && (reinterpret_cast<uintptr_t>(dst) & 3) == 0) {
                    *reinterpret_cast<unsigned *>(dst) = h[j >> 1];
                    dst += 2;
                    left -= 2;
                    if (left == 0) { left = o.hw; dst += gap; }
                } else {
                    *dst++ = static_cast<unsigned short>(h[j >> 1]);
                    if (--left == 0) { left = o.hw; dst += gap; }
                    *dst++ = static_cast<unsigned short>(h[j >> 1] >> 16);
                    if (--left == 0) { left = o.hw; dst += gap; }
                }
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
__global__ void __launch_bounds__(kThreads, kBlocksPerSM)
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
            const float zero[V] = {};
            store_codes<V>(out, i * V, zero);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0)
            for (long long e = nvec * V; e < n; ++e) store_code(out, e, 0u);
        return;
    }
    const float inv = __fdiv_rn(1.0f, delta);
    unsigned nnz = 0, sat = 0;
    float nz = 0.f;
    // two vectors in flight per thread
    for (; i + stride < nvec; i += 2 * stride) {
        float a[V], b[V];
        Vec<T>::load(x + i * V, a);
        Vec<T>::load(x + (i + stride) * V, b);
        float fa[V], fb[V];
        codes_of<V>(a, i * V, seed, inv, fa, nz, sat);
        codes_of<V>(b, (i + stride) * V, seed, inv, fb, nz, sat);
        store_codes<V>(out, i * V, fa);
        store_codes<V>(out, (i + stride) * V, fb);
    }
    if (i < nvec) {
        float a[V];
        Vec<T>::load(x + i * V, a);
        float fa[V];
        codes_of<V>(a, i * V, seed, inv, fa, nz, sat);
        store_codes<V>(out, i * V, fa);
    }
    nnz = static_cast<unsigned>(nz);                // a thread's share is far below 2^24 elements
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
// vectors); same decision as codes_of. Returns the code as a float.
__device__ __forceinline__ float code_single(float x, long long e, unsigned long long seed, float inv, unsigned &sat) {
    const unsigned long long r = mix64(seed + (static_cast<unsigned long long>(e >> 1) + 1ull) * kGamma);
    const float u = dither((e & 1) ? static_cast<unsigned>(r >> 32) : static_cast<unsigned>(r));
    const float t = __fmaf_rn(x, inv, u);
    if (fabsf(t) <= 127.f) return __fadd_rd(t, kMagic) - kMagic;
    return __uint_as_float(careful_bits(x, inv, u, sat)) - kMagic;
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

template <int V>
__device__ __forceinline__ void store_bytes(int8_t *dense8, long long e0, const float (&f)[V]) {
    unsigned pk[V / 4];
    pack_bytes<V>(f, pk);
    if (V == 4) *reinterpret_cast<unsigned *>(dense8 + e0) = pk[0];
    else *reinterpret_cast<uint2 *>(dense8 + e0) = make_uint2(pk[0], pk[V / 4 - 1]);
}

// V: elements per load (plane size % V == 0), or 1 for element-wise loads (any plane size).
// Three ways to fill a tile. Planes smaller than a tile's 64 positions: the tile's 64 channels of one
// image are one contiguous run of delta_z, read as whole vectors whatever the plane size. Otherwise,
// plane size % V == 0: a thread takes the same V positions of two neighbouring channels and writes
// the two codes of a position as one word. Otherwise element by element.
// mask (fp32 tensors only, may be null): x is delta_a and the gradient is delta_a where mask != 0, else 0
__device__ __forceinline__ void apply_mask(const unsigned char *mask, long long e, float (&v)[4]) {
    if (mask != nullptr) {
        const uchar4 m = __ldg(reinterpret_cast<const uchar4 *>(mask + e));
        v[0] = m.x ? v[0] : 0.f; v[1] = m.y ? v[1] : 0.f; v[2] = m.z ? v[2] : 0.f; v[3] = m.w ? v[3] : 0.f;
    }
}
__device__ __forceinline__ void apply_mask(const unsigned char *, long long, float (&)[8]) {}

template <typename T, int V, bool STACK, bool MASKED>
__global__ void __launch_bounds__(kThreads)
quantize_nhwc_kernel(const T *__restrict__ x, int B, int C, int HW, unsigned long long seed,
                     const float *__restrict__ delta_p, unsigned short *__restrict__ out,
                     int8_t *__restrict__ dense8, DeviceState *__restrict__ st, int count,
                     unsigned short *__restrict__ out_stack, int plane_w, int stack_g,
                     const unsigned char *__restrict__ mask_in) {
    const unsigned char *mask = MASKED ? mask_in : nullptr;
    __shared__ __align__(16) unsigned char tile[2][kTileBytes];
    constexpr int VV = (V > 1) ? V : 4;               // vector length of the paired path
    constexpr int VF = Vec<T>::V;                     // vector length of the contiguous path
    chain_wait();
    chain_release();
    const float delta = *delta_p;
    const bool live = (delta > 0.f) && (delta < __int_as_float(0x7f800000));
    const float inv = live ? __fdiv_rn(1.0f, delta) : 0.f;
    const int ct = (C + kTC - 1) / kTC, pt = (HW + kTP - 1) / kTP;
    const long long ntiles = static_cast<long long>(B) * ct * pt;
    const bool flat = HW < kTP;
    unsigned nnz = 0, sat = 0;
    float nz = 0.f;
    int buf = 0;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x, buf ^= 1) {
        const int b = static_cast<int>(t / (ct * pt));
        const int rem = static_cast<int>(t - static_cast<long long>(b) * ct * pt);
        const int c0 = (rem / pt) * kTC, p0 = (rem % pt) * kTP;
        unsigned char *tl = tile[buf];
        if (flat) {
            // (b, c0 .. c0+63, every position): C % 8 == 0, so the run starts on a 16-byte boundary and on
            // an even element, and holds a whole number of vectors
            const int nch = C - c0 < kTC ? C - c0 : kTC;
            const long long base = (static_cast<long long>(b) * C + c0) * HW;
            const int nvec = nch * HW / VF;
            for (int v = threadIdx.x; v < nvec; v += kThreads) {
                float f[VF] = {};
                if (live) {
                    float a[VF];
                    Vec<T>::load(x + base + v * VF, a);
                    apply_mask(mask, base + v * VF, a);
                    codes_of<VF>(a, base + v * VF, seed, inv, f, nz, sat);
                }
                if (dense8 != nullptr) store_bytes<VF>(dense8, base + v * VF, f);
                int c = (v * VF) / HW, pp = v * VF - c * HW;
#pragma unroll
                for (int j = 0; j < VF; ++j) {
                    *reinterpret_cast<unsigned short *>(tl + tile_off(pp, c)) = static_cast<unsigned short>(__float_as_uint(f[j]) >> 16);
                    if (++pp == HW) { pp = 0; ++c; }
                }
            }
        } else if (V > 1) {
            constexpr int VPR = kTP / VV;            // vectors per channel row of the tile
#pragma unroll
            for (int i = 0; i < (kTC / 2 * VPR) / kThreads; ++i) {
                const int v = threadIdx.x + kThreads * i;
                const int c = 2 * (v / VPR), pv = (v % VPR) * VV;
                float f0[VV] = {}, f1[VV] = {};
                const bool in = c0 + c < C && p0 + pv < HW;       // C is even, HW % V == 0: whole vectors, both channels
                const long long e0 = (static_cast<long long>(b) * C + c0 + c) * HW + p0 + pv, e1 = e0 + HW;
                if (in && live) {
                    float a0[VV], a1[VV];
                    TileLoad<T, VV>::ld(x + e0, a0);
                    TileLoad<T, VV>::ld(x + e1, a1);
                    apply_mask(mask, e0, a0);
                    apply_mask(mask, e1, a1);
                    codes_of<VV>(a0, e0, seed, inv, f0, nz, sat);
                    codes_of<VV>(a1, e1, seed, inv, f1, nz, sat);
                }
                if (in && dense8 != nullptr) {
                    store_bytes<VV>(dense8, e0, f0);
                    store_bytes<VV>(dense8, e1, f1);
                }
#pragma unroll
                for (int j = 0; j < VV; ++j)
                    *reinterpret_cast<unsigned *>(tl + tile_off(pv + j, c)) =
                        __byte_perm(__float_as_uint(f0[j]), __float_as_uint(f1[j]), 0x7632);
            }
        } else {
#pragma unroll 4
            for (int i = 0; i < (kTC * kTP) / kThreads; ++i) {
                const int id = threadIdx.x + kThreads * i;
                const int c = id / kTP, pp = id % kTP;
                float f = 0.f;
                const bool in = c0 + c < C && p0 + pp < HW;
                const long long e = (static_cast<long long>(b) * C + c0 + c) * HW + p0 + pp;
                if (in && live) f = code_single((mask == nullptr || __ldg(mask + e)) ? Vec<T>::one(x + e) : 0.f, e, seed, inv, sat);
                if (in && dense8 != nullptr) dense8[e] = static_cast<int8_t>(static_cast<int>(f));
                nnz += f != 0.f;
                *reinterpret_cast<unsigned short *>(tl + tile_off(pp, c)) = static_cast<unsigned short>(__float_as_uint(f) >> 16);
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
            // Second copy for the weight-gradient kernel of tiny planes: the images one below the other as tall
            // images, a row of zeros after every image (what a tap that leaves an image must read).
            if (STACK && pp < HW + plane_w && c0 + ch * 8 < C) {
                const uint4 val = pp < HW ? *reinterpret_cast<const uint4 *>(tl + tile_off(pp, ch * 8)) : make_uint4(0u, 0u, 0u, 0u);
                const long long row = static_cast<long long>(b) * (HW + plane_w) + pp;   // any number of images per tall image
                *reinterpret_cast<uint4 *>(out_stack + row * C + c0 + ch * 8) = val;
            }
        }
        // the other buffer is written next; this one again only after the next barrier
    }
    nnz += static_cast<unsigned>(nz);
    nnz = __reduce_add_sync(kFull, nnz);
    sat = __reduce_add_sync(kFull, sat);
    if ((threadIdx.x & 31) == 0 && count) {
        if (nnz) atomicAdd(&st->nnz, static_cast<unsigned long long>(nnz));
        if (sat) atomicAdd(&st->saturated, static_cast<unsigned long long>(sat));
    }
}

template <typename T, int V>
cudaError_t run_nhwc(dbp_ctx *ctx, const void *delta, int B, int C, int HW, unsigned long long seed, const float *delta_p,
                     void *out, int8_t *dense8, bool count, void *out_stack, int plane_w, int stack_g, const uint8_t *mask) {
    const long long ntiles = static_cast<long long>(B) * ((C + kTC - 1) / kTC) * ((HW + kTP - 1) / kTP);
    long long blocks = ntiles < static_cast<long long>(ctx->sm_count) * 6 ? ntiles : static_cast<long long>(ctx->sm_count) * 6;
    if (blocks < 1) blocks = 1;
    const unsigned char *m = static_cast<const unsigned char *>(mask);
    auto go = [&](auto kern, unsigned short *stack) {
        return launch_chained(kern, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, ctx->stream,
                              static_cast<const T *>(delta), B, C, HW, seed, delta_p, static_cast<unsigned short *>(out), dense8,
                              ctx->state, count ? 1 : 0, stack, stack ? plane_w : 0, stack ? stack_g : 0, m);
    };
    unsigned short *st = static_cast<unsigned short *>(out_stack);
    if (mask != nullptr)      // fp32 only (checked by the caller)
        return st ? go(quantize_nhwc_kernel<T, V, true, true>, st) : go(quantize_nhwc_kernel<T, V, false, true>, st);
    return st ? go(quantize_nhwc_kernel<T, V, true, false>, st) : go(quantize_nhwc_kernel<T, V, false, false>, st);
}

// ---------------------------------------------------------------- bf16 planes of odd sizes
// Planes whose size is no multiple of 4 (7 x 7, 9 x 9, ...) written at a pitch that is a multiple of 8: the codes
// of eight consecutive elements then belong to unaligned places of one or two planes. A block takes a run of
// whole planes (a multiple of eight of them, so that the run starts on a 16-byte boundary and on an even
// element), quantizes it with whole-vector loads as everywhere, places the codes in shared memory at their pitch,
// and the run leaves as one contiguous copy (the padding of a plane is never read by anybody).
constexpr int kOddMaxSmem = 12 * 1024;            // bytes of the staged run (planes x pitch bf16)

template <typename T>
__global__ void __launch_bounds__(kThreads)
quantize_planes_odd_kernel(const T *__restrict__ x, long long nplanes, int hw, int pitch, int planes_per_run,
                           unsigned long long seed, const float *__restrict__ delta_p, unsigned short *__restrict__ out,
                           int8_t *__restrict__ dense8, DeviceState *__restrict__ st, int count) {
    constexpr int V = Vec<T>::V;
    __shared__ __align__(16) unsigned short run_s[kOddMaxSmem / 2];
    chain_wait();
    chain_release();
    const float delta = *delta_p;
    const bool live = (delta > 0.f) && (delta < __int_as_float(0x7f800000));
    const float inv = live ? __fdiv_rn(1.0f, delta) : 0.f;
    const long long nruns = (nplanes + planes_per_run - 1) / planes_per_run;
    unsigned sat = 0;
    float nz = 0.f;
    for (long long r = blockIdx.x; r < nruns; r += gridDim.x) {
        const long long pl0 = r * planes_per_run;
        const int np = static_cast<int>(nplanes - pl0 < planes_per_run ? nplanes - pl0 : planes_per_run);   // a multiple of 8
        const long long e_base = pl0 * hw;
        const int nvec = np * hw / V;
        for (int v = threadIdx.x; v < nvec; v += kThreads) {
            float f[V] = {};
            const long long e0 = e_base + static_cast<long long>(v) * V;
            if (live) {
                float a[V];
                Vec<T>::load(x + e0, a);
                codes_of<V>(a, e0, seed, inv, f, nz, sat);
            }
            if (dense8 != nullptr) store_bytes<V>(dense8, e0, f);
            int pl = (v * V) / hw, pp = v * V - pl * hw;
#pragma unroll
            for (int j = 0; j < V; ++j) {
                run_s[pl * pitch + pp] = static_cast<unsigned short>(__float_as_uint(f[j]) >> 16);
                if (++pp == hw) { pp = 0; ++pl; }
            }
        }
        __syncthreads();
        const int n16 = np * pitch / 8;
        uint4 *dst = reinterpret_cast<uint4 *>(out + pl0 * pitch);
        for (int i = threadIdx.x; i < n16; i += kThreads) dst[i] = reinterpret_cast<const uint4 *>(run_s)[i];
        __syncthreads();
    }
    unsigned nnz = static_cast<unsigned>(nz);
    nnz = __reduce_add_sync(kFull, nnz);
    sat = __reduce_add_sync(kFull, sat);
    if ((threadIdx.x & 31) == 0 && count) {
        if (nnz) atomicAdd(&st->nnz, static_cast<unsigned long long>(nnz));
        if (sat) atomicAdd(&st->saturated, static_cast<unsigned long long>(sat));
    }
}

}  // namespace

int launch_quantize_dense(dbp_ctx *ctx, const void *delta, int dtype, long long numel,
                          unsigned long long seed, const float *delta_p, int8_t *dense,
                          void *planes_bf16, long long hw, long long pitch, bool count) {
    const int v = dtype == DBP_F32 ? 4 : 8;
    // odd plane sizes at a padded pitch: whole runs of planes through shared memory
    if (planes_bf16 != nullptr && hw > 0 && pitch != hw && (hw & 3) != 0 && numel % hw == 0 && (numel / hw) % 8 == 0 &&
        8 * pitch * 2 <= kOddMaxSmem && hw < (1 << 20)) {
        const long long nplanes = numel / hw;
        int per_run = static_cast<int>(kOddMaxSmem / 2 / pitch / 8 * 8);          // planes per run: a multiple of 8
        const long long want = (4096 + 8 * hw - 1) / (8 * hw) * 8;               // about 4096 elements a run
        if (per_run > want) per_run = static_cast<int>(want);
        long long nruns = (nplanes + per_run - 1) / per_run;
        long long blocks = nruns < static_cast<long long>(ctx->sm_count) * 8 ? nruns : static_cast<long long>(ctx->sm_count) * 8;
        cudaError_t e;
        if (dtype == DBP_F32)
            e = launch_chained(quantize_planes_odd_kernel<float>, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, ctx->stream,
                               static_cast<const float *>(delta), nplanes, static_cast<int>(hw), static_cast<int>(pitch), per_run, seed,
                               delta_p, static_cast<unsigned short *>(planes_bf16), dense, ctx->state, count ? 1 : 0);
        else
            e = launch_chained(quantize_planes_odd_kernel<__nv_bfloat16>, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, ctx->stream,
                               static_cast<const __nv_bfloat16 *>(delta), nplanes, static_cast<int>(hw), static_cast<int>(pitch), per_run,
                               seed, delta_p, static_cast<unsigned short *>(planes_bf16), dense, ctx->state, count ? 1 : 0);
        return cuda_ok(e);
    }
    long long blocks = (numel / v + 2 * kThreads - 1) / (2 * kThreads);
    if (blocks < 1) blocks = 1;
    const long long cap = static_cast<long long>(ctx->sm_count) * kBlocksPerSM;
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
                         unsigned long long seed, const float *delta_p, void *codes_nhwc, int8_t *dense8, bool count,
                         void *codes_stack, int plane_w, int stack_g, const uint8_t *mask) {
    if (C % 8 != 0 || B * C * HW >= (1ll << 40) || HW >= (1ll << 30)) return DBP_EUNSUPPORTED;
    if (mask != nullptr && dtype != DBP_F32) return DBP_EUNSUPPORTED;
    // the stacked copy is written by the path for planes smaller than a tile; the rows of image b start at
    // b (HW + W) however many images make up a tall image: the stacking only adds the zero rows
    if (codes_stack != nullptr && (HW >= kTP || plane_w <= 0 || stack_g <= 0 || HW + plane_w > kTP)) return DBP_EINVAL;
    const int b = static_cast<int>(B), c = static_cast<int>(C), hw = static_cast<int>(HW);
    cudaError_t e;
    if (dtype == DBP_F32)
        e = hw % 4 == 0 ? run_nhwc<float, 4>(ctx, delta, b, c, hw, seed, delta_p, codes_nhwc, dense8, count, codes_stack, plane_w, stack_g, mask)
                        : run_nhwc<float, 1>(ctx, delta, b, c, hw, seed, delta_p, codes_nhwc, dense8, count, codes_stack, plane_w, stack_g, mask);
    else
        e = hw % 8 == 0   ? run_nhwc<__nv_bfloat16, 8>(ctx, delta, b, c, hw, seed, delta_p, codes_nhwc, dense8, count, codes_stack, plane_w, stack_g, mask)
            : hw % 4 == 0 ? run_nhwc<__nv_bfloat16, 4>(ctx, delta, b, c, hw, seed, delta_p, codes_nhwc, dense8, count, codes_stack, plane_w, stack_g, mask)
                          : run_nhwc<__nv_bfloat16, 1>(ctx, delta, b, c, hw, seed, delta_p, codes_nhwc, dense8, count, codes_stack, plane_w, stack_g, mask);
    return cuda_ok(e);
}

}  // namespace dbp
