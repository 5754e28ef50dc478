// NSD quantization kernels: one-pass statistics (Algorithm 1, std line), dither + quantize +
// compaction (Section 3.1, Eq. (nsd)), and expansion of the sparse structure to dense codes.
//
// Both streaming kernels are bound by HBM bandwidth: 128-bit loads of delta_z, 128-bit stores
// of the packed codes, bitmap words and offsets assembled with warp shuffles.
#include "dbp_internal.cuh"

namespace dbp {

namespace {

constexpr int kThreads = 256;
constexpr unsigned kFull = 0xffffffffu;

template <typename T>
struct Elem;

template <>
struct Elem<float> {
    static constexpr int EPT = 4;  // elements per 128-bit load
    __device__ static void load(const float *p, float (&v)[4]) {
        float4 q = __ldg(reinterpret_cast<const float4 *>(p));
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    }
    __device__ static float one(const float *p) { return __ldg(p); }
    // read-once data: do not keep the line in L1
    __device__ static void load_stream(const float *p, float (&v)[4]) {
        unsigned a, b, c, d;
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "l"(p));
        v[0] = __uint_as_float(a); v[1] = __uint_as_float(b); v[2] = __uint_as_float(c); v[3] = __uint_as_float(d);
    }
};

template <>
struct Elem<__nv_bfloat16> {
    static constexpr int EPT = 8;
    __device__ static void load(const __nv_bfloat16 *p, float (&v)[8]) {
        uint4 q = __ldg(reinterpret_cast<const uint4 *>(p));
        const unsigned w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);           // bf16 -> fp32 is exact
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    __device__ static float one(const __nv_bfloat16 *p) {
        return __uint_as_float(static_cast<unsigned>(__ldg(reinterpret_cast<const unsigned short *>(p))) << 16);
    }
    __device__ static void load_stream(const __nv_bfloat16 *p, float (&v)[8]) {
        unsigned w[4];
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "l"(p));
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

// ---------------------------------------------------------------- statistics (sigma, Delta)
// Sum and sum of squares of every element's distance from a pivot (the tensor's first element):
// fp32 inside one 128-bit chunk, fp64 across chunks, per-block partials combined in a fixed order
// by the last block to finish, so the step size does not depend on scheduling. The variance is
// shift-invariant, and with the pivot inside the data's range the moments stay of the order of
// sigma: a constant tensor gives exactly 0 and a mean far from 0 costs no accuracy (raw moments
// would cancel). sigma is the population standard deviation about the mean; Delta = scale * sigma
// rounded once to fp32.
// MASKED (fp32 only): the tensor is delta_a and the statistics are those of delta_a where mask != 0, else 0 (the
// ReLU derivative folded into the read; one byte per element).
template <bool MASKED>
__device__ __forceinline__ void mask4(const unsigned char *mask, long long e, float (&v)[4]) {
    if (MASKED) {
        const uchar4 m = __ldg(reinterpret_cast<const uchar4 *>(mask + e));
        v[0] = m.x ? v[0] : 0.f; v[1] = m.y ? v[1] : 0.f; v[2] = m.z ? v[2] : 0.f; v[3] = m.w ? v[3] : 0.f;
    }
}
template <bool MASKED>
__device__ __forceinline__ void mask4(const unsigned char *, long long, float (&)[8]) {}   // bf16 tensors take no mask

template <typename T, bool MASKED = false>
__global__ void __launch_bounds__(kThreads)
statistics_kernel(const T *__restrict__ x, long long n, double *__restrict__ partials,
                  DeviceState *__restrict__ st, float scale, float *__restrict__ delta_out,
                  unsigned long long *__restrict__ nnz_out, uint4 *__restrict__ zero_ptr, long long zero_n16,
                  const void *__restrict__ w_src, unsigned short *__restrict__ w_dst, int w_f32, long long w_cout, int w_cin,
                  const unsigned char *__restrict__ mask, int w_phase_cin) {
    constexpr int EPT = Elem<T>::EPT;
    const long long nvec = n / EPT;
    chain_wait();
    chain_release();
    // side job for the layer's weight-gradient kernel, which adds its partial sums into dW: clear it
    for (long long i = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x; i < zero_n16;
         i += static_cast<long long>(gridDim.x) * kThreads)
        zero_ptr[i] = make_uint4(0u, 0u, 0u, 0u);
    // side job for the layer's 3x3 input-gradient kernel: weights [co][ci][9] -> [co][tap][ci] bf16 (for fp32
    // weights two pieces: taps 0-8 the values rounded to bf16, taps 9-17 the remainders rounded to bf16).
    // w_phase_cin > 0: the layer is a stride-2 layer run on the four phase images of its input; w_src holds that
    // layer's own weights [co][w_phase_cin][9] and channel ph * w_phase_cin + c of the re-laid weights is phase
    // ph = 2 py + px of channel c, whose tap (ty, tx) is the strided layer's tap ky = 0 for (py, ty) = (1, 0),
    // 1 for (0, 1), 2 for (1, 1), kx likewise, and zero for every other pair.
    if (w_src != nullptr) {
        const int per_co = 9 * w_cin, taps = w_f32 ? 18 : 9;
        for (long long co = blockIdx.x; co < w_cout; co += gridDim.x) {
            unsigned short *dst = w_dst + co * taps * w_cin;
            // a thread takes one channel and all nine taps: nine independent loads, then stores that run along ci
            for (int ci = threadIdx.x; ci < w_cin; ci += kThreads) {
                int ph = 0;
                long long base = (co * w_cin + ci) * 9;
                if (w_phase_cin > 0) {
                    ph = ci / w_phase_cin;
                    base = (co * w_phase_cin + (ci - ph * w_phase_cin)) * 9;
                }
                int k[9];                                                  // source tap, or -1 for a zero weight
#pragma unroll
                for (int t = 0; t < 9; ++t) {
                    const int ty = t / 3, tx = t % 3;
                    k[t] = t;
                    if (w_phase_cin > 0) {
                        const int ky = (ph & 2) ? (ty == 0 ? 0 : (ty == 1 ? 2 : -1)) : (ty == 1 ? 1 : -1);
                        const int kx = (ph & 1) ? (tx == 0 ? 0 : (tx == 1 ? 2 : -1)) : (tx == 1 ? 1 : -1);
                        k[t] = (ky >= 0 && kx >= 0) ? ky * 3 + kx : -1;
                    }
                }
                if (w_f32) {
                    float w[9];
#pragma unroll
                    for (int t = 0; t < 9; ++t) w[t] = k[t] >= 0 ? __ldg(static_cast<const float *>(w_src) + base + k[t]) : 0.f;
#pragma unroll
                    for (int t = 0; t < 9; ++t) {
                        const __nv_bfloat16 hi = __float2bfloat16_rn(w[t]);
                        const __nv_bfloat16 lo = __float2bfloat16_rn(w[t] - __bfloat162float(hi));
                        dst[t * w_cin + ci] = *reinterpret_cast<const unsigned short *>(&hi);
                        dst[per_co + t * w_cin + ci] = *reinterpret_cast<const unsigned short *>(&lo);
                    }
                } else {
                    unsigned short w[9];
#pragma unroll
                    for (int t = 0; t < 9; ++t)
                        w[t] = k[t] >= 0 ? __ldg(static_cast<const unsigned short *>(w_src) + base + k[t]) : static_cast<unsigned short>(0);
#pragma unroll
                    for (int t = 0; t < 9; ++t) dst[t * w_cin + ci] = w[t];
                }
            }
        }
    }
    double d1 = 0.0, d2 = 0.0;
    const float pivot = (!MASKED || __ldg(mask)) ? Elem<T>::one(x) : 0.f;
    const long long stride = static_cast<long long>(gridDim.x) * kThreads;
    // whole tiles of kUnroll x kThreads 128-bit vectors, a block at a time: kUnroll loads in flight
    // per thread, consecutive threads on consecutive vectors
    constexpr int kUnroll = 8;
    const long long tile = static_cast<long long>(kUnroll) * kThreads, ntile = nvec / tile;
    for (long long t = blockIdx.x; t < ntile; t += gridDim.x) {
        const T *p = x + (t * tile + threadIdx.x) * EPT;
        float v[kUnroll][EPT];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) Elem<T>::load_stream(p + static_cast<long long>(u) * kThreads * EPT, v[u]);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) mask4<MASKED>(mask, (t * tile + threadIdx.x + static_cast<long long>(u) * kThreads) * EPT, v[u]);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            float s1 = 0.f, s2 = 0.f;
#pragma unroll
            for (int j = 0; j < EPT; ++j) {
                const float c = v[u][j] - pivot;
                s1 += c;
                s2 = fmaf(c, c, s2);
            }
            d1 += static_cast<double>(s1);
            d2 += static_cast<double>(s2);
        }
    }
    // the vectors after the last whole tile
    long long i = ntile * tile + static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x;
    for (; i < nvec; i += stride) {
        float v[EPT];
        Elem<T>::load(x + i * EPT, v);
        mask4<MASKED>(mask, i * EPT, v);
        float s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const float c = v[j] - pivot;
            s1 += c;
            s2 = fmaf(c, c, s2);
        }
        d1 += static_cast<double>(s1);
        d2 += static_cast<double>(s2);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (long long i = nvec * EPT; i < n; ++i) {
            const float xi = (!MASKED || __ldg(mask + i)) ? Elem<T>::one(x + i) : 0.f;
            const double c = static_cast<double>(xi) - static_cast<double>(pivot);
            d1 += c;
            d2 += c * c;
        }
    }
    __shared__ double sh1[kThreads / 32], sh2[kThreads / 32];
    __shared__ bool is_last;
    d1 = warp_sum(d1);
    d2 = warp_sum(d2);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { sh1[warp] = d1; sh2[warp] = d2; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0;
        for (int w = 0; w < kThreads / 32; ++w) { a += sh1[w]; b += sh2[w]; }
        partials[2 * blockIdx.x] = a;
        partials[2 * blockIdx.x + 1] = b;
        __threadfence();
        const unsigned t = atomicAdd(&st->ticket, 1u);
        is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    // the last block adds the partials: every thread a strided share (loads independent of one
    // another), then warps and the block in a fixed order
    __threadfence();
    double a = 0.0, b = 0.0;
#pragma unroll 4
    for (int blk = threadIdx.x; blk < static_cast<int>(gridDim.x); blk += kThreads) {
        a += __ldcg(partials + 2 * blk);
        b += __ldcg(partials + 2 * blk + 1);
    }
    a = warp_sum(a);
    b = warp_sum(b);
    __syncthreads();                 // sh1/sh2 were read by thread 0 above
    if (lane == 0) { sh1[warp] = a; sh2[warp] = b; }
    __syncthreads();
    if (warp != 0) return;
    a = 0.0; b = 0.0;
    for (int w = 0; w < kThreads / 32; ++w) { a += sh1[w]; b += sh2[w]; }
    if (lane == 0) {
        float delta = 0.f;
        if (!isfinite(a) || !isfinite(b)) {
            st->nonfinite = 1;                      // every code becomes 0
        } else {
            const double mean = a / static_cast<double>(n);
            double var = b / static_cast<double>(n) - mean * mean;
            if (var < 0.0) var = 0.0;
            delta = static_cast<float>(static_cast<double>(scale) * sqrt(var));
        }
        st->delta = delta;
        st->nnz = 0ull;
        st->ticket = 0u;
        if (delta_out) *delta_out = delta;
        if (nnz_out) *nnz_out = 0ull;
    }
}

__global__ void set_step_kernel(const float *__restrict__ delta_in, DeviceState *st,
                                float *delta_out, unsigned long long *nnz_out) {
    const float d = *delta_in;
    st->delta = d;
    st->nnz = 0ull;
    if (delta_out) *delta_out = d;
    if (nnz_out) *nnz_out = 0ull;
}

// ---------------------------------------------------------------- dither + quantize + compact
// SplitMix64 output number c of the sequence started at `seed` (counter-based: no state).
__device__ __forceinline__ unsigned long long splitmix64_mix(unsigned long long z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// u = (2k+1) 2^-24 from the top 23 bits k of h: (1 + k 2^-23) - (1 - 2^-24), exact.
__device__ __forceinline__ float dither_from_bits(unsigned h) {
    return __uint_as_float(0x3f800000u | (h >> 9)) - 0.99999994f;
}

// q = floor(x / Delta + u) with one rounding, clipped to [-127, 127]; NaN gives 0.
// floor and the conversion to int are one round-down addition of 1.5 * 2^23 (exact for the
// clamped range) and an integer subtraction.
__device__ __forceinline__ int quantize_one(float x, float inv, float u, unsigned &sat) {
    const float t = __fmaf_rn(x, inv, u);
    const float tc = fminf(fmaxf(t, -127.f), 127.99999f);
    const bool num = (t == t);
    sat += (num && tc != t) ? 1u : 0u;
    const int q = __float_as_int(__fadd_rd(tc, 12582912.0f)) - 0x4B400000;
    return num ? q : 0;
}

// One warp owns one 1024-element segment at a time: ITER 128-bit loads per lane, codes
// packed through a per-warp shared staging line, one coalesced store each of the 32 bitmap
// words, the 32 offsets and the packed codes.
template <typename T>
__global__ void __launch_bounds__(kThreads)
quantize_kernel(const T *__restrict__ x, long long n, unsigned long long seed,
                const float *__restrict__ delta_p, uint32_t *__restrict__ bitmap,
                uint16_t *__restrict__ offsets, int8_t *__restrict__ values,
                int8_t *__restrict__ dense, DeviceState *__restrict__ st,
                unsigned long long *__restrict__ nnz_out) {
    constexpr int EPT = Elem<T>::EPT;
    constexpr int ITER = kSegment / (32 * EPT);  // 8 (fp32) or 4 (bf16)
    constexpr int LPW = 32 / EPT;                // lanes that share one bitmap word
    constexpr int NW = EPT / 4;                  // packed code words per lane and iteration
    __shared__ __align__(16) int8_t stage[kThreads / 32][kSegment];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long nseg = (n + kSegment - 1) / kSegment;
    const long long nwarps = static_cast<long long>(gridDim.x) * (kThreads / 32);
    const long long first = static_cast<long long>(blockIdx.x) * (kThreads / 32) + warp;
    const float delta = *delta_p;
    const bool live = (delta > 0.f) && (delta < __int_as_float(0x7f800000));
    if (!live) {   // sigma = 0 or non-finite input: every code is 0
        for (long long seg = first; seg < nseg; seg += nwarps) {
            bitmap[seg * kWordsPerSegment + lane] = 0u;
            offsets[seg * kWordsPerSegment + lane] = 0;
            if (dense != nullptr) {
                const long long e0 = seg * kSegment + lane * 32;
                if (e0 + 32 <= n) {
                    reinterpret_cast<uint4 *>(dense + e0)[0] = make_uint4(0u, 0u, 0u, 0u);
                    reinterpret_cast<uint4 *>(dense + e0)[1] = make_uint4(0u, 0u, 0u, 0u);
                } else {
                    for (int j = 0; j < 32; ++j)
                        if (e0 + j < n) dense[e0 + j] = 0;
                }
            }
        }
        return;
    }
    const float inv = __fdiv_rn(1.0f, delta);
    const int sub = lane % LPW;                  // my position inside the word
    unsigned long long nnz_local = 0ull;
    unsigned sat = 0;

    for (long long seg = first; seg < nseg; seg += nwarps) {
        const bool full = (seg + 1) * kSegment <= n;
        unsigned running = 0, my_word = 0, my_off = 0;
#pragma unroll
        for (int it = 0; it < ITER; ++it) {
            const long long e0 = seg * kSegment + it * (32 * EPT) + lane * EPT;
            float v[EPT];
            if (full || e0 + EPT <= n) {
                Elem<T>::load(x + e0, v);
            } else {
#pragma unroll
                for (int j = 0; j < EPT; ++j) v[j] = (e0 + j < n) ? Elem<T>::one(x + e0 + j) : 0.f;
            }
            unsigned pk[NW];
#pragma unroll
            for (int w = 0; w < NW; ++w) pk[w] = 0u;
            unsigned bits = 0;
            unsigned long long z = seed + (static_cast<unsigned long long>(e0 >> 1) + 1ull) * 0x9E3779B97F4A7C15ull;
#pragma unroll
            for (int j = 0; j < EPT; j += 2) {
                const unsigned long long r = splitmix64_mix(z);
                z += 0x9E3779B97F4A7C15ull;
                const int q0 = quantize_one(v[j], inv, dither_from_bits(static_cast<unsigned>(r)), sat);
                const int q1 = quantize_one(v[j + 1], inv, dither_from_bits(static_cast<unsigned>(r >> 32)), sat);
                pk[j >> 2] |= (static_cast<unsigned>(q0) & 0xffu) << (8 * (j & 3));
                pk[j >> 2] |= (static_cast<unsigned>(q1) & 0xffu) << (8 * ((j + 1) & 3));
                bits |= (q0 != 0 ? 1u : 0u) << j;
                bits |= (q1 != 0 ? 1u : 0u) << (j + 1);
            }
            if (!full) {   // elements past the end carry no code (their x was read as 0 already)
#pragma unroll
                for (int j = 0; j < EPT; ++j)
                    if (e0 + j >= n) { bits &= ~(1u << j); pk[j >> 2] &= ~(0xffu << (8 * (j & 3))); }
            }
            // bitmap word shared by LPW consecutive lanes
            unsigned word = bits << (EPT * sub);
#pragma unroll
            for (int o = 1; o < LPW; o <<= 1) word |= __shfl_xor_sync(kFull, word, o);
            // exclusive rank of my first code inside the segment: warp scan of the lane counts
            const unsigned pc = __popc(bits);
            unsigned incl = pc;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned up = __shfl_up_sync(kFull, incl, o);
                if (lane >= o) incl += up;
            }
            const unsigned total = __shfl_sync(kFull, incl, 31);
            unsigned rank = running + incl - pc;
            const unsigned word_off = rank;      // for a word's first lane: codes before the word
            // non-zero codes to the staging line, in element order
            unsigned b = bits;
            while (b) {
                const int j = __ffs(b) - 1;
                b &= b - 1;
                const unsigned wsel = (NW == 1 || j < 4) ? pk[0] : pk[NW - 1];
                stage[warp][rank++] = static_cast<int8_t>((wsel >> (8 * (j & 3))) & 0xffu);
            }
            if (dense != nullptr) {
                if (full || e0 + EPT <= n) {
                    if (EPT == 4) *reinterpret_cast<unsigned *>(dense + e0) = pk[0];
                    else *reinterpret_cast<uint2 *>(dense + e0) = make_uint2(pk[0], pk[NW - 1]);
                } else {
#pragma unroll
                    for (int j = 0; j < EPT; ++j)
                        if (e0 + j < n) dense[e0 + j] = static_cast<int8_t>((pk[j >> 2] >> (8 * (j & 3))) & 0xffu);
                }
            }
            // lane (it*EPT + w) keeps word w of this iteration and its offset
            const unsigned wv = __shfl_sync(kFull, word, (lane % EPT) * LPW);
            const unsigned ov = __shfl_sync(kFull, word_off, (lane % EPT) * LPW);
            if (lane / EPT == it) { my_word = wv; my_off = ov; }
            running += total;
        }
        __syncwarp();
        bitmap[seg * kWordsPerSegment + lane] = my_word;
        offsets[seg * kWordsPerSegment + lane] = static_cast<uint16_t>(my_off);
        for (unsigned i = lane * 16; i < running; i += 512)
            *reinterpret_cast<uint4 *>(values + seg * kSegment + i) =
                *reinterpret_cast<const uint4 *>(&stage[warp][i]);
        __syncwarp();
        nnz_local += running;
    }
    sat = __reduce_add_sync(kFull, sat);
    if (lane == 0) {
        if (nnz_local) {
            atomicAdd(&st->nnz, nnz_local);
            if (nnz_out) atomicAdd(nnz_out, nnz_local);
        }
        if (sat) atomicAdd(&st->saturated, static_cast<unsigned long long>(sat));
    }
}

// One warp per segment, one lane per bitmap word: 32 codes written as two 128-bit stores.
__global__ void __launch_bounds__(kThreads)
decode_kernel(const uint32_t *__restrict__ bitmap, const uint16_t *__restrict__ offsets,
              const int8_t *__restrict__ values, long long n, int8_t *__restrict__ dense) {
    const int lane = threadIdx.x & 31;
    const long long nseg = (n + kSegment - 1) / kSegment;
    const long long nwarps = static_cast<long long>(gridDim.x) * (kThreads / 32);
    for (long long seg = static_cast<long long>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5); seg < nseg; seg += nwarps) {
        const long long w = seg * kWordsPerSegment + lane;
        unsigned word = bitmap[w];
        const int8_t *src = values + seg * kSegment + offsets[w];
        unsigned pk[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        while (word) {
            const int b = __ffs(word) - 1;
            word &= word - 1;
            pk[b >> 2] |= (static_cast<unsigned>(*src++) & 0xffu) << (8 * (b & 3));
        }
        const long long e0 = w * 32;
        if (e0 + 32 <= n) {
            uint4 *dst = reinterpret_cast<uint4 *>(dense + e0);
            dst[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            dst[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
        } else {
            for (int j = 0; j < 32; ++j)
                if (e0 + j < n) dense[e0 + j] = static_cast<int8_t>((pk[j >> 2] >> (8 * (j & 3))) & 0xff);
        }
    }
}

}  // namespace

constexpr int kStatBlocksPerSM = 2;

int launch_statistics(dbp_ctx *ctx, const void *delta, int dtype, long long numel, float scale,
                      const float *delta_in, float *delta_out, unsigned long long *nnz_out, const SideJobs &jobs,
                      const uint8_t *mask) {
    if (mask != nullptr && dtype != DBP_F32) return DBP_EUNSUPPORTED;
    uint4 *zp = static_cast<uint4 *>(jobs.zero);
    const long long zn = jobs.zero ? static_cast<long long>(jobs.zero_bytes / 16) : 0;
    unsigned short *wd = static_cast<unsigned short *>(jobs.w_dst);
    const int wci = static_cast<int>(jobs.Cin);
    if (!(scale > 0.f)) {      // the step size is given: no statistics kernel, so no side jobs either (the caller sees to the weights)
        if (jobs.zero && cudaMemsetAsync(jobs.zero, 0, jobs.zero_bytes, ctx->stream) != cudaSuccess) return fail_cuda("clearing dW");
        note_launch();
        set_step_kernel<<<1, 1, 0, ctx->stream>>>(delta_in, ctx->state, delta_out, nnz_out);
        return cuda_ok(cudaGetLastError());
    }
    const int ept = dtype == DBP_F32 ? 4 : 8;
    long long blocks = numel / ept / (kThreads * 8);          // one block per tile of eight vectors per thread
    if (blocks < 1) blocks = 1;
    // the side jobs want blocks of their own when the tensor is small (a block beyond the tensor's tiles adds zeros)
    if (jobs.w_src != nullptr && blocks < jobs.Cout) blocks = jobs.Cout;
    if (jobs.zero != nullptr && blocks < static_cast<long long>(jobs.zero_bytes / (16 * kThreads * 4))) blocks = static_cast<long long>(jobs.zero_bytes / (16 * kThreads * 4));
    if (blocks > ctx->partial_blocks) blocks = ctx->partial_blocks;
    // two resident blocks per SM, each walking several tiles, finish sooner than one block per tile: fewer partial
    // sums for the last block to add and fewer tickets (measured on the ResNet-50 layer set: 0.70 against 0.73 ms
    // per step for 48 layers; one block per SM: 0.76). The weight re-laying side job wants one block per output channel.
    if (jobs.w_src == nullptr && blocks > static_cast<long long>(ctx->sm_count) * kStatBlocksPerSM)
        blocks = static_cast<long long>(ctx->sm_count) * kStatBlocksPerSM;
    cudaError_t e;
    const unsigned char *nomask = nullptr;
    if (dtype == DBP_F32 && mask != nullptr)
        e = launch_chained(statistics_kernel<float, true>, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, ctx->stream,
                           static_cast<const float *>(delta), numel, ctx->partials, ctx->state, scale, delta_out, nnz_out, zp, zn, jobs.w_src, wd, jobs.w_f32, jobs.Cout, wci,
                           static_cast<const unsigned char *>(mask), jobs.phase_cin);
    else if (dtype == DBP_F32)
        e = launch_chained(statistics_kernel<float, false>, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, ctx->stream,
                           static_cast<const float *>(delta), numel, ctx->partials, ctx->state, scale, delta_out, nnz_out, zp, zn, jobs.w_src, wd, jobs.w_f32, jobs.Cout, wci, nomask, jobs.phase_cin);
    else
        e = launch_chained(statistics_kernel<__nv_bfloat16, false>, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, ctx->stream,
                           static_cast<const __nv_bfloat16 *>(delta), numel, ctx->partials, ctx->state, scale, delta_out, nnz_out, zp, zn, jobs.w_src, wd, jobs.w_f32, jobs.Cout, wci, nomask, jobs.phase_cin);
    return cuda_ok(e);
}

int launch_quantize(dbp_ctx *ctx, const void *delta, int dtype, long long numel,
                    unsigned long long seed, const float *delta_p, uint32_t *bitmap,
                    uint16_t *offsets, int8_t *values, int8_t *dense,
                    unsigned long long *nnz_out) {
    const long long nseg = (numel + kSegment - 1) / kSegment;
    long long blocks = (nseg + kThreads / 32 - 1) / (kThreads / 32);
    const long long cap = static_cast<long long>(ctx->sm_count) * 8;
    if (blocks > cap) blocks = cap;
    if (dtype == DBP_F32)
        { note_launch(); quantize_kernel<float><<<static_cast<unsigned>(blocks), kThreads, 0, ctx->stream>>>(
            static_cast<const float *>(delta), numel, seed, delta_p, bitmap, offsets, values, dense,
            ctx->state, nnz_out); }
    else
        { note_launch(); quantize_kernel<__nv_bfloat16><<<static_cast<unsigned>(blocks), kThreads, 0, ctx->stream>>>(
            static_cast<const __nv_bfloat16 *>(delta), numel, seed, delta_p, bitmap, offsets, values,
            dense, ctx->state, nnz_out); }
    return cuda_ok(cudaGetLastError());
}

int launch_decode(dbp_ctx *ctx, const uint32_t *bitmap, const uint16_t *offsets,
                  const int8_t *values, long long numel, int8_t *dense) {
    const long long nseg = (numel + kSegment - 1) / kSegment;
    long long blocks = (nseg + kThreads / 32 - 1) / (kThreads / 32);
    const long long cap = static_cast<long long>(ctx->sm_count) * 8;
    if (blocks > cap) blocks = cap;
    note_launch();
    decode_kernel<<<static_cast<unsigned>(blocks), kThreads, 0, ctx->stream>>>(bitmap, offsets, values,
                                                                            numel, dense);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dbp
