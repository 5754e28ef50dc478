// nsd_step_size_noalloc: the NSD step size Delta = scale * std(delta) for callers that must
// not allocate device memory. The reduction's scratch (per-block partial sums and the
// last-block ticket) lives in a fixed array that is part of the library image, so the call
// needs no context, no workspace and no cudaMalloc.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "dbp.h"

namespace dbp {
void note_launch();     // the library's launch count (dbp_kernel_launches)
}
using dbp::note_launch;

namespace {

constexpr int kThreads = 256;
constexpr int kMaxBlocks = 1024;
constexpr int kMaxDevices = 64;

struct Scratch {
    double partials[2 * kMaxBlocks];   // (sum, sum of squares) per block
    unsigned int ticket;               // blocks that have published their partials
};

// One copy per GPU that loads the library, held until the process exits (about 16 KB).
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(Scratch)];

template <typename T>
struct Load;
template <>
struct Load<float> {
    static constexpr int EPT = 4;
    __device__ static void vec(const float *p, float (&v)[4]) {
        const float4 q = __ldg(reinterpret_cast<const float4 *>(p));
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    }
    __device__ static float one(const float *p) { return __ldg(p); }
};
template <>
struct Load<__nv_bfloat16> {
    static constexpr int EPT = 8;
    __device__ static void vec(const __nv_bfloat16 *p, float (&v)[8]) {
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

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Same arithmetic as the library's statistics step: moments of the distance from a pivot (the
// first element; the variance does not depend on it, and a constant tensor gives exactly 0), fp32
// inside a 128-bit chunk, fp64 across chunks, block partials combined in a fixed order by the last
// block to finish.
template <typename T>
__global__ void __launch_bounds__(kThreads)
step_size_kernel(const T *__restrict__ x, long long n, float scale, Scratch *__restrict__ sc,
                 float *__restrict__ delta_out) {
    constexpr int EPT = Load<T>::EPT;
    const long long nvec = n / EPT;
    double d1 = 0.0, d2 = 0.0;
    const float pivot = Load<T>::one(x);
    const long long stride = static_cast<long long>(gridDim.x) * kThreads;
    for (long long i = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x; i < nvec; i += stride) {
        float v[EPT];
        Load<T>::vec(x + i * EPT, v);
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
            const double c = static_cast<double>(Load<T>::one(x + i)) - static_cast<double>(pivot);
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
        sc->partials[2 * blockIdx.x] = a;
        sc->partials[2 * blockIdx.x + 1] = b;
        __threadfence();
        is_last = (atomicAdd(&sc->ticket, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last || warp != 0) return;
    __threadfence();
    double a = 0.0, b = 0.0;
    for (int blk = lane; blk < static_cast<int>(gridDim.x); blk += 32) {
        a += __ldcg(sc->partials + 2 * blk);
        b += __ldcg(sc->partials + 2 * blk + 1);
    }
    a = warp_sum(a);
    b = warp_sum(b);
    if (lane == 0) {
        float delta = 0.f;                  // non-finite input: step 0 (every code would be 0)
        if (isfinite(a) && isfinite(b)) {
            const double mean = a / static_cast<double>(n);
            double var = b / static_cast<double>(n) - mean * mean;
            if (var < 0.0) var = 0.0;
            delta = static_cast<float>(static_cast<double>(scale) * sqrt(var));
        }
        *delta_out = delta;
        sc->ticket = 0u;
    }
}

// Device address of the scratch array, looked up once per device. In host code the array's
// name is only a handle for the runtime, not an address a kernel could use.
std::mutex g_mutex;
Scratch *g_scratch_ptr[kMaxDevices] = {nullptr};

int scratch_for_current_device(Scratch **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DBP_ECUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return DBP_ECUDA;
        }
        g_scratch_ptr[dev] = static_cast<Scratch *>(ptr);
    }
    *out = g_scratch_ptr[dev];
    return DBP_OK;
}

}  // namespace

extern "C" int nsd_step_size_noalloc(const void *delta, int dtype, long long numel, float scale,
                                     float *delta_out, void *cuda_stream) {
    if (!delta || !delta_out || numel <= 0 || !(scale > 0.f)) return DBP_EINVAL;
    if (dtype != DBP_F32 && dtype != DBP_BF16) return DBP_EINVAL;
    if ((reinterpret_cast<uintptr_t>(delta) & 15u) != 0) return DBP_EINVAL;
    if (numel > DBP_NOALLOC_MAX_NUMEL) return DBP_ECAPACITY;
    Scratch *sc = nullptr;
    const int rc = scratch_for_current_device(&sc);
    if (rc) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the ticket must start at zero even if an earlier call was cut short
    if (cudaMemsetAsync(&sc->ticket, 0, sizeof(unsigned int), stream) != cudaSuccess) return DBP_ECUDA;
    const int ept = dtype == DBP_F32 ? 4 : 8;
    long long blocks = (numel / ept + kThreads * 4 - 1) / (kThreads * 4);
    if (blocks < 1) blocks = 1;
    if (blocks > kMaxBlocks) blocks = kMaxBlocks;
    if (dtype == DBP_F32)
        { note_launch(); step_size_kernel<float><<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(
            static_cast<const float *>(delta), numel, scale, sc, delta_out); }
    else
        { note_launch(); step_size_kernel<__nv_bfloat16><<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(
            static_cast<const __nv_bfloat16 *>(delta), numel, scale, sc, delta_out); }
    return cudaGetLastError() == cudaSuccess ? DBP_OK : DBP_ECUDA;
}
