// Stride-2 convolution layers (the down-sampling 3x3 and 1x1 layers of residual networks) as stride-1 layers
// on the four phase images of the input ("analogous for convolutional layers", Section 3; the quantized gradient
// and both products of Eqs. (qda), (qdw) are unchanged, only the indexing of the activations differs).
//
//   z[b,co,y,x] = sum_{ci,ky,kx} W[co,ci,ky,kx] X[b,ci,2y+ky-p,2x+kx-p],   p = (k-1)/2, H and W even.
//
// With X'[b,(py,px,ci),y,x] = X[b,ci,2y+py,2x+px] (py, px in {0,1}; half the height and width, four times the
// channels) the input row 2y+ky-1 of a 3x3 layer is row y-1 of the odd phase (ky = 0), row y of the even phase
// (ky = 1) or row y of the odd phase (ky = 2); columns likewise. So the layer is the stride-1 3x3 layer
//   z = W' * X',  W'[co,(py,px,ci),ty,tx] = W[co,ci,ky(py,ty),kx(px,tx)],
//   ky(1,0) = 0, ky(0,1) = 1, ky(1,1) = 2, every other (phase, tap) pair a zero weight,
// whose zero padding is the zero padding of the strided layer. Its weight gradient holds dW at the nine non-zero
// places and its input gradient is dX in the same phase layout. A 1x1 layer reads the (0,0) phase alone:
// X' = X[:, :, ::2, ::2], W' = W, and dX is zero at every position with an odd coordinate.
//
// The kernels here only move data between the two layouts; the quantizer and the products are the stride-1 ones.
#include "dbp_internal.cuh"

namespace dbp {

namespace {

inline int blocks_of(long long n, int threads, int cap) {
    long long b = (n + threads - 1) / threads;
    if (b < 1) b = 1;
    return static_cast<int>(b < cap ? b : cap);
}

// NP pairs of neighbouring columns as one vector
template <typename T, int NP> struct Cols;
template <> struct Cols<float, 1> { using vec = float2; using half = float; };
template <> struct Cols<float, 2> { using vec = float4; using half = float2; };
template <> struct Cols<__nv_bfloat16, 1> { using vec = unsigned; using half = unsigned short; };
template <> struct Cols<__nv_bfloat16, 2> { using vec = uint2; using half = unsigned; };

// even-numbered and odd-numbered elements of a vector of 2 NP columns
__device__ __forceinline__ void split_cols(const float2 v, float &e, float &o) { e = v.x; o = v.y; }
__device__ __forceinline__ void split_cols(const float4 v, float2 &e, float2 &o) { e = make_float2(v.x, v.z); o = make_float2(v.y, v.w); }
__device__ __forceinline__ void split_cols(const unsigned v, unsigned short &e, unsigned short &o) {
    e = static_cast<unsigned short>(v & 0xffffu); o = static_cast<unsigned short>(v >> 16);
}
__device__ __forceinline__ void split_cols(const uint2 v, unsigned &e, unsigned &o) {
    e = __byte_perm(v.x, v.y, 0x5410); o = __byte_perm(v.x, v.y, 0x7632);
}
__device__ __forceinline__ float2 join_cols(const float e, const float o) { return make_float2(e, o); }
__device__ __forceinline__ float4 join_cols(const float2 e, const float2 o) { return make_float4(e.x, o.x, e.y, o.y); }
__device__ __forceinline__ unsigned join_cols(const unsigned short e, const unsigned short o) {
    return static_cast<unsigned>(e) | (static_cast<unsigned>(o) << 16);
}
__device__ __forceinline__ uint2 join_cols(const unsigned e, const unsigned o) {
    return make_uint2(__byte_perm(e, o, 0x5410), __byte_perm(e, o, 0x7632));
}

// X [planes][H][W] -> X' [b][phase][ci][H/2][W/2]. One thread per run of 2 NP neighbouring input columns (one aligned
// vector load; W is a multiple of 2 NP): the even columns go to phase (py, 0), the odd ones to (py, 1), NP elements
// each. phases = 1 keeps the (0,0) phase only (even rows, even columns). Index arithmetic in 32 bits (the host
// checks that the number of runs fits).
template <typename T, int NP>
__global__ void __launch_bounds__(256) phases_of_kernel(const T *__restrict__ X, T *__restrict__ Xp, unsigned planes,
                                                        unsigned Cin, unsigned H, unsigned W, int phases) {
    using V = typename Cols<T, NP>::vec;
    using Hf = typename Cols<T, NP>::half;
    const unsigned Ho = H / 2, Wo = W / 2, Wq = Wo / NP;
    const unsigned rows = phases == 1 ? Ho : H;                   // input rows visited per plane
    const unsigned n = planes * rows * Wq;
    const size_t phase_stride = static_cast<size_t>(Cin) * Ho * Wo;
    for (unsigned i = blockIdx.x * 256u + threadIdx.x; i < n; i += gridDim.x * 256u) {
        const unsigned r = i / Wq, xq = i - r * Wq;
        const unsigned plane = r / rows, yr = r - plane * rows;   // plane = b * Cin + ci
        const unsigned b = plane / Cin, ci = plane - b * Cin;
        const unsigned y = phases == 1 ? 2 * yr : yr;
        const unsigned py = y & 1, yo = y >> 1;
        const V v = *reinterpret_cast<const V *>(X + (static_cast<size_t>(plane) * H + y) * W + 2 * NP * xq);
        Hf e, o;
        split_cols(v, e, o);
        T *dst = Xp + ((static_cast<size_t>(b) * phases + (phases == 1 ? 0 : py * 2)) * Cin + ci) * Ho * Wo +
                 static_cast<size_t>(yo) * Wo + NP * xq;
        *reinterpret_cast<Hf *>(dst) = e;
        if (phases != 1) *reinterpret_cast<Hf *>(dst + phase_stride) = o;
    }
}

// dX' [b][phase][ci][H/2][W/2] -> dX [b][ci][H][W], one thread per run of 2 NP neighbouring output columns;
// phases = 1: only even rows and columns receive a value, the rest is zero.
template <typename T, int NP>
__global__ void __launch_bounds__(256) from_phases_kernel(const T *__restrict__ dXp, T *__restrict__ dX, unsigned planes,
                                                          unsigned Cin, unsigned H, unsigned W, int phases) {
    using V = typename Cols<T, NP>::vec;
    using Hf = typename Cols<T, NP>::half;
    const unsigned Ho = H / 2, Wo = W / 2, Wq = Wo / NP;
    const unsigned n = planes * H * Wq;
    const size_t phase_stride = static_cast<size_t>(Cin) * Ho * Wo;
    for (unsigned i = blockIdx.x * 256u + threadIdx.x; i < n; i += gridDim.x * 256u) {
        const unsigned r = i / Wq, xq = i - r * Wq;
        const unsigned plane = r / H, y = r - plane * H;
        const unsigned b = plane / Cin, ci = plane - b * Cin;
        const unsigned py = y & 1, yo = y >> 1;
        Hf e = Hf(), o = Hf();                                     // zero bits are zero values in both types
        if (phases != 1) {
            const T *src = dXp + ((static_cast<size_t>(b) * 4 + py * 2) * Cin + ci) * Ho * Wo + static_cast<size_t>(yo) * Wo + NP * xq;
            e = *reinterpret_cast<const Hf *>(src);
            o = *reinterpret_cast<const Hf *>(src + phase_stride);
        } else if (py == 0) {
            e = *reinterpret_cast<const Hf *>(dXp + (static_cast<size_t>(plane) * Ho + yo) * Wo + NP * xq);
        }
        *reinterpret_cast<V *>(dX + (static_cast<size_t>(plane) * H + y) * W + 2 * NP * xq) = join_cols(e, o);
    }
}

// tap of the strided layer that (phase bit, tap of the stride-1 layer) stands for, or -1
__device__ __forceinline__ int strided_tap(int phase_bit, int t) {
    return phase_bit ? (t == 0 ? 0 : (t == 1 ? 2 : -1)) : (t == 1 ? 1 : -1);
}

// W [Cout][Cin][3][3] -> W' [Cout][4 Cin][3][3]  (I: index type, 32 bits where the element count allows)
template <typename T, typename I>
__global__ void __launch_bounds__(256) phase_weights_kernel(const T *__restrict__ W, T *__restrict__ Wp, I Cout, I Cin) {
    const I n = Cout * 4 * Cin * 9;
    for (I i = blockIdx.x * I(256) + threadIdx.x; i < n; i += gridDim.x * I(256)) {
        const I r = i / 9;
        const int t = static_cast<int>(i - r * 9);
        const I co = r / (4 * Cin), cp = r - co * 4 * Cin;
        const int ph = static_cast<int>(cp / Cin);
        const I ci = cp - ph * Cin;
        const int ky = strided_tap(ph >> 1, t / 3), kx = strided_tap(ph & 1, t % 3);
        Wp[i] = (ky >= 0 && kx >= 0) ? W[(co * Cin + ci) * 9 + ky * 3 + kx] : static_cast<T>(0.f);
    }
}

// dW' [Cout][4 Cin][3][3] -> dW [Cout][Cin][3][3]: the nine places that hold the strided layer's taps
template <typename I>
__global__ void __launch_bounds__(256) strided_dw_kernel(const float *__restrict__ dWp, float *__restrict__ dW, I Cout, I Cin) {
    const I n = Cout * Cin * 9;
    for (I i = blockIdx.x * I(256) + threadIdx.x; i < n; i += gridDim.x * I(256)) {
        const I r = i / 9;
        const int t = static_cast<int>(i - r * 9);
        const I co = r / Cin, ci = r - co * Cin;
        const int ky = t / 3, kx = t % 3;
        // ky = 0 -> (odd phase, tap 0); 1 -> (even phase, tap 1); 2 -> (odd phase, tap 1)
        const int py = ky != 1, ty = ky == 0 ? 0 : 1;
        const int px = kx != 1, tx = kx == 0 ? 0 : 1;
        dW[i] = dWp[((co * 4 + py * 2 + px) * Cin + ci) * 9 + ty * 3 + tx];
    }
}

}  // namespace

// runs of columns that the layout kernels index with 32 bits
static bool fits32(long long n) { return n < (1ll << 31); }

int launch_phases_of(dbp_ctx *ctx, const void *X, void *Xp, int io, long long B, long long Cin, int H, int W, int phases) {
    const int np = W % 4 == 0 ? 2 : 1;
    const long long n = B * Cin * (phases == 1 ? H / 2 : H) * (W / 2 / np);
    if (!fits32(B * Cin * H * (W / 2))) return DBP_EUNSUPPORTED;
    const int g = blocks_of(n, 256, ctx->sm_count * 16);
    const unsigned planes = static_cast<unsigned>(B * Cin), c = static_cast<unsigned>(Cin), h = H, w = W;
    note_launch();
    if (io == DBP_F32) {
        const float *in = static_cast<const float *>(X);
        float *out = static_cast<float *>(Xp);
        if (np == 2) phases_of_kernel<float, 2><<<g, 256, 0, ctx->stream>>>(in, out, planes, c, h, w, phases);
        else phases_of_kernel<float, 1><<<g, 256, 0, ctx->stream>>>(in, out, planes, c, h, w, phases);
    } else {
        const __nv_bfloat16 *in = static_cast<const __nv_bfloat16 *>(X);
        __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(Xp);
        if (np == 2) phases_of_kernel<__nv_bfloat16, 2><<<g, 256, 0, ctx->stream>>>(in, out, planes, c, h, w, phases);
        else phases_of_kernel<__nv_bfloat16, 1><<<g, 256, 0, ctx->stream>>>(in, out, planes, c, h, w, phases);
    }
    return cuda_ok(cudaGetLastError());
}

int launch_from_phases(dbp_ctx *ctx, const void *dXp, void *dX, int f32, long long B, long long Cin, int H, int W, int phases) {
    const int np = W % 4 == 0 ? 2 : 1;
    const long long n = B * Cin * H * (W / 2 / np);
    if (!fits32(B * Cin * H * (W / 2))) return DBP_EUNSUPPORTED;
    const int g = blocks_of(n, 256, ctx->sm_count * 16);
    const unsigned planes = static_cast<unsigned>(B * Cin), c = static_cast<unsigned>(Cin), h = H, w = W;
    note_launch();
    if (f32) {
        const float *in = static_cast<const float *>(dXp);
        float *out = static_cast<float *>(dX);
        if (np == 2) from_phases_kernel<float, 2><<<g, 256, 0, ctx->stream>>>(in, out, planes, c, h, w, phases);
        else from_phases_kernel<float, 1><<<g, 256, 0, ctx->stream>>>(in, out, planes, c, h, w, phases);
    } else {
        const __nv_bfloat16 *in = static_cast<const __nv_bfloat16 *>(dXp);
        __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(dX);
        if (np == 2) from_phases_kernel<__nv_bfloat16, 2><<<g, 256, 0, ctx->stream>>>(in, out, planes, c, h, w, phases);
        else from_phases_kernel<__nv_bfloat16, 1><<<g, 256, 0, ctx->stream>>>(in, out, planes, c, h, w, phases);
    }
    return cuda_ok(cudaGetLastError());
}

int launch_phase_weights(dbp_ctx *ctx, const void *W, void *Wp, int io, long long Cout, long long Cin) {
    const long long n = Cout * 4 * Cin * 9;
    const int g = blocks_of(n, 256, ctx->sm_count * 16);
    note_launch();
    if (io == DBP_F32) {
        const float *in = static_cast<const float *>(W);
        float *out = static_cast<float *>(Wp);
        if (fits32(n)) phase_weights_kernel<float, unsigned><<<g, 256, 0, ctx->stream>>>(in, out, static_cast<unsigned>(Cout), static_cast<unsigned>(Cin));
        else phase_weights_kernel<float, long long><<<g, 256, 0, ctx->stream>>>(in, out, Cout, Cin);
    } else {
        const __nv_bfloat16 *in = static_cast<const __nv_bfloat16 *>(W);
        __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(Wp);
        if (fits32(n)) phase_weights_kernel<__nv_bfloat16, unsigned><<<g, 256, 0, ctx->stream>>>(in, out, static_cast<unsigned>(Cout), static_cast<unsigned>(Cin));
        else phase_weights_kernel<__nv_bfloat16, long long><<<g, 256, 0, ctx->stream>>>(in, out, Cout, Cin);
    }
    return cuda_ok(cudaGetLastError());
}

int launch_strided_dw(dbp_ctx *ctx, const float *dWp, float *dW, long long Cout, long long Cin) {
    const long long n = Cout * Cin * 9;
    const int g = blocks_of(n, 256, ctx->sm_count * 16);
    note_launch();
    if (fits32(4 * n)) strided_dw_kernel<unsigned><<<g, 256, 0, ctx->stream>>>(dWp, dW, static_cast<unsigned>(Cout), static_cast<unsigned>(Cin));
    else strided_dw_kernel<long long><<<g, 256, 0, ctx->stream>>>(dWp, dW, Cout, Cin);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dbp
