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

template <typename T> struct Pair;
template <> struct Pair<float> { using type = float2; };
template <> struct Pair<__nv_bfloat16> { using type = __nv_bfloat162; };

// X [planes][H][W] -> X' [b][phase][ci][H/2][W/2], one thread per pair of neighbouring input columns (an aligned
// 2-element load; W is even). phases = 1 keeps the (0,0) phase only.
template <typename T>
__global__ void __launch_bounds__(256) phases_of_kernel(const T *__restrict__ X, T *__restrict__ Xp, long long B,
                                                        long long Cin, int H, int W, int phases) {
    using P = typename Pair<T>::type;
    const int Ho = H / 2, Wo = W / 2;
    const long long rows = phases == 1 ? Ho : H;                  // input rows visited per plane
    const long long n = B * Cin * rows * Wo;
    for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += gridDim.x * 256ll) {
        const int xo = static_cast<int>(i % Wo);
        const long long r = i / Wo;
        const int yr = static_cast<int>(r % rows);
        const long long plane = r / rows;                         // b * Cin + ci
        const long long b = plane / Cin, ci = plane - b * Cin;
        const int y = phases == 1 ? 2 * yr : yr;
        const int py = y & 1, yo = y >> 1;
        const P v = *reinterpret_cast<const P *>(X + (plane * H + y) * W + 2 * xo);
        const long long o0 = (((b * phases + (phases == 1 ? 0 : py * 2)) * Cin + ci) * Ho + yo) * Wo + xo;
        Xp[o0] = v.x;
        if (phases != 1) Xp[o0 + Cin * Ho * Wo] = v.y;
    }
}

// dX' [b][phase][ci][H/2][W/2] -> dX [b][ci][H][W], one thread per pair of neighbouring output columns;
// phases = 1: only even rows and columns receive a value, the rest is zero.
template <typename T>
__global__ void __launch_bounds__(256) from_phases_kernel(const T *__restrict__ dXp, T *__restrict__ dX, long long B,
                                                          long long Cin, int H, int W, int phases) {
    using P = typename Pair<T>::type;
    const int Ho = H / 2, Wo = W / 2;
    const long long n = B * Cin * H * Wo;
    for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += gridDim.x * 256ll) {
        const int xo = static_cast<int>(i % Wo);
        const long long r = i / Wo;
        const int y = static_cast<int>(r % H);
        const long long plane = r / H;
        const long long b = plane / Cin, ci = plane - b * Cin;
        const int py = y & 1, yo = y >> 1;
        P v;
        v.x = static_cast<T>(0.f);
        v.y = static_cast<T>(0.f);
        if (phases != 1) {
            const long long o0 = (((b * 4 + py * 2) * Cin + ci) * Ho + yo) * Wo + xo;
            v.x = dXp[o0];
            v.y = dXp[o0 + Cin * Ho * Wo];
        } else if (py == 0) {
            v.x = dXp[((b * Cin + ci) * Ho + yo) * Wo + xo];
        }
        *reinterpret_cast<P *>(dX + (plane * H + y) * W + 2 * xo) = v;
    }
}

// tap of the strided layer that (phase bit, tap of the stride-1 layer) stands for, or -1
__device__ __forceinline__ int strided_tap(int phase_bit, int t) {
    return phase_bit ? (t == 0 ? 0 : (t == 1 ? 2 : -1)) : (t == 1 ? 1 : -1);
}

// W [Cout][Cin][3][3] -> W' [Cout][4 Cin][3][3]
template <typename T>
__global__ void __launch_bounds__(256) phase_weights_kernel(const T *__restrict__ W, T *__restrict__ Wp, long long Cout,
                                                            long long Cin) {
    const long long n = Cout * 4 * Cin * 9;
    for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += gridDim.x * 256ll) {
        const int t = static_cast<int>(i % 9);
        const long long r = i / 9;
        const long long cp = r % (4 * Cin), co = r / (4 * Cin);
        const int ph = static_cast<int>(cp / Cin);
        const long long ci = cp - ph * Cin;
        const int ky = strided_tap(ph >> 1, t / 3), kx = strided_tap(ph & 1, t % 3);
        Wp[i] = (ky >= 0 && kx >= 0) ? W[(co * Cin + ci) * 9 + ky * 3 + kx] : static_cast<T>(0.f);
    }
}

// dW' [Cout][4 Cin][3][3] -> dW [Cout][Cin][3][3]: the nine places that hold the strided layer's taps
__global__ void __launch_bounds__(256) strided_dw_kernel(const float *__restrict__ dWp, float *__restrict__ dW,
                                                         long long Cout, long long Cin) {
    const long long n = Cout * Cin * 9;
    for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += gridDim.x * 256ll) {
        const int t = static_cast<int>(i % 9);
        const long long r = i / 9;
        const long long ci = r % Cin, co = r / Cin;
        const int ky = t / 3, kx = t % 3;
        // ky = 0 -> (odd phase, tap 0); 1 -> (even phase, tap 1); 2 -> (odd phase, tap 1)
        const int py = ky != 1, ty = ky == 0 ? 0 : 1;
        const int px = kx != 1, tx = kx == 0 ? 0 : 1;
        dW[i] = dWp[((co * 4 + py * 2 + px) * Cin + ci) * 9 + ty * 3 + tx];
    }
}

}  // namespace

int launch_phases_of(dbp_ctx *ctx, const void *X, void *Xp, int io, long long B, long long Cin, int H, int W, int phases) {
    const long long n = B * Cin * (phases == 1 ? H / 2 : H) * (W / 2);
    const int g = blocks_of(n, 256, ctx->sm_count * 16);
    note_launch();
    if (io == DBP_F32)
        phases_of_kernel<float><<<g, 256, 0, ctx->stream>>>(static_cast<const float *>(X), static_cast<float *>(Xp), B, Cin, H, W, phases);
    else
        phases_of_kernel<__nv_bfloat16><<<g, 256, 0, ctx->stream>>>(static_cast<const __nv_bfloat16 *>(X),
                                                                    static_cast<__nv_bfloat16 *>(Xp), B, Cin, H, W, phases);
    return cuda_ok(cudaGetLastError());
}

int launch_from_phases(dbp_ctx *ctx, const void *dXp, void *dX, int f32, long long B, long long Cin, int H, int W, int phases) {
    const long long n = B * Cin * H * (W / 2);
    const int g = blocks_of(n, 256, ctx->sm_count * 16);
    note_launch();
    if (f32)
        from_phases_kernel<float><<<g, 256, 0, ctx->stream>>>(static_cast<const float *>(dXp), static_cast<float *>(dX), B, Cin, H, W, phases);
    else
        from_phases_kernel<__nv_bfloat16><<<g, 256, 0, ctx->stream>>>(static_cast<const __nv_bfloat16 *>(dXp),
                                                                      static_cast<__nv_bfloat16 *>(dX), B, Cin, H, W, phases);
    return cuda_ok(cudaGetLastError());
}

int launch_phase_weights(dbp_ctx *ctx, const void *W, void *Wp, int io, long long Cout, long long Cin) {
    const int g = blocks_of(Cout * 4 * Cin * 9, 256, ctx->sm_count * 16);
    note_launch();
    if (io == DBP_F32)
        phase_weights_kernel<float><<<g, 256, 0, ctx->stream>>>(static_cast<const float *>(W), static_cast<float *>(Wp), Cout, Cin);
    else
        phase_weights_kernel<__nv_bfloat16><<<g, 256, 0, ctx->stream>>>(static_cast<const __nv_bfloat16 *>(W),
                                                                        static_cast<__nv_bfloat16 *>(Wp), Cout, Cin);
    return cuda_ok(cudaGetLastError());
}

int launch_strided_dw(dbp_ctx *ctx, const float *dWp, float *dW, long long Cout, long long Cin) {
    const int g = blocks_of(Cout * Cin * 9, 256, ctx->sm_count * 16);
    note_launch();
    strided_dw_kernel<<<g, 256, 0, ctx->stream>>>(dWp, dW, Cout, Cin);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dbp
