/*
 * dbp.h -- C ABI of the dithered-backprop library for NVIDIA B200 (sm_100a).
 *
 * The library computes the backward pass of linear and convolution layers in which the
 * preactivation gradient delta_z is first quantized by non-subtractive dither (NSD) and the
 * resulting sparse tensor of small-integer codes drives both backward products
 * (Wiedemann et al., "Dithered backprop", Section 3: Eq. (nsd), Algorithm 1,
 * Eqs. (qdz), (qda), (qdw)).
 *
 * Conventions for every call
 *   - Unless a function name ends in `_host`, every data pointer is a DEVICE pointer owned by
 *     the caller, to contiguous row-major memory whose base is 16-byte aligned. The library
 *     allocates only its own per-context workspace.
 *   - Calls enqueue work on the context's CUDA stream and return without synchronising
 *     (the `_host` variants and dbp_last_device_status synchronise the stream).
 *   - Return value: DBP_OK or a negative dbp_status. Errors the host can see (null or
 *     misaligned pointers, bad sizes, unsupported kernel size) return before anything is
 *     enqueued. Conditions only the device can see (non-finite delta, codes clipped to
 *     +-127) leave all outputs defined and are reported by dbp_last_device_status.
 *   - There is no CPU fallback: every step runs in the library's CUDA kernels.
 *   - One context per host thread and stream; calls on one context are not re-entrant.
 */
#ifndef DBP_H_
#define DBP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dbp_ctx dbp_ctx;

typedef enum { DBP_F32 = 0, DBP_BF16 = 1 } dbp_dtype;

typedef enum {
    DBP_OK = 0,
    DBP_EINVAL = -1,        /* null / misaligned pointer, non-positive size, bad enum */
    DBP_EUNSUPPORTED = -2,  /* kernel size, stride or padding outside {1x1, 3x3; 1, 2; (k-1)/2} and {5x5; 1; 2} */
    DBP_ECUDA = -3,         /* a CUDA runtime call failed */
    DBP_ENOMEM = -4,        /* workspace allocation failed */
    DBP_ENONFINITE = -5,    /* device: delta holds NaN or Inf (all codes were set to 0) */
    DBP_ESATURATED = -6,    /* device: some codes were clipped to +-127 */
    DBP_ECAPACITY = -7,     /* a caller-provided size is smaller than required */
    DBP_ETIMEOUT = -8       /* device: a bounded wait inside a kernel expired (results undefined) */
} dbp_status;

/* flags for the backward calls */
#define DBP_FORCE_SPARSE 1u /* always use the sparse gather kernels */
#define DBP_FORCE_DENSE  2u /* always use the dense tensor-core path; DBP_EUNSUPPORTED where it
                               does not exist (it covers bf16 linear and 1x1 layers and bf16 or fp32 3x3
                               layers, channel counts multiples of 8, 3x3 images up to 62 wide; fp32
                               operands enter the tensor cores as two bf16 pieces each) */
#define DBP_DX_F32       4u /* with io = DBP_BF16: write dX as fp32 instead of bf16 */
#define DBP_DW_ASYNC     8u /* dense path with both dW and dX asked for: the call returns with dX (and db)
                               ordered on the context's stream as usual, while dW is still being computed on
                               the context's second stream. dW (and the scratch it needs) is ordered into the
                               context's stream by dbp_join, by dbp_last_device_status / dbp_last_step, or by
                               dbp_destroy; until then the caller must not read dW nor overwrite X. This is the
                               order a training step needs: the layer below depends on dX only, the weight
                               gradients are needed by the optimizer at the end. */

/*
 * Density crossover (Section 3.4: the sparse products cost O(p_nz m k n), a dense product
 * O(m k n) at a much higher arithmetic rate on tensor cores). Without a FORCE flag a layer
 * that the dense path supports uses it when the context's estimate of p_nz exceeds
 * `crossover`; the estimate is the density last measured on a layer of the same shape on this
 * context (read back asynchronously, so no call waits for it; 1.0, i.e. dense, until the first
 * measurement of that shape has arrived). crossover >= 1 disables the dense path, crossover <= 0
 * always prefers it. The default is 0: on B200 the tensor-core path measured 2.3x to 11x faster than
 * the gather kernels at every density between 22 % and 0.6 %.
 */
int dbp_set_crossover(dbp_ctx *ctx, float crossover);

/* Elements per segment of the sparse structure (see dbp_sparse). */
#define DBP_SEGMENT 1024

/*
 * Sparse form of the quantized gradient delta~ = Delta * q (the "sparse tensors with low
 * precision non-zero values" of Section 1; the paper fixes no storage format, this one is
 * the library's). The tensor is taken flat, element i at its row-major offset.
 *   bitmap  : bit (i & 31) of word (i >> 5) is 1 iff q_i != 0.
 *   values  : the non-zero int8 codes of segment g (elements g*1024 ... g*1024+1023) in
 *             element order, packed from values[g*1024]; bytes past the segment's count
 *             are unspecified.
 *   offsets : offsets[w] = number of non-zero codes of word w's segment that precede word w.
 *             So code i lives at values[(i>>10)*1024 + offsets[i>>5] + popc(bitmap[i>>5] &
 *             ((1u << (i&31)) - 1))].
 *   delta   : device scalar, the step size Delta used.
 *   nnz     : device scalar, number of non-zero codes.
 * Buffer sizes for a given numel come from dbp_sparse_bytes.
 */
typedef struct dbp_sparse {
    uint32_t *bitmap;
    uint16_t *offsets;
    int8_t *values;
    float *delta;
    long long *nnz;
    long long numel;
} dbp_sparse;

/* Context. `device` is a CUDA ordinal; `cuda_stream` is a cudaStream_t (NULL = default
 * stream). The context owns its workspace and frees it in dbp_destroy. The workspace grows
 * (cudaMalloc, which synchronises the device) the first time a call needs more of it than any
 * call before: the dense codes of delta (1 and/or 2 bytes per element), re-laid weights,
 * activations copied to 16-byte aligned planes, the split-K partial blocks of dW. Calls of
 * sizes seen before allocate nothing. Kernels of consecutive calls on one context may overlap at
 * their edges (a kernel becomes resident while the one before it drains) but never read data
 * before the kernel that writes it has completed. */
int dbp_create(dbp_ctx **out, int device, void *cuda_stream);
int dbp_destroy(dbp_ctx *ctx);
int dbp_set_stream(dbp_ctx *ctx, void *cuda_stream);
/* Kernels the library has launched in this process so far (every launch is counted). */
long long dbp_kernel_launches(void);

/* fp32 FMA throughput of the context's device in TFLOP/s, measured with dependent FMA chains on
 * every lane (the arithmetic ceiling of the sparse gather kernels). Synchronises. */
int dbp_measure_fma_peak(dbp_ctx *ctx, double *tflops);

/* Makes the context's stream wait for every dW computation that earlier DBP_DW_ASYNC calls left
 * running (a stream-ordered join: nothing blocks on the host). */
int dbp_join(dbp_ctx *ctx);
const char *dbp_status_string(int status);
/* Text of the most recent DBP_ECUDA on the calling thread: which step failed and the CUDA
 * runtime's message (empty if none yet). The pointer stays valid; the text changes with the next
 * failure on this thread. */
const char *dbp_last_error(void);

/* Synchronises the stream, then reports the device-side condition of the calls since the
 * previous report (DBP_OK, DBP_ETIMEOUT, DBP_ENONFINITE or DBP_ESATURATED, the first that
 * applies) and the number of clipped codes; both outputs may be NULL. Clears the record. */
int dbp_last_device_status(dbp_ctx *ctx, int *status, long long *saturated);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper). Every wait inside
 * the tensor-core kernels gives up after a clock budget, records DBP_ETIMEOUT for
 * dbp_last_device_status and lets the kernel return. This call enqueues a one-warp kernel that
 * runs the same wait, with a budget of `cycles` SM clocks (0 ... 10^8), on a barrier nothing
 * ever arrives on: afterwards dbp_last_device_status reports DBP_ETIMEOUT once and the context
 * keeps working. It touches no product kernel and no caller data.
 */
int dbp_selftest_bounded_wait(dbp_ctx *ctx, long long cycles);

/*
 * Per-kernel device timing (a measurement aid, off by default). While enabled, every kernel
 * the library launches is bracketed by CUDA events on the context's stream.
 * dbp_profile_read synchronises the stream and returns, for one kernel kind, the summed
 * device time in milliseconds and the number of launches since the previous read of that
 * kind (either output may be NULL). The events themselves cost a few microseconds of stream
 * time each, so dbp_profile_select can restrict the timing to some kinds: bit k of
 * `kind_mask` set = launches of kind k are timed (default: all kinds).
 */
typedef enum {
    DBP_K_STATISTICS = 0, /* sigma / Delta reduction */
    DBP_K_QUANTIZE = 1,   /* dither + quantize + compact */
    DBP_K_WEIGHT_TAPS = 2,/* weight re-layout for dX */
    DBP_K_DX = 3,         /* sparse input-gradient product */
    DBP_K_DW = 4,         /* sparse weight-gradient product */
    DBP_K_DB = 5,         /* bias gradient */
    DBP_K_DECODE = 6,     /* sparse -> dense codes */
    DBP_K_GLUE = 7,       /* ReLU derivative / max-pool routing */
    DBP_K_DX_DENSE = 8,   /* tensor-core input-gradient product */
    DBP_K_DW_DENSE = 9,   /* tensor-core weight-gradient product (with its split-K reduction) */
    DBP_K_FUSED = 10,     /* whole backward pass of a small fp32 linear layer (two chained launches) */
    DBP_K_COUNT = 11
} dbp_kernel_kind;
int dbp_profile_enable(dbp_ctx *ctx, int on);
int dbp_profile_select(dbp_ctx *ctx, unsigned kind_mask);
int dbp_profile_read(dbp_ctx *ctx, int kind, double *milliseconds, long long *launches);

/*
 * Where the TMA-fed 3x3 kernels' issuing threads stood still (a measurement aid). Each of those
 * kernels has one thread that issues MMAs and one or two that issue copies; every time one of them
 * waits on a barrier the SM clocks it waited are added to a counter, summed over all CTAs:
 *   [0] MMA thread waiting for a code tile        [1] MMA thread waiting for weights / activations
 *   [2] MMA thread waiting for a free accumulator [3] code-copy thread waiting for a free buffer
 *   [4] weight/activation-copy thread waiting for a free buffer
 *   [5] dX: epilogue thread 0 waiting for an accumulator; dW: clocks its additions into dW took
 *   [6] lifetime of the MMA thread                [7] CTAs that reported
 * dbp_wait_stats synchronises the stream, copies the DBP_WAIT_SLOTS counters to `out` (host) and
 * clears them when `reset` is non-zero.
 */
#define DBP_WAIT_SLOTS 8
int dbp_wait_stats(dbp_ctx *ctx, unsigned long long *out, int reset);

/* Bytes the caller must allocate for each array of a dbp_sparse over `numel` elements. */
int dbp_sparse_bytes(long long numel, size_t *bitmap_bytes, size_t *offsets_bytes,
                     size_t *values_bytes);

/*
 * Algorithm 1 (NSD): sigma = population std of delta over all `numel` elements,
 * Delta = scale * sigma, q_i = floor(delta_i / Delta + u_i) (Eq. (nsd) with the dither
 * nu_i = (u_i - 1/2) Delta), clipped to [-127, 127].
 *   delta    : numel elements of `dtype`.
 *   seed     : u_i comes from output (i >> 1) of the SplitMix64 sequence started at `seed`
 *              (low 32 bits for even i, high for odd); its top 23 bits k give
 *              u_i = (2k+1) 2^-24.
 *   scale    : s > 0. If scale <= 0 the step is read from the device scalar *delta_in.
 *   out      : arrays sized by dbp_sparse_bytes; out->numel is set by the call;
 *              *out->delta and *out->nnz are written on the device.
 * sigma = 0 is not an error (Delta = 0, every code 0).
 */
int nsd_quantize(dbp_ctx *ctx, const void *delta, int dtype, long long numel,
                 unsigned long long seed, float scale, const float *delta_in, dbp_sparse *out);

/*
 * Step size and non-zero count of the context's most recent quantization (the one inside the
 * latest nsd_quantize or dithered_*_backward call): Algorithm 1's Delta and the nnz of
 * Eq. (nsd)'s codes, for callers that passed no dbp_sparse. HOST outputs (either may be NULL);
 * the call synchronises the context's stream.
 */
int dbp_last_step(dbp_ctx *ctx, float *delta_out, long long *nnz_out);

/*
 * Seed of layer `layer` (0-based, forward order) of a network whose backward pass was given
 * `seed`: every layer draws its own dither (Eq. (qdz) quantizes each layer's delta_z
 * independently), so layer l uses output l of the SplitMix64 sequence started at `seed`.
 * Pure host function; no context needed.
 */
unsigned long long dbp_layer_seed(unsigned long long seed, int layer);

/* Expands a dbp_sparse to one int8 code per element (codes: numel bytes, device). */
int nsd_decode_dense(dbp_ctx *ctx, const dbp_sparse *q, int8_t *codes);

/*
 * Dithered backward of a linear layer z = a W^T (Eqs. (qdz), (qda), (qdw), row-major batch
 * form): quantizes delta [B,N] as in nsd_quantize, then
 *     dX[b,k] = Delta sum_j q[b,j] W[j,k]      dW[j,k] = Delta sum_b q[b,j] X[b,k]
 *     db[j]   = Delta sum_b q[b,j]
 * X [B,K], W [N,K], delta [B,N] are of dtype `io`; dW [N,K] and db [N] are fp32; dX [B,K]
 * is of dtype `io` (fp32 with DBP_DX_F32). Any of dW, dX, db may be NULL (skipped).
 * q_out may be NULL; otherwise it receives the sparse structure (arrays sized for B*N).
 * Outputs are overwritten, not accumulated.
 * fp32 layers with B*N <= 2^17, no q_out and no FORCE flag run as two chained kernels (statistics, dither
 * and quantization; then the products; profiling kind DBP_K_FUSED): same results to the same tolerances,
 * Delta and nnz through dbp_last_step.
 */
int dithered_linear_backward(dbp_ctx *ctx, const void *delta, const void *X, const void *W,
                             int io, long long B, long long N, long long K,
                             unsigned long long seed, float scale, const float *delta_in,
                             dbp_sparse *q_out, float *dW, void *dX, float *db,
                             unsigned flags);

/*
 * The same for a convolution layer ("analogous for convolutional layers", Section 3):
 * cross-correlation, NCHW, square kernel k in {1, 3}, stride 1 or 2, zero padding (k-1)/2; also k = 5 with
 * stride 1 and padding 2 (the 5x5 layers of LeNet-5-like networks; these run on the gather kernels only).
 * H and Wd are the height and width of X. Stride 1: delta [B,Cout,H,W], X [B,Cin,H,W], W [Cout,Cin,k,k]:
 *     dX[b,ci,y,x]     = Delta sum_{co,ky,kx} q[b,co,y-ky+p,x-kx+p] W[co,ci,ky,kx]
 *     dW[co,ci,ky,kx]  = Delta sum_{b,y,x}    q[b,co,y,x] X[b,ci,y+ky-p,x+kx-p]
 *     db[co]           = Delta sum_{b,y,x}    q[b,co,y,x]
 * Stride 2 (the down-sampling layers of residual networks; H and Wd even, else DBP_EUNSUPPORTED):
 * delta [B,Cout,H/2,W/2] is the gradient at the layer's own output positions, X and dX stay [B,Cin,H,W]:
 *     dW[co,ci,ky,kx]  = Delta sum_{b,y,x} q[b,co,y,x] X[b,ci,2y+ky-p,2x+kx-p]
 *     dX[b,ci,y',x']   = Delta sum of q[b,co,y,x] W[co,ci,ky,kx] over the (co,ky,kx,y,x) with 2y+ky-p = y', 2x+kx-p = x'
 * computed as the stride-1 layer on the four phase images of X (layout kernels on the context's stream around
 * the same quantizer and product kernels; workspaces of the size of X, dX and 4x the weights). Such a call always
 * joins its weight-gradient kernels before it returns (DBP_DW_ASYNC is ignored). q_out describes delta as given.
 * Other k, stride or pad return DBP_EUNSUPPORTED.
 */
int dithered_conv_backward(dbp_ctx *ctx, const void *delta, const void *X, const void *W,
                           int io, long long B, long long Cin, long long Cout, long long H,
                           long long Wd, int k, int stride, int pad,
                           unsigned long long seed, float scale, const float *delta_in,
                           dbp_sparse *q_out, float *dW, void *dX, float *db, unsigned flags);

/*
 * Host-buffer variants: every pointer (delta, X, W, dW, dX, db, and the two scalars) is a
 * HOST pointer. The call copies the inputs to the device workspace, runs the same kernels,
 * copies the results back and synchronises. delta_out / nnz_out (may be NULL) receive the
 * step size and the number of non-zero codes.
 */
int dithered_linear_backward_host(dbp_ctx *ctx, const void *delta, const void *X, const void *W,
                                  int io, long long B, long long N, long long K,
                                  unsigned long long seed, float scale,
                                  float *dW, void *dX, float *db, unsigned flags,
                                  float *delta_out, long long *nnz_out);
int dithered_conv_backward_host(dbp_ctx *ctx, const void *delta, const void *X, const void *W,
                                int io, long long B, long long Cin, long long Cout, long long H,
                                long long Wd, int k, int stride, int pad,
                                unsigned long long seed, float scale,
                                float *dW, void *dX, float *db, unsigned flags,
                                float *delta_out, long long *nnz_out);

/*
 * delta_z = delta_a (.) f'(z) folded into the next call (the elementwise step in front of Eq. (qdz)): `mask`
 * (DEVICE, one byte per element of delta, non-zero where z > 0; must stay valid until that call's kernels have
 * run) makes the next dithered_linear_backward / dithered_conv_backward on this context treat its `delta`
 * argument as delta_a and quantize delta_a (.) mask. fp32 only (DBP_EUNSUPPORTED otherwise, at that call).
 * Small linear layers and fp32 3x3 layers on the tensor-core kernels apply the mask while they read delta_a
 * (no extra pass, no delta_z in memory; the mask must then start on a 4-byte boundary, else the next form is
 * taken); other layers run the ReLU-derivative kernel into a workspace first. The setting is consumed by that one call.
 * mask = NULL clears it.
 */
int dbp_set_relu_mask(dbp_ctx *ctx, const uint8_t *mask);

/*
 * Elementwise steps between layers of a network's backward pass (Section 3, backward
 * equations): delta_z = delta_a (.) f'(z) for ReLU, with the derivative given as one byte
 * per element (0 or 1), and the 2x2 max-pool routing of a pooled gradient g [planes,h,w] to
 * out [planes,2h,2w], argmax in {0,1,2,3} being the row-major position of the forward
 * maximum inside each window. fp32 device arrays.
 */
int dbp_relu_backward(dbp_ctx *ctx, const float *delta_a, const uint8_t *mask, float *delta_z,
                      long long numel);
int dbp_maxpool2x2_backward(dbp_ctx *ctx, const float *g, const int8_t *argmax, float *out,
                            long long planes, long long h, long long w);

/*
 * Step size without any allocation (the paper has no counterpart: this entry point exists
 * for the way the library is embedded, not for the method).
 *
 * Every other call needs a dbp_ctx, and a context allocates: dbp_create and the first call
 * of each size call cudaMalloc for the workspace. Some hosts cannot do that at the point
 * where they need the step size -- a serving process whose device memory is handed out once
 * at start-up and then frozen, a real-time loop that must not hit the implicit device
 * synchronisation of cudaMalloc/cudaFree, a plug-in that runs inside someone else's memory
 * budget. For them this call computes Delta = scale * std(delta) (Algorithm 1's first two
 * lines; it agrees with nsd_quantize's Delta within 1e-6 relative) with no context and no
 * allocation of any kind: the reduction's scratch is a fixed array of about 16 KB inside the
 * library image, present on every GPU that loads the library until the process exits.
 *
 *   delta      : DEVICE pointer, numel elements of dtype (DBP_F32 / DBP_BF16), 16-byte aligned.
 *   numel      : 1 ... DBP_NOALLOC_MAX_NUMEL; larger tensors return DBP_ECAPACITY and nothing
 *                is enqueued.
 *   scale      : s > 0.
 *   delta_out  : DEVICE pointer to one float, written by the kernel.
 *   cuda_stream: cudaStream_t to enqueue on (NULL = default stream); the call does not
 *                synchronise. It runs on the CURRENT device.
 *
 * The first call on each device looks up the device address of the scratch array (a runtime
 * query, no allocation); make that first call outside any stream capture.
 * All calls on one device share the one scratch array, which keeps whatever the previous
 * call left in it; the call resets the part that must start at zero. Two calls whose
 * kernels can overlap on the same GPU (different streams, different threads) race on it:
 * serialise them. Non-finite input gives Delta = 0.
 */
#define DBP_NOALLOC_MAX_NUMEL (1ll << 31)
int nsd_step_size_noalloc(const void *delta, int dtype, long long numel, float scale,
                          float *delta_out, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DBP_H_ */
