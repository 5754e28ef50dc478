// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "dbp.h"

namespace dbp {

constexpr int kSegment = DBP_SEGMENT;          // elements per sparse segment
constexpr int kWordsPerSegment = kSegment / 32;

// Device-side scalars of one context.
struct DeviceState {
    float delta;                        // step size of the internal quantization
    int nonfinite;                      // set when delta_z held NaN/Inf
    unsigned int ticket;                // last-block election of the statistics kernel
    int tc_timeout;                     // a bounded wait of a tensor-core kernel expired
    unsigned long long nnz;             // non-zero codes of the internal quantization
    unsigned long long saturated;       // clipped codes since the last report
};

struct ProfSlot {
    cudaEvent_t begin, end;
    int kind;
};

struct Workspace {
    void *ptr = nullptr;
    size_t bytes = 0;
};

}  // namespace dbp

struct dbp_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    int sm_count = 148;
    dbp::DeviceState *state = nullptr;  // device
    double *partials = nullptr;         // device, statistics partial sums
    unsigned long long *wait_stats = nullptr;   // device, DBP_WAIT_SLOTS counters of SM clocks spent waiting
    int partial_blocks = 0;
    // The codes of a layer exist in two sets of buffers used in turn: with DBP_DW_ASYNC the dW kernels of
    // one call may still read their set while the next call's quantization writes the other one.
    dbp::Workspace dense_codes[2];      // int8 per element of delta
    dbp::Workspace x_padded;            // activations copied to 16-byte aligned planes
    dbp::Workspace codes16[2];          // bf16 code planes for the TMA-fed kernels
    dbp::Workspace w_taps;              // fp32 weights as [Cout][k*k][Cin]
    dbp::Workspace sp_bitmap, sp_offsets, sp_values;  // internal dbp_sparse
    dbp::Workspace tc_partials;         // split-K partial blocks of the dense dW kernel
    dbp::Workspace codes_nhwc[2];       // bf16 codes [B][position][Cout] for the TMA-fed 3x3 kernels
    const uint8_t *next_mask = nullptr; // ReLU mask for the next backward call (dbp_set_relu_mask)
    dbp::Workspace dz_tmp;              // delta_z = delta_a (.) mask when that call cannot fold the mask into its loads
    dbp::Workspace codes_stack[2];      // the same codes with G images stacked into one tall image (tiny planes, dW)
    const void *phase_w_src = nullptr;  // that layer's own weights: its W argument is a workspace for the phase weights, not yet written
    float *phase_dw_out = nullptr;      // that layer's dW: the 3x3 weight-gradient kernels write it directly when they run in phase mode ...
    bool phase_dw_done = false;         // ... and say so here
    int phase_cin = 0;                  // > 0 while a stride-2 3x3 layer runs as a stride-1 layer on phase images: its own channel count
    dbp::Workspace s2_x, s2_w, s2_dx, s2_dw;   // stride-2 layers: phase images of X, phase weights, and the two products in that layout
    float *delta_sets = nullptr;        // device float[2]: the step size that belongs to each set
    int code_set = 0;                   // the set the next call writes
    cudaEvent_t ev_set_free[2] = {nullptr, nullptr};   // recorded on the dW stream after the set's last reader
    bool set_busy[2] = {false, false};
    bool aux_pending = false;           // dW work on the second stream that the caller's stream is not yet ordered after
    dbp::Workspace dw_acc;              // fp32 [tap][Cout][Cin] that the 3x3 dW CTAs add into; zero between calls
    bool dw_acc_clean = false;
    dbp::Workspace io[8];               // staging for the *_host entry points
    // *_host entry points: X goes up and dX comes down on streams of their own, so that the two
    // directions of the host link work at the same time; the events order them against the
    // kernels (dX done -> its read-back may start; X up -> the dW kernels may start)
    // the dense dW kernels of a layer run beside its dX kernel on a stream of their own (they only
    // share inputs): forked after the quantization, joined before the call returns to the caller's stream
    cudaStream_t aux = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_x_up = nullptr, ev_dx_done = nullptr;
    cudaEvent_t hook_after_dx = nullptr, hook_before_dw = nullptr;   // set only during a *_host call
    // density above which the dense path is preferred. Measured (sparse against dense time for a 1x1, a 3x3 and a
    // linear layer, densities 22 % ... 0.6 %): the tensor-core path is 2.3x to 11x faster at every density, the gather
    // kernels' time being mostly the scan of the dense codes; so wherever the dense path exists it is the default.
    float crossover = 0.0f;
    // densities measured so far, by layer shape (the path choice of a call uses its own shape's entry)
    struct DensityEntry { unsigned long long key; float density; };
    std::vector<DensityEntry> densities;
    unsigned long long nnz_host_key = 0;         // shape whose read-back is in flight
    unsigned long long *nnz_host = nullptr;   // pinned: asynchronous read-back of nnz
    long long nnz_host_numel = 0;
    cudaEvent_t nnz_event = nullptr;
    bool nnz_pending = false;
    bool profiling = false;
    unsigned prof_mask = 0xffffffffu;   // kinds that are timed while profiling is on
    std::vector<dbp::ProfSlot> prof;    // event pairs, reused after every read
    size_t prof_used = 0;
    double prof_ms[DBP_K_COUNT] = {0};
    long long prof_launches[DBP_K_COUNT] = {0};
};

namespace dbp {

int ws_reserve(dbp_ctx *ctx, Workspace &w, size_t bytes);

// ---- nsd_kernels.cu
// Work the statistics kernel does on the side for the layer's product kernels (its blocks have time to spare
// and this saves launches): clearing a buffer (16-byte aligned, a multiple of 16 bytes), and re-laying 3x3
// weights [Cout][Cin][9] as [Cout][taps][Cin] bf16 (taps = 9 for bf16 weights; 18 for fp32 weights, split into
// two bf16 pieces: taps 0-8 the rounded values, 9-17 what the rounding left over).
struct SideJobs {
    void *zero = nullptr;
    size_t zero_bytes = 0;
    const void *w_src = nullptr;       // null: no weights to re-lay
    void *w_dst = nullptr;
    int w_f32 = 0;
    long long Cout = 0, Cin = 0;
    int phase_cin = 0;                 // > 0: w_src holds a stride-2 layer's own weights [Cout][phase_cin][9], Cin = 4 phase_cin
};
int launch_statistics(dbp_ctx *ctx, const void *delta, int dtype, long long numel, float scale,
                      const float *delta_in, float *delta_out, unsigned long long *nnz_out,
                      const SideJobs &jobs = SideJobs(), const uint8_t *mask = nullptr);
int launch_quantize(dbp_ctx *ctx, const void *delta, int dtype, long long numel,
                    unsigned long long seed, const float *delta_p, uint32_t *bitmap,
                    uint16_t *offsets, int8_t *values, int8_t *dense,
                    unsigned long long *nnz_out);
// ---- nsd_dense.cu: the same codes, dense array only (no sparse structure)
// dense: int8 codes in delta's order (or null); planes_bf16: bf16 codes as [numel / hw][pitch]
// (or null), pitch a multiple of 8
int launch_quantize_dense(dbp_ctx *ctx, const void *delta, int dtype, long long numel,
                          unsigned long long seed, const float *delta_p, int8_t *dense,
                          void *planes_bf16, long long hw, long long pitch, bool count);
// position-major bf16 codes [B][HW][C] for the TMA-fed 3x3 kernels (and int8 codes in delta's order
// when dense8 is not null)
int launch_quantize_nhwc(dbp_ctx *ctx, const void *delta, int dtype, long long B, long long C, long long HW,
                         unsigned long long seed, const float *delta_p, void *codes_nhwc, int8_t *dense8, bool count,
                         void *codes_stack = nullptr, int plane_w = 0, int stack_g = 0, const uint8_t *mask = nullptr);
int launch_decode(dbp_ctx *ctx, const uint32_t *bitmap, const uint16_t *offsets,
                  const int8_t *values, long long numel, int8_t *dense);

// ---- small_linear.cu: one launch for the whole backward pass of a small fp32 linear layer
bool small_linear_fits(const dbp_ctx *ctx, long long B, long long N, long long K, bool want_dw, bool want_dx);
int launch_small_linear(dbp_ctx *ctx, const float *delta, const float *X, const float *W, long long B, long long N,
                        long long K, unsigned long long seed, float scale, const float *delta_in, float *dW, float *dX,
                        float *db, float *delta_set, const uint8_t *mask = nullptr);

// ---- product_kernels.cu
struct ConvShape {
    long long B, Cin, Cout, H, W;
    int k;
};
// weights as [Cout][k*k][Cin]; kept in their own dtype unless to_f32
int launch_weight_taps(dbp_ctx *ctx, const void *W, int dtype, const ConvShape &s, void *w_taps,
                       bool to_f32);
int launch_conv_dx_streamed(dbp_ctx *ctx, const int8_t *codes, const void *w_taps, int w_dtype,
                            const float *delta_p, const ConvShape &s, void *dX, bool dx_bf16);
int launch_conv_dx(dbp_ctx *ctx, const int8_t *codes, const float *w_taps, const float *delta_p,
                   const ConvShape &s, void *dX, bool dx_bf16);
int launch_conv_dw(dbp_ctx *ctx, const int8_t *codes, const void *X, int dtype,
                   const float *delta_p, const ConvShape &s, float *dW);
int launch_conv_dw_streamed(dbp_ctx *ctx, const int8_t *codes, const void *X, int dtype,
                            const float *delta_p, const ConvShape &s, float *dW);
// ---- tc_dense.cu
bool tc_supported(const ConvShape &s, int io);
int launch_tc_dw(dbp_ctx *ctx, const int8_t *codes, const void *X, const float *delta_p,
                 const ConvShape &s, float *dW, int *err_flag);
int launch_tc_dx(dbp_ctx *ctx, const int8_t *codes, const void *W, const float *delta_p,
                 const ConvShape &s, void *dX, bool dx_bf16, int *err_flag);
// ---- tma_dx.cu: 1x1 dX with TMA-fed operands; codes as bf16 planes [B*Cout][tma_code_pitch]
bool tma_dx_supported(const ConvShape &s, int io);
long long tma_code_pitch(const ConvShape &s);
int launch_tma_dx(dbp_ctx *ctx, const void *codes_bf16, const void *W, const float *delta_p,
                  const ConvShape &s, void *dX, bool dx_bf16, int *err_flag);
// ---- tma_dw.cu: 1x1 dW with TMA-fed operands (same code planes)
bool tma_dw_supported(const ConvShape &s, int io);
int launch_tma_dw(dbp_ctx *ctx, const void *codes_bf16, const void *X, const float *delta_p,
                  const ConvShape &s, float *dW, int *err_flag);
// planes of H x W bf16 values -> rows of Wp values (multiple of 8), extra columns zero
int launch_pad_planes(dbp_ctx *ctx, const void *in, void *out, long long planes, int H, int W, int Wp);
// dW = Delta * sum of nsplit partial blocks of nw floats (nw % 4 == 0), fixed order
int launch_dw_sum(dbp_ctx *ctx, const float *partials, int nsplit, long long nw, const float *delta_p, float *dW);
// ---- tc3_tma_dx.cu / tc3_tma_dw.cu: 3x3 products with TMA-fed operands; codes as bf16 [B][H*W][Cout]
bool tc3_tma_supported(const ConvShape &s, int io);
bool tc3_tma_dw_supported(const ConvShape &s, int io);     // dW alone: also fp32 layers with any Cin
// io: the operands' type; fp32 weights / activations are split into two bf16 pieces on the way in
// weights_ready: ctx->w_taps already holds the re-laid weights (the statistics kernel did it on the side)
int launch_tc3_tma_dx(dbp_ctx *ctx, const void *codes_nhwc, const void *W, int io, const float *delta_p,
                      const ConvShape &s, void *dX, bool dx_bf16, int *err_flag, bool weights_ready = false);
int launch_tc3_tma_dw(dbp_ctx *ctx, const void *codes_nhwc, const void *X, int io, const float *delta_p,
                      const ConvShape &s, float *dW, int *err_flag, int stack_g = 0, int real_h = 0);
// Planes of fewer than 64 positions: how many images of a batch to stack into one tall image (one zero row after
// every image) for the weight-gradient kernel, whose work comes in segments of one image; 0: do not stack.
int tc3_stack_images(const ConvShape &s, int io);
int launch_bias_grad(dbp_ctx *ctx, const int8_t *codes, const float *delta_p, const ConvShape &s,
                     float *db);
int launch_relu_backward(dbp_ctx *ctx, const float *da, const uint8_t *mask, float *dz,
                         long long n);
int launch_maxpool_backward(dbp_ctx *ctx, const float *g, const int8_t *argmax, float *out,
                            long long planes, long long h, long long w);

// ---- strided_conv.cu: layout changes around a stride-2 layer run as a stride-1 layer on the input's phase images
// (phases = 4: all four, channel (py*2+px)*Cin + ci; phases = 1: the even rows and columns only)
int launch_phases_of(dbp_ctx *ctx, const void *X, void *Xp, int io, long long B, long long Cin, int H, int W, int phases);
int launch_from_phases(dbp_ctx *ctx, const void *dXp, void *dX, int f32, long long B, long long Cin, int H, int W, int phases);
int launch_phase_weights(dbp_ctx *ctx, const void *W, void *Wp, int io, long long Cout, long long Cin);
int launch_strided_dw(dbp_ctx *ctx, const float *dWp, float *dW, long long Cout, long long Cin);

// ---- selftest.cu
int launch_bounded_wait_selftest(dbp_ctx *ctx, long long budget);
// fp32 FMA throughput of the device (dependent chains on every lane of every SM), TFLOP/s
int measure_fma_peak(dbp_ctx *ctx, double *tflops);

// Brackets one kernel launch with events while profiling is on.
struct KernelTimer {
    dbp_ctx *ctx;
    ProfSlot *slot = nullptr;
    KernelTimer(dbp_ctx *c, int kind) : ctx(c) {
        if (!c->profiling || !((c->prof_mask >> kind) & 1u)) return;
        if (c->prof_used == c->prof.size()) {
            ProfSlot s;
            if (cudaEventCreate(&s.begin) != cudaSuccess) return;
            if (cudaEventCreate(&s.end) != cudaSuccess) { cudaEventDestroy(s.begin); return; }
            s.kind = kind;
            c->prof.push_back(s);
        }
        slot = &c->prof[c->prof_used++];
        slot->kind = kind;
        cudaEventRecord(slot->begin, c->stream);
    }
    ~KernelTimer() {
        if (slot) cudaEventRecord(slot->end, ctx->stream);
    }
};

// Split of a K loop of `kunits` steps over CTAs when `tiles` output tiles exist and one CTA fits
// per SM: the CTAs run in ceil(tiles * split / sms) waves of ceil(kunits / split) steps each, so
// a split that spills a few CTAs into another wave doubles the time. Picks the split with the
// fewest wave-steps (a CTA's fixed cost counted as two steps, a small charge per split for the
// partial sums); *per_split receives the steps per CTA. The returned split has no empty part.
inline long long choose_split(long long tiles, long long kunits, int sms, long long *per_split) {
    long long best = 1, best_per = kunits;
    double best_cost = 1e300;
    const long long smax = kunits < 4ll * sms ? kunits : 4ll * sms;
    for (long long want = 1; want <= smax; ++want) {
        const long long per = (kunits + want - 1) / want, split = (kunits + per - 1) / per;
        const long long waves = (tiles * split + sms - 1) / sms;
        const double cost = static_cast<double>(waves) * static_cast<double>(per + 2) + 0.05 * static_cast<double>(split);
        if (cost < best_cost) { best_cost = cost; best = split; best_per = per; }
    }
    *per_split = best_per;
    return best;
}

// Records where a CUDA call failed and what the runtime said (read back with dbp_last_error);
// returns DBP_ECUDA.
int fail_cuda(const char *what, cudaError_t e);
inline int fail_cuda(const char *what) { return fail_cuda(what, cudaGetLastError()); }

// Every kernel launch of the library passes here (a process-wide count, read by dbp_kernel_launches).
void note_launch();

inline int cuda_ok(cudaError_t e) { return e == cudaSuccess ? DBP_OK : fail_cuda("launch", e); }

// Programmatic dependent launch: a kernel launched with launch_chained may become resident while
// the kernel before it in the stream is still draining; it must call chain_wait() before it
// touches global memory (the wait returns once the earlier kernel has completed and its writes
// are visible), and chain_release() lets the kernel after it do the same. Both are no-ops for a
// kernel launched the ordinary way.
#ifdef __CUDACC__
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                  Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    note_launch();
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
#endif

}  // namespace dbp
