// C ABI entry points (see include/dbp.h): argument checks, workspace, kernel sequencing.
#include <new>

#include "dbp_internal.cuh"

#include <atomic>
#include <cstdlib>
#include <cstdio>

namespace dbp {

namespace {
thread_local char g_last_error[192] = "";
std::atomic<long long> g_launches{0};
}

void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

int fail_cuda(const char *what, cudaError_t e) {
    std::snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, cudaGetErrorString(e));
    return DBP_ECUDA;
}

int ws_reserve(dbp_ctx *ctx, Workspace &w, size_t bytes) {
    if (bytes <= w.bytes) return DBP_OK;
    // the stream may still be using the old block
    if (w.ptr) {
        if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return DBP_ECUDA;
        if (ctx->aux && cudaStreamSynchronize(ctx->aux) != cudaSuccess) return DBP_ECUDA;
        cudaFree(w.ptr);
        w.ptr = nullptr;
        w.bytes = 0;
    }
    const size_t want = (bytes + (size_t(1) << 20) - 1) & ~((size_t(1) << 20) - 1);
    if (cudaMalloc(&w.ptr, want) != cudaSuccess) {
        cudaGetLastError();
        w.ptr = nullptr;
        return DBP_ENOMEM;
    }
    w.bytes = want;
    return DBP_OK;
}

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

size_t elem_size(int dtype) { return dtype == DBP_F32 ? 4 : 2; }

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// Quantize delta into `sp` (caller's arrays, or the context's internal ones) and into the
// context's dense code buffer, which the product kernels read.
int quantize_for_products(dbp_ctx *ctx, const void *delta, int dtype, long long numel,
                          unsigned long long seed, float scale, const float *delta_in,
                          dbp_sparse *q_out, const float **delta_p, const int8_t **codes,
                          bool want8 = true, long long planes_hw = 0, long long planes_pitch = 0,
                          const void **codes16 = nullptr, const ConvShape *nhwc = nullptr,
                          const void **codes_nhwc = nullptr, const SideJobs &jobs = SideJobs(),
                          int stack_g = 0, const void **codes_stack = nullptr, const uint8_t *mask = nullptr) {
    int rc = DBP_OK;
    dbp_sparse sp;
    sp.bitmap = nullptr; sp.offsets = nullptr; sp.values = nullptr; sp.delta = nullptr; sp.nnz = nullptr;
    sp.numel = numel;
    if (q_out) {
        if (!q_out->bitmap || !q_out->offsets || !q_out->values || !q_out->delta || !q_out->nnz) return DBP_EINVAL;
        if (!aligned16(q_out->bitmap) || !aligned16(q_out->offsets) || !aligned16(q_out->values)) return DBP_EINVAL;
        q_out->numel = numel;
        sp = *q_out;
    }
    const int k = ctx->code_set;
    if ((rc = ws_reserve(ctx, ctx->dense_codes[k], static_cast<size_t>(numel) + 16))) return rc;
    int8_t *dense = static_cast<int8_t *>(ctx->dense_codes[k].ptr);
    // The set's previous readers (an earlier call's dW kernels on the second stream) must be done before its step
    // size and its codes are written again. The wait stands in front of the statistics kernel, where the stream
    // already holds the previous call's fork event: stream operations between two kernels stop their programmatic
    // overlap, so they are kept at one boundary per call.
    if (ctx->set_busy[k]) {
        if (cudaStreamWaitEvent(ctx->stream, ctx->ev_set_free[k], 0) != cudaSuccess) return fail_cuda("waiting for the code buffers");
        ctx->set_busy[k] = false;
    }
    {
        KernelTimer t(ctx, DBP_K_STATISTICS);
        // without a caller's dbp_sparse the step size also goes to the set's own scalar: the product kernels
        // read it there (the context's scalar is overwritten by the next call's statistics)
        rc = launch_statistics(ctx, delta, dtype, numel, scale, delta_in, q_out ? sp.delta : ctx->delta_sets + k,
                               reinterpret_cast<unsigned long long *>(sp.nnz), jobs, mask);
    }
    if (rc) return rc;
    {
        KernelTimer t(ctx, DBP_K_QUANTIZE);
        // the sparse structure is written only for a caller who asked for it; the bf16 planes
        // of the TMA-fed kernels come from the dense kernel (a second pass when both are wanted)
        void *p16 = nullptr;
        if (codes16) {
            const long long planes = numel / planes_hw;
            if ((rc = ws_reserve(ctx, ctx->codes16[k], static_cast<size_t>(planes) * planes_pitch * 2 + 1024))) return rc;
            p16 = ctx->codes16[k].ptr;
            *codes16 = p16;
        }
        void *pn = nullptr;
        if (nhwc) {
            if ((rc = ws_reserve(ctx, ctx->codes_nhwc[k], static_cast<size_t>(numel) * 2 + 1024))) return rc;
            pn = ctx->codes_nhwc[k].ptr;
            *codes_nhwc = pn;
        }
        void *ps = nullptr;
        if (nhwc && stack_g > 0 && codes_stack) {
            // tall images of stack_g images each: (H + 1) W rows per image
            const size_t rows = static_cast<size_t>(nhwc->B) * (nhwc->H + 1) * nhwc->W;
            if ((rc = ws_reserve(ctx, ctx->codes_stack[k], rows * nhwc->Cout * 2 + 1024))) return rc;
            ps = ctx->codes_stack[k].ptr;
            *codes_stack = ps;
        }
        if (q_out) {
            rc = launch_quantize(ctx, delta, dtype, numel, seed, &ctx->state->delta, sp.bitmap, sp.offsets,
                                 sp.values, dense, reinterpret_cast<unsigned long long *>(sp.nnz));
            if (!rc && p16)
                rc = launch_quantize_dense(ctx, delta, dtype, numel, seed, &ctx->state->delta, nullptr, p16,
                                           planes_hw, planes_pitch, false);
            if (!rc && pn)
                rc = launch_quantize_nhwc(ctx, delta, dtype, nhwc->B, nhwc->Cout, nhwc->H * nhwc->W, seed,
                                          &ctx->state->delta, pn, nullptr, false, ps, static_cast<int>(nhwc->W), stack_g);
        } else if (pn) {
            rc = launch_quantize_nhwc(ctx, delta, dtype, nhwc->B, nhwc->Cout, nhwc->H * nhwc->W, seed,
                                      &ctx->state->delta, pn, want8 ? dense : nullptr, true, ps, static_cast<int>(nhwc->W), stack_g, mask);
        } else {
            rc = launch_quantize_dense(ctx, delta, dtype, numel, seed, &ctx->state->delta, want8 ? dense : nullptr,
                                       p16, planes_hw, planes_pitch, true);
        }
    }
    if (rc) return rc;
    *delta_p = q_out ? &ctx->state->delta : ctx->delta_sets + k;
    if (q_out && cudaMemcpyAsync(ctx->delta_sets + k, &ctx->state->delta, sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream) != cudaSuccess)
        return fail_cuda("copying the step size");
    if (q_out) *delta_p = ctx->delta_sets + k;
    *codes = dense;
    return DBP_OK;
}

int conv_backward_impl(dbp_ctx *ctx, const void *delta, const void *X, const void *W, int io,
                       const ConvShape &s, unsigned long long seed, float scale,
                       const float *delta_in, dbp_sparse *q_out, float *dW, void *dX, float *db,
                       unsigned flags) {
    if (!ctx || !delta) return DBP_EINVAL;
    // a ReLU mask set for this call: consumed here whatever happens next
    const uint8_t *mask = ctx->next_mask;
    ctx->next_mask = nullptr;
    if (io != DBP_F32 && io != DBP_BF16) return DBP_EINVAL;
    if (s.B <= 0 || s.Cin <= 0 || s.Cout <= 0 || s.H <= 0 || s.W <= 0) return DBP_EINVAL;
    if (s.B > 65535 * 32 || s.Cin > (1 << 20) || s.Cout > (1 << 20) || s.H > 4096 || s.W > 4096) return DBP_EINVAL;
    if (!(scale > 0.f) && !delta_in) return DBP_EINVAL;
    if ((dW && !X) || (dX && !W)) return DBP_EINVAL;
    if (!aligned16(delta) || !aligned16(X) || !aligned16(W) || !aligned16(dW) || !aligned16(dX)) return DBP_EINVAL;
    if ((flags & DBP_FORCE_SPARSE) && (flags & DBP_FORCE_DENSE)) return DBP_EINVAL;
    // 3x3 on the tensor cores: both products, or (fp32, any Cin: a network's first layer) the weight gradient alone
    const bool t3_full = tc3_tma_supported(s, io);
    const bool t3_dw_only = !t3_full && dW && !dX && tc3_tma_dw_supported(s, io);
    const bool can_dense = tc_supported(s, io) || t3_full || t3_dw_only;
    if ((flags & DBP_FORCE_DENSE) && !can_dense) return DBP_EUNSUPPORTED;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    const long long numel = s.B * s.Cout * s.H * s.W;
    const float *delta_p = nullptr;
    const int8_t *codes = nullptr;
    if (mask && io != DBP_F32) return DBP_EUNSUPPORTED;
    // small fp32 layers with one position per image (linear layers): two chained launches
    // Masks are read four bytes at a time where they are folded into a kernel's loads. One that does not start on
    // a 4-byte boundary is applied by the ReLU-derivative kernel here and now, and the call goes on without it.
    if (mask != nullptr && (reinterpret_cast<uintptr_t>(mask) & 3) != 0) {
        const long long n0 = numel;
        if (ctx->aux_pending) {
            const int jr = dbp_join(ctx);
            if (jr) return jr;
        }
        const int wr = ws_reserve(ctx, ctx->dz_tmp, static_cast<size_t>(n0) * sizeof(float));
        if (wr) return wr;
        KernelTimer t(ctx, DBP_K_GLUE);
        const int gr = launch_relu_backward(ctx, static_cast<const float *>(delta), mask, static_cast<float *>(ctx->dz_tmp.ptr), n0);
        if (gr) return gr;
        delta = ctx->dz_tmp.ptr;
        mask = nullptr;
    }
    const bool mask_vec = true;
    if (io == DBP_F32 && s.k == 1 && s.H == 1 && s.W == 1 && !q_out && (dW || dX) && (!db || dW) && mask_vec &&
        !(flags & (DBP_FORCE_SPARSE | DBP_FORCE_DENSE)) && small_linear_fits(ctx, s.B, s.Cout, s.Cin, dW != nullptr, dX != nullptr)) {
        if (ctx->aux_pending) {
            const int jr = dbp_join(ctx);
            if (jr) return jr;
        }
        // a *_host call: X is still on its way up on another stream, and dX is read back after an event
        if (dW && ctx->hook_before_dw && cudaStreamWaitEvent(ctx->stream, ctx->hook_before_dw, 0) != cudaSuccess) return DBP_ECUDA;
        int rc;
        {
            KernelTimer t(ctx, DBP_K_FUSED);
            rc = launch_small_linear(ctx, static_cast<const float *>(delta), static_cast<const float *>(X),
                                     static_cast<const float *>(W), s.B, s.Cout, s.Cin, seed, scale, delta_in, dW,
                                     static_cast<float *>(dX), db, ctx->delta_sets ? ctx->delta_sets + ctx->code_set : nullptr, mask);
        }
        if (!rc && ctx->hook_after_dx && cudaEventRecord(ctx->hook_after_dx, ctx->stream) != cudaSuccess) return DBP_ECUDA;
        return rc;
    }
    // While the stream is being captured into a CUDA graph the density read-back is left alone
    // (an event recorded inside a capture cannot be queried): the choice of path is the one the
    // last eager call would have made, and it is frozen into the graph.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(ctx->stream, &cap) != cudaSuccess) return DBP_ECUDA;
    const bool capturing = cap != cudaStreamCaptureStatusNone;
    // pick up the density of the last finished quantization, if its read-back has landed
    // The estimate that decides is the density last measured on a layer of THIS shape (1.0, i.e. dense, until
    // one has been read back): a layer's own sparsity level picks its path, not its neighbour's.
    const unsigned long long shape_key =
        ((((((static_cast<unsigned long long>(s.B) * 1000003ull + s.Cin) * 1000003ull + s.Cout) * 1000003ull + s.H) * 1000003ull + s.W) * 8ull +
          s.k) * 2ull + io);
    if (!capturing && ctx->nnz_pending && cudaEventQuery(ctx->nnz_event) == cudaSuccess) {
        const float dns = static_cast<float>(static_cast<double>(*ctx->nnz_host) / static_cast<double>(ctx->nnz_host_numel));
        bool found = false;
        for (auto &e : ctx->densities)
            if (e.key == ctx->nnz_host_key) { e.density = dns; found = true; }
        if (!found) ctx->densities.push_back({ctx->nnz_host_key, dns});
        ctx->nnz_pending = false;
    }
    cudaGetLastError();   // cudaErrorNotReady from the query is not an error
    float density_estimate = 1.0f;
    for (const auto &e : ctx->densities)
        if (e.key == shape_key) density_estimate = e.density;
    const bool dense = can_dense && !(flags & DBP_FORCE_SPARSE) &&
                       ((flags & DBP_FORCE_DENSE) || ctx->crossover <= 0.f || density_estimate > ctx->crossover);
    // which dense kernels run: the TMA-fed ones read bf16 code planes, the others int8 codes
    const bool dx_tma = dense && dX && tma_dx_supported(s, io);
    const bool dw_tma = dense && dW && tma_dw_supported(s, io);
    const bool any_tma = dx_tma || dw_tma;
    // a call that does not itself fork its dW first orders the earlier calls' outstanding dW work into the
    // stream: it may use the workspaces that work is still using
    if (ctx->aux_pending && !(dense && dX && dW)) {
        const int jr = dbp_join(ctx);
        if (jr) return jr;
    }
    // 3x3 layers: the TMA-fed kernels read the codes position-major
    const bool t3 = dense && (dX || dW) && (t3_full || t3_dw_only);
    // fp32 3x3 layers on the tensor-core kernels apply the mask while they read delta_a (statistics and the
    // position-major quantizer); with a caller's sparse structure, or on any other path, delta_z is made first
    const bool fold3 = mask && mask_vec && io == DBP_F32 && !q_out && t3;
    const uint8_t *mask_q = fold3 ? mask : nullptr;
    if (mask && !fold3) {      // every other path reads delta_z from memory: make it
        const int wr = ws_reserve(ctx, ctx->dz_tmp, static_cast<size_t>(numel) * sizeof(float));
        if (wr) return wr;
        KernelTimer t(ctx, DBP_K_GLUE);
        const int gr = launch_relu_backward(ctx, static_cast<const float *>(delta), mask, static_cast<float *>(ctx->dz_tmp.ptr), numel);
        if (gr) return gr;
        delta = ctx->dz_tmp.ptr;
    }
    const bool need8 = !dense || db || (!t3 && ((dX && !dx_tma) || (dW && !dw_tma)));
    const void *codes16 = nullptr, *codes_n = nullptr;
    // what the statistics kernel does on the side: the TMA-fed 1x1 dW kernel adds its partial sums into dW, so dW
    // is cleared; the 3x3 dX kernel reads the weights tap by tap, so they are re-laid
    SideJobs jobs;
    if (dw_tma) { jobs.zero = dW; jobs.zero_bytes = sizeof(float) * static_cast<size_t>(s.Cout) * s.Cin; }
    const bool w_side = t3 && dX && scale > 0.f;
    if (w_side) {
        const int taps = io == DBP_F32 ? 18 : 9;
        const int wr = ws_reserve(ctx, ctx->w_taps, sizeof(__nv_bfloat16) * static_cast<size_t>(s.Cout) * s.Cin * taps);
        if (wr) return wr;
        jobs.w_src = W; jobs.w_dst = ctx->w_taps.ptr; jobs.w_f32 = io == DBP_F32; jobs.Cout = s.Cout; jobs.Cin = s.Cin;
    }
    // a stride-2 layer run on phase images: W is a workspace for the phase weights that nobody has written yet.
    // The re-laying side job makes its tap-major copy straight from the layer's own weights; any other path reads
    // the phase weights themselves, which are made here
    if (ctx->phase_w_src != nullptr && dX) {
        if (w_side && ctx->phase_cin > 0 && s.Cin == 4ll * ctx->phase_cin) {
            jobs.w_src = ctx->phase_w_src;
            jobs.phase_cin = ctx->phase_cin;
        } else {
            KernelTimer t(ctx, DBP_K_GLUE);
            const int pr = launch_phase_weights(ctx, ctx->phase_w_src, const_cast<void *>(W), io, s.Cout, s.Cin / 4);
            if (pr) return pr;
        }
    }
    // tiny planes: the weight-gradient kernel reads the images stacked into tall ones
    const int stack_g = (t3 && dW) ? tc3_stack_images(s, io) : 0;
    const void *codes_st = nullptr;
    int rc = quantize_for_products(ctx, delta, io, numel, seed, scale, delta_in, q_out, &delta_p, &codes, need8,
                                   s.H * s.W, any_tma ? tma_code_pitch(s) : 0, any_tma ? &codes16 : nullptr,
                                   t3 ? &s : nullptr, t3 ? &codes_n : nullptr, jobs, stack_g, &codes_st, t3 ? mask_q : nullptr);
    if (rc) return rc;
    // (the density decides nothing while the threshold is 0: no read-back then, one stream operation less)
    if (!capturing && ctx->crossover > 0.f && !ctx->nnz_pending && ctx->nnz_host && ctx->nnz_event) {
        ctx->nnz_host_numel = numel;
        ctx->nnz_host_key = shape_key;
        if (cudaMemcpyAsync(ctx->nnz_host, &ctx->state->nnz, sizeof(unsigned long long), cudaMemcpyDeviceToHost,
                            ctx->stream) == cudaSuccess &&
            cudaEventRecord(ctx->nnz_event, ctx->stream) == cudaSuccess)
            ctx->nnz_pending = true;
    }
    if (dense) {
        // dX and dW read the same codes and nothing of each other: with both asked for, dW goes to the
        // context's second stream, so that its CTAs start as SMs come free instead of after the last dX CTA
        const bool forked = dX && dW && ctx->aux != nullptr;
        // (forking after the dX kernel instead, which would keep the quantizer -> dX boundary free of stream
        // operations, measured slower: dW then starts a kernel later and meets the next layer's dX)
        if (forked && (cudaEventRecord(ctx->ev_fork, ctx->stream) != cudaSuccess ||
                       cudaStreamWaitEvent(ctx->aux, ctx->ev_fork, 0) != cudaSuccess))
            return fail_cuda("forking the dW stream");
        if (dX) {
            KernelTimer t(ctx, DBP_K_DX_DENSE);
            const bool dx_bf16 = (io == DBP_BF16) && !(flags & DBP_DX_F32);
            rc = dx_tma ? launch_tma_dx(ctx, codes16, W, delta_p, s, dX, dx_bf16, &ctx->state->tc_timeout)
                 : t3   ? launch_tc3_tma_dx(ctx, codes_n, W, io, delta_p, s, dX, dx_bf16, &ctx->state->tc_timeout, w_side)
                        : launch_tc_dx(ctx, codes, W, delta_p, s, dX, dx_bf16, &ctx->state->tc_timeout);
            if (rc) return rc;
        }
        if (ctx->hook_after_dx && cudaEventRecord(ctx->hook_after_dx, ctx->stream) != cudaSuccess) return DBP_ECUDA;
        cudaStream_t caller = ctx->stream;
        if (forked) ctx->stream = ctx->aux;          // the dW launchers enqueue on the context's stream
        if (dW && ctx->hook_before_dw && cudaStreamWaitEvent(ctx->stream, ctx->hook_before_dw, 0) != cudaSuccess) rc = DBP_ECUDA;
        if (dW && !rc) {
            KernelTimer t(ctx, DBP_K_DW_DENSE);
            rc = dw_tma ? launch_tma_dw(ctx, codes16, X, delta_p, s, dW, &ctx->state->tc_timeout)
                 : (t3 && stack_g > 0)
                     ? launch_tc3_tma_dw(ctx, codes_st, X, io, delta_p,
                                         ConvShape{s.B / stack_g, s.Cin, s.Cout, static_cast<long long>(stack_g) * (s.H + 1), s.W, 3}, dW,
                                         &ctx->state->tc_timeout, stack_g, static_cast<int>(s.H))
                 : t3   ? launch_tc3_tma_dw(ctx, codes_n, X, io, delta_p, s, dW, &ctx->state->tc_timeout)
                        : launch_tc_dw(ctx, codes, X, delta_p, s, dW, &ctx->state->tc_timeout);
        }
        ctx->stream = caller;
        if (forked) {
            // the set's buffers are free once the dW kernels are done; with DBP_DW_ASYNC the caller's stream is
            // ordered after them only by the next user of the set, by dbp_join or by a synchronising call
            const int k = ctx->code_set;
            if (cudaEventRecord(ctx->ev_set_free[k], ctx->aux) != cudaSuccess) return fail_cuda("recording the end of dW");
            if ((flags & DBP_DW_ASYNC) && !rc) {
                ctx->set_busy[k] = true;
                ctx->aux_pending = true;
                ctx->code_set = k ^ 1;
            } else if (cudaStreamWaitEvent(caller, ctx->ev_set_free[k], 0) != cudaSuccess) {
                return fail_cuda("joining the dW stream");
            }
        }
        if (rc) return rc;
        if (db) {
            KernelTimer t(ctx, DBP_K_DB);
            rc = launch_bias_grad(ctx, codes, delta_p, s, db);
            if (rc) return rc;
        }
        return DBP_OK;
    }
    if (dX) {
        const size_t wb = sizeof(float) * static_cast<size_t>(s.Cout) * s.Cin * s.k * s.k;
        if ((rc = ws_reserve(ctx, ctx->w_taps, wb))) return rc;
        void *wt = ctx->w_taps.ptr;
        const bool dx_bf16 = (io == DBP_BF16) && !(flags & DBP_DX_F32);
        // streamed kernel: weight rows must be 16-byte multiples; otherwise the generic one
        const bool streamed = s.k != 5 && (s.Cin * static_cast<long long>(elem_size(io))) % 16 == 0;
        {
            KernelTimer t(ctx, DBP_K_WEIGHT_TAPS);
            rc = launch_weight_taps(ctx, W, io, s, wt, !streamed);
        }
        if (rc) return rc;
        {
            KernelTimer t(ctx, DBP_K_DX);
            rc = streamed ? launch_conv_dx_streamed(ctx, codes, wt, io, delta_p, s, dX, dx_bf16)
                          : launch_conv_dx(ctx, codes, static_cast<const float *>(wt), delta_p, s, dX, dx_bf16);
        }
        if (rc) return rc;
    }
    if (ctx->hook_after_dx && cudaEventRecord(ctx->hook_after_dx, ctx->stream) != cudaSuccess) return DBP_ECUDA;
    if (dW && ctx->hook_before_dw && cudaStreamWaitEvent(ctx->stream, ctx->hook_before_dw, 0) != cudaSuccess) return DBP_ECUDA;
    if (dW) {
        KernelTimer t(ctx, DBP_K_DW);
        rc = s.k == 5 ? DBP_EUNSUPPORTED : launch_conv_dw_streamed(ctx, codes, X, io, delta_p, s, dW);
        if (rc == DBP_EUNSUPPORTED) rc = launch_conv_dw(ctx, codes, X, io, delta_p, s, dW);
        if (rc) return rc;
    }
    if (db) {
        KernelTimer t(ctx, DBP_K_DB);
        rc = launch_bias_grad(ctx, codes, delta_p, s, db);
        if (rc) return rc;
    }
    return DBP_OK;
}

// A stride-2 layer (k = 1 or 3, pad (k-1)/2, even H and W) as the stride-1 layer on the phase images of X
// (strided_conv.cu): delta is that layer's own gradient [B][Cout][H/2][W/2] and is quantized as it is; X, W, dX
// and dW pass through layout kernels on the context's stream. The weight-gradient kernels of such a call are
// always joined before it returns (the workspaces they read are reused by the next strided call).
int conv_backward_stride2(dbp_ctx *ctx, const void *delta, const void *X, const void *W, int io, const ConvShape &s,
                          unsigned long long seed, float scale, const float *delta_in, dbp_sparse *q_out, float *dW,
                          void *dX, float *db, unsigned flags) {
    if (!ctx || !delta) return DBP_EINVAL;
    const uint8_t *mask = ctx->next_mask;
    ctx->next_mask = nullptr;
    if (io != DBP_F32 && io != DBP_BF16) return DBP_EINVAL;
    if (s.B <= 0 || s.Cin <= 0 || s.Cout <= 0 || s.H <= 0 || s.W <= 0 || s.H > 8192 || s.W > 8192) return DBP_EINVAL;
    if ((s.H & 1) || (s.W & 1)) return DBP_EUNSUPPORTED;
    if (s.B * s.Cin * s.H * (s.W / 2) >= (1ll << 31)) return DBP_EUNSUPPORTED;      // the layout kernels index in 32 bits
    if ((dW && !X) || (dX && !W)) return DBP_EINVAL;
    if (!aligned16(X) || !aligned16(W) || !aligned16(dW) || !aligned16(dX)) return DBP_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    const int phases = s.k == 1 ? 1 : 4;
    const int Ho = static_cast<int>(s.H / 2), Wo = static_cast<int>(s.W / 2);
    const ConvShape in{s.B, s.Cin * phases, s.Cout, Ho, Wo, s.k};
    const size_t es = elem_size(io);
    const bool dx_f32 = io == DBP_F32 || (flags & DBP_DX_F32);
    const size_t nxp = static_cast<size_t>(in.B) * in.Cin * Ho * Wo, nwp = static_cast<size_t>(in.Cout) * in.Cin * s.k * s.k;
    int rc;
    if (dW && (rc = ws_reserve(ctx, ctx->s2_x, nxp * es))) return rc;
    if (dX && (rc = ws_reserve(ctx, ctx->s2_dx, nxp * (dx_f32 ? 4 : 2)))) return rc;
    if (dX && s.k == 3 && (rc = ws_reserve(ctx, ctx->s2_w, nwp * es))) return rc;
    if (dW && s.k == 3 && (rc = ws_reserve(ctx, ctx->s2_dw, nwp * sizeof(float)))) return rc;
    // a *_host call: X is still on its way up on another stream, and dX is read back after an event
    cudaEvent_t after_dx = ctx->hook_after_dx;
    ctx->hook_after_dx = nullptr;
    if (dW) {
        if (ctx->hook_before_dw && cudaStreamWaitEvent(ctx->stream, ctx->hook_before_dw, 0) != cudaSuccess) return DBP_ECUDA;
        ctx->hook_before_dw = nullptr;
        KernelTimer t(ctx, DBP_K_GLUE);
        if ((rc = launch_phases_of(ctx, X, ctx->s2_x.ptr, io, s.B, s.Cin, static_cast<int>(s.H), static_cast<int>(s.W), phases))) return rc;
    }
    ctx->next_mask = mask;
    ctx->phase_cin = s.k == 3 ? static_cast<int>(s.Cin) : 0;      // the 3x3 tensor-core kernels skip the taps that are zero by construction
    ctx->phase_dw_out = (s.k == 3 && dW) ? dW : nullptr;
    ctx->phase_w_src = (s.k == 3 && dX) ? W : nullptr;            // the phase weights are made inside, in the form the path wants
    ctx->phase_dw_done = false;
    rc = conv_backward_impl(ctx, delta, dW ? ctx->s2_x.ptr : nullptr, dX ? (s.k == 3 ? ctx->s2_w.ptr : W) : nullptr, io, in,
                            seed, scale, delta_in, q_out,
                            dW ? (s.k == 3 ? static_cast<float *>(ctx->s2_dw.ptr) : dW) : nullptr,
                            dX ? ctx->s2_dx.ptr : nullptr, db, flags & ~DBP_DW_ASYNC);
    ctx->phase_cin = 0;
    ctx->phase_dw_out = nullptr;
    ctx->phase_w_src = nullptr;
    if (rc) return rc;
    if (dX) {
        KernelTimer t(ctx, DBP_K_GLUE);
        if ((rc = launch_from_phases(ctx, ctx->s2_dx.ptr, dX, dx_f32 ? 1 : 0, s.B, s.Cin, static_cast<int>(s.H),
                                     static_cast<int>(s.W), phases)))
            return rc;
        if (after_dx && cudaEventRecord(after_dx, ctx->stream) != cudaSuccess) return DBP_ECUDA;
    }
    if (dW && s.k == 3 && !ctx->phase_dw_done) {
        KernelTimer t(ctx, DBP_K_GLUE);
        if ((rc = launch_strided_dw(ctx, static_cast<const float *>(ctx->s2_dw.ptr), dW, s.Cout, s.Cin))) return rc;
    }
    return DBP_OK;
}

bool conv_form_supported(int k, int stride, int pad) {
    return ((k == 1 || k == 3) && (stride == 1 || stride == 2) && pad == (k - 1) / 2) || (k == 5 && stride == 1 && pad == 2);
}

int conv_backward_any(dbp_ctx *ctx, const void *delta, const void *X, const void *W, int io, const ConvShape &s,
                      int stride, unsigned long long seed, float scale, const float *delta_in, dbp_sparse *q_out,
                      float *dW, void *dX, float *db, unsigned flags) {
    return stride == 2 ? conv_backward_stride2(ctx, delta, X, W, io, s, seed, scale, delta_in, q_out, dW, dX, db, flags)
                       : conv_backward_impl(ctx, delta, X, W, io, s, seed, scale, delta_in, q_out, dW, dX, db, flags);
}

}  // namespace
}  // namespace dbp

using namespace dbp;

extern "C" {

int dbp_create(dbp_ctx **out, int device, void *cuda_stream) {
    if (!out) return DBP_EINVAL;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        cudaGetLastError();
        return DBP_ECUDA;
    }
    DeviceGuard guard(device);
    if (!guard.ok) return DBP_ECUDA;
    dbp_ctx *ctx = new (std::nothrow) dbp_ctx();
    if (!ctx) return DBP_ENOMEM;
    ctx->device = device;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) == cudaSuccess) ctx->sm_count = prop.multiProcessorCount;
    ctx->partial_blocks = ctx->sm_count * 8;
    if (cudaMalloc(&ctx->wait_stats, sizeof(unsigned long long) * DBP_WAIT_SLOTS) != cudaSuccess ||
        cudaMemset(ctx->wait_stats, 0, sizeof(unsigned long long) * DBP_WAIT_SLOTS) != cudaSuccess ||
        cudaMalloc(&ctx->state, sizeof(DeviceState)) != cudaSuccess ||
        cudaMalloc(&ctx->partials, sizeof(double) * 2 * ctx->partial_blocks) != cudaSuccess ||
        cudaMemset(ctx->state, 0, sizeof(DeviceState)) != cudaSuccess) {
        cudaGetLastError();
        dbp_destroy(ctx);
        return DBP_ENOMEM;
    }
    if (cudaStreamCreateWithFlags(&ctx->aux, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_set_free[0], cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_set_free[1], cudaEventDisableTiming) != cudaSuccess ||
        cudaMalloc(&ctx->delta_sets, 2 * sizeof(float)) != cudaSuccess ||
        cudaMallocHost(&ctx->nnz_host, sizeof(unsigned long long)) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->nnz_event, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        dbp_destroy(ctx);
        return DBP_ENOMEM;
    }
    *out = ctx;
    return DBP_OK;
}

const char *dbp_last_error(void) { return g_last_error; }

long long dbp_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int dbp_measure_fma_peak(dbp_ctx *ctx, double *tflops) {
    if (!ctx || !tflops) return DBP_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    return measure_fma_peak(ctx, tflops);
}

int dbp_join(dbp_ctx *ctx) {
    if (!ctx) return DBP_EINVAL;
    if (!ctx->aux_pending) return DBP_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    // everything enqueued on the second stream so far: one event, and the caller's stream waits for it
    if (cudaEventRecord(ctx->ev_join, ctx->aux) != cudaSuccess || cudaStreamWaitEvent(ctx->stream, ctx->ev_join, 0) != cudaSuccess)
        return fail_cuda("joining the dW stream");
    ctx->aux_pending = false;
    ctx->set_busy[0] = ctx->set_busy[1] = false;
    return DBP_OK;
}

int dbp_set_crossover(dbp_ctx *ctx, float crossover) {
    if (!ctx || crossover != crossover) return DBP_EINVAL;
    ctx->crossover = crossover;
    return DBP_OK;
}

int dbp_destroy(dbp_ctx *ctx) {
    if (!ctx) return DBP_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    if (ctx->aux) cudaStreamSynchronize(ctx->aux);
    Workspace *all[] = {&ctx->dense_codes[0], &ctx->dense_codes[1], &ctx->codes16[0], &ctx->codes16[1],
                        &ctx->codes_nhwc[0], &ctx->codes_nhwc[1], &ctx->codes_stack[0], &ctx->codes_stack[1], &ctx->dz_tmp, &ctx->s2_x, &ctx->s2_w, &ctx->s2_dx, &ctx->s2_dw, &ctx->dw_acc, &ctx->x_padded, &ctx->w_taps, &ctx->sp_bitmap, &ctx->sp_offsets, &ctx->sp_values,
                        &ctx->tc_partials};
    for (Workspace *w : all) if (w->ptr) cudaFree(w->ptr);
    for (Workspace &w : ctx->io) if (w.ptr) cudaFree(w.ptr);
    for (ProfSlot &p : ctx->prof) { cudaEventDestroy(p.begin); cudaEventDestroy(p.end); }
    if (ctx->nnz_host) cudaFreeHost(ctx->nnz_host);
    if (ctx->nnz_event) cudaEventDestroy(ctx->nnz_event);
    if (ctx->aux) { cudaStreamSynchronize(ctx->aux); cudaStreamDestroy(ctx->aux); }
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    for (cudaEvent_t e : ctx->ev_set_free) if (e) cudaEventDestroy(e);
    if (ctx->delta_sets) cudaFree(ctx->delta_sets);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->copy_in) { cudaStreamSynchronize(ctx->copy_in); cudaStreamDestroy(ctx->copy_in); }
    if (ctx->copy_out) { cudaStreamSynchronize(ctx->copy_out); cudaStreamDestroy(ctx->copy_out); }
    if (ctx->ev_x_up) cudaEventDestroy(ctx->ev_x_up);
    if (ctx->ev_dx_done) cudaEventDestroy(ctx->ev_dx_done);
    if (ctx->state) cudaFree(ctx->state);
    if (ctx->wait_stats) cudaFree(ctx->wait_stats);
    if (ctx->partials) cudaFree(ctx->partials);
    delete ctx;
    return DBP_OK;
}

int dbp_set_stream(dbp_ctx *ctx, void *cuda_stream) {
    if (!ctx) return DBP_EINVAL;
    if (int jr = dbp_join(ctx)) return jr;           // outstanding dW work is ordered into the old stream
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    return DBP_OK;
}

const char *dbp_status_string(int status) {
    switch (status) {
        case DBP_OK: return "ok";
        case DBP_EINVAL: return "invalid argument";
        case DBP_EUNSUPPORTED: return "unsupported configuration";
        case DBP_ECUDA: return "CUDA runtime error";
        case DBP_ENOMEM: return "out of memory";
        case DBP_ENONFINITE: return "non-finite value in delta";
        case DBP_ESATURATED: return "codes clipped to +-127";
        case DBP_ECAPACITY: return "buffer too small";
        case DBP_ETIMEOUT: return "bounded device wait expired";
        default: return "unknown status";
    }
}

int dbp_last_device_status(dbp_ctx *ctx, int *status, long long *saturated) {
    if (!ctx) return DBP_EINVAL;
    if (int jr = dbp_join(ctx)) return jr;
    DeviceGuard guard(ctx->device);
    DeviceState h;
    if (cudaMemcpyAsync(&h, ctx->state, sizeof(h), cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess ||
        cudaStreamSynchronize(ctx->stream) != cudaSuccess)
        return DBP_ECUDA;
    if (status)
        *status = h.tc_timeout ? DBP_ETIMEOUT : h.nonfinite ? DBP_ENONFINITE : (h.saturated ? DBP_ESATURATED : DBP_OK);
    if (saturated) *saturated = static_cast<long long>(h.saturated);
    if (h.tc_timeout) ctx->dw_acc_clean = false;        // a kernel gave up half way: its scratch may hold partial sums
    if (h.nonfinite || h.saturated || h.tc_timeout) {
        if (cudaMemsetAsync(&ctx->state->nonfinite, 0, sizeof(int), ctx->stream) != cudaSuccess ||
            cudaMemsetAsync(&ctx->state->tc_timeout, 0, sizeof(int), ctx->stream) != cudaSuccess ||
            cudaMemsetAsync(&ctx->state->saturated, 0, sizeof(unsigned long long), ctx->stream) != cudaSuccess)
            return DBP_ECUDA;
    }
    return DBP_OK;
}

int dbp_selftest_bounded_wait(dbp_ctx *ctx, long long cycles) {
    if (!ctx || cycles < 0 || cycles > 100000000ll) return DBP_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    return launch_bounded_wait_selftest(ctx, cycles);
}

int dbp_wait_stats(dbp_ctx *ctx, unsigned long long *out, int reset) {
    if (!ctx || !out) return DBP_EINVAL;
    if (int jr = dbp_join(ctx)) return jr;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    if (cudaMemcpyAsync(out, ctx->wait_stats, sizeof(unsigned long long) * DBP_WAIT_SLOTS, cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess ||
        cudaStreamSynchronize(ctx->stream) != cudaSuccess)
        return fail_cuda("reading the wait counters");
    if (reset && cudaMemsetAsync(ctx->wait_stats, 0, sizeof(unsigned long long) * DBP_WAIT_SLOTS, ctx->stream) != cudaSuccess)
        return fail_cuda("clearing the wait counters");
    return DBP_OK;
}

int dbp_profile_enable(dbp_ctx *ctx, int on) {
    if (!ctx) return DBP_EINVAL;
    ctx->profiling = on != 0;
    return DBP_OK;
}

int dbp_profile_select(dbp_ctx *ctx, unsigned kind_mask) {
    if (!ctx) return DBP_EINVAL;
    ctx->prof_mask = kind_mask;
    return DBP_OK;
}

int dbp_profile_read(dbp_ctx *ctx, int kind, double *milliseconds, long long *launches) {
    if (!ctx || kind < 0 || kind >= DBP_K_COUNT) return DBP_EINVAL;
    if (int jr = dbp_join(ctx)) return jr;
    DeviceGuard guard(ctx->device);
    if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return DBP_ECUDA;
    for (size_t i = 0; i < ctx->prof_used; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, ctx->prof[i].begin, ctx->prof[i].end) != cudaSuccess) {
            cudaGetLastError();
            continue;
        }
        ctx->prof_ms[ctx->prof[i].kind] += ms;
        ctx->prof_launches[ctx->prof[i].kind] += 1;
    }
    ctx->prof_used = 0;
    if (milliseconds) *milliseconds = ctx->prof_ms[kind];
    if (launches) *launches = ctx->prof_launches[kind];
    ctx->prof_ms[kind] = 0.0;
    ctx->prof_launches[kind] = 0;
    return DBP_OK;
}

int dbp_sparse_bytes(long long numel, size_t *bitmap_bytes, size_t *offsets_bytes, size_t *values_bytes) {
    if (numel <= 0) return DBP_EINVAL;
    const size_t nseg = (static_cast<size_t>(numel) + kSegment - 1) / kSegment;
    if (bitmap_bytes) *bitmap_bytes = nseg * kWordsPerSegment * sizeof(uint32_t);
    if (offsets_bytes) *offsets_bytes = nseg * kWordsPerSegment * sizeof(uint16_t);
    if (values_bytes) *values_bytes = nseg * kSegment;
    return DBP_OK;
}

int nsd_quantize(dbp_ctx *ctx, const void *delta, int dtype, long long numel, unsigned long long seed,
                 float scale, const float *delta_in, dbp_sparse *out) {
    if (!ctx || !delta || !out || numel <= 0) return DBP_EINVAL;
    if (dtype != DBP_F32 && dtype != DBP_BF16) return DBP_EINVAL;
    if (!(scale > 0.f) && !delta_in) return DBP_EINVAL;
    if (!out->bitmap || !out->offsets || !out->values || !out->delta || !out->nnz) return DBP_EINVAL;
    if (!aligned16(delta) || !aligned16(out->bitmap) || !aligned16(out->offsets) || !aligned16(out->values))
        return DBP_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    out->numel = numel;
    int rc;
    {
        KernelTimer t(ctx, DBP_K_STATISTICS);
        rc = launch_statistics(ctx, delta, dtype, numel, scale, delta_in, out->delta,
                               reinterpret_cast<unsigned long long *>(out->nnz));
    }
    if (rc) return rc;
    KernelTimer t(ctx, DBP_K_QUANTIZE);
    return launch_quantize(ctx, delta, dtype, numel, seed, &ctx->state->delta, out->bitmap, out->offsets,
                           out->values, nullptr, reinterpret_cast<unsigned long long *>(out->nnz));
}

int dbp_last_step(dbp_ctx *ctx, float *delta_out, long long *nnz_out) {
    if (!ctx) return DBP_EINVAL;
    if (int jr = dbp_join(ctx)) return jr;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    DeviceState h;
    if (cudaMemcpyAsync(&h, ctx->state, sizeof(h), cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess ||
        cudaStreamSynchronize(ctx->stream) != cudaSuccess)
        return DBP_ECUDA;
    if (delta_out) *delta_out = h.delta;
    if (nnz_out) *nnz_out = static_cast<long long>(h.nnz);
    return DBP_OK;
}

unsigned long long dbp_layer_seed(unsigned long long seed, int layer) {
    unsigned long long z = seed + (static_cast<unsigned long long>(layer) + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

int nsd_decode_dense(dbp_ctx *ctx, const dbp_sparse *q, int8_t *codes) {
    if (!ctx || !q || !codes || q->numel <= 0 || !q->bitmap || !q->offsets || !q->values) return DBP_EINVAL;
    if (!aligned16(codes)) return DBP_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    KernelTimer t(ctx, DBP_K_DECODE);
    return launch_decode(ctx, q->bitmap, q->offsets, q->values, q->numel, codes);
}

int dithered_linear_backward(dbp_ctx *ctx, const void *delta, const void *X, const void *W, int io,
                             long long B, long long N, long long K, unsigned long long seed, float scale,
                             const float *delta_in, dbp_sparse *q_out, float *dW, void *dX, float *db,
                             unsigned flags) {
    // [B,N] x [N,K]: the 1x1 convolution with one position per image has the same layout
    ConvShape s{B, K, N, 1, 1, 1};
    return conv_backward_impl(ctx, delta, X, W, io, s, seed, scale, delta_in, q_out, dW, dX, db, flags);
}

int dithered_conv_backward(dbp_ctx *ctx, const void *delta, const void *X, const void *W, int io,
                           long long B, long long Cin, long long Cout, long long H, long long Wd, int k,
                           int stride, int pad, unsigned long long seed, float scale,
                           const float *delta_in, dbp_sparse *q_out, float *dW, void *dX, float *db,
                           unsigned flags) {
    if (!conv_form_supported(k, stride, pad)) return DBP_EUNSUPPORTED;
    ConvShape s{B, Cin, Cout, H, Wd, k};
    return conv_backward_any(ctx, delta, X, W, io, s, stride, seed, scale, delta_in, q_out, dW, dX, db, flags);
}

static int host_backward(dbp_ctx *ctx, const void *delta, const void *X, const void *W, int io,
                         const ConvShape &s, unsigned long long seed, float scale, float *dW, void *dX,
                         float *db, unsigned flags, float *delta_out, long long *nnz_out, int stride = 1) {
    if (!ctx || !delta) return DBP_EINVAL;
    if (io != DBP_F32 && io != DBP_BF16) return DBP_EINVAL;
    if (s.B <= 0 || s.Cin <= 0 || s.Cout <= 0 || s.H <= 0 || s.W <= 0) return DBP_EINVAL;
    if ((dW && !X) || (dX && !W)) return DBP_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    const size_t es = elem_size(io);
    const size_t nd = static_cast<size_t>(s.B) * s.Cout * (s.H / stride) * (s.W / stride);   // delta: the layer's output positions
    const size_t nx = static_cast<size_t>(s.B) * s.Cin * s.H * s.W;
    const size_t nw = static_cast<size_t>(s.Cout) * s.Cin * s.k * s.k;
    const size_t dx_es = (io == DBP_BF16 && !(flags & DBP_DX_F32)) ? 2 : 4;
    int rc;
    if ((rc = ws_reserve(ctx, ctx->io[0], nd * es)) || (rc = ws_reserve(ctx, ctx->io[1], X ? nx * es : 16)) ||
        (rc = ws_reserve(ctx, ctx->io[2], W ? nw * es : 16)) || (rc = ws_reserve(ctx, ctx->io[3], dW ? nw * 4 : 16)) ||
        (rc = ws_reserve(ctx, ctx->io[4], dX ? nx * dx_es : 16)) || (rc = ws_reserve(ctx, ctx->io[5], db ? s.Cout * 4 : 16)))
        return rc;
    cudaStream_t st = ctx->stream;
    if (!ctx->copy_in) {
        if (cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_x_up, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_dx_done, cudaEventDisableTiming) != cudaSuccess)
            return DBP_ECUDA;
    }
    // delta and W go up on the context's stream (dX needs only them); X goes up beside them on
    // its own stream and is waited for before the dW kernels; dX comes down on a third stream
    // as soon as its kernel is done, while X is still going up and dW is being computed.
    // Staging buffers are free here: the previous *_host call ended with every stream idle.
    if (cudaMemcpyAsync(ctx->io[0].ptr, delta, nd * es, cudaMemcpyHostToDevice, st) != cudaSuccess) return DBP_ECUDA;
    if (W && cudaMemcpyAsync(ctx->io[2].ptr, W, nw * es, cudaMemcpyHostToDevice, st) != cudaSuccess) return DBP_ECUDA;
    if (X) {
        if (cudaMemcpyAsync(ctx->io[1].ptr, X, nx * es, cudaMemcpyHostToDevice, ctx->copy_in) != cudaSuccess ||
            cudaEventRecord(ctx->ev_x_up, ctx->copy_in) != cudaSuccess)
            return DBP_ECUDA;
        ctx->hook_before_dw = ctx->ev_x_up;
    }
    if (dX) ctx->hook_after_dx = ctx->ev_dx_done;
    rc = conv_backward_any(ctx, ctx->io[0].ptr, X ? ctx->io[1].ptr : nullptr, W ? ctx->io[2].ptr : nullptr, io, s, stride,
                            seed, scale, nullptr, nullptr, dW ? static_cast<float *>(ctx->io[3].ptr) : nullptr,
                            dX ? ctx->io[4].ptr : nullptr, db ? static_cast<float *>(ctx->io[5].ptr) : nullptr,
                            flags & ~DBP_DW_ASYNC);      // the results are copied back right away
    ctx->hook_before_dw = nullptr;
    ctx->hook_after_dx = nullptr;
    if (rc) {
        cudaStreamSynchronize(ctx->copy_in);
        return rc;
    }
    if (dX && (cudaStreamWaitEvent(ctx->copy_out, ctx->ev_dx_done, 0) != cudaSuccess ||
               cudaMemcpyAsync(dX, ctx->io[4].ptr, nx * dx_es, cudaMemcpyDeviceToHost, ctx->copy_out) != cudaSuccess))
        return DBP_ECUDA;
    if (dW && cudaMemcpyAsync(dW, ctx->io[3].ptr, nw * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DBP_ECUDA;
    if (db && cudaMemcpyAsync(db, ctx->io[5].ptr, s.Cout * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DBP_ECUDA;
    DeviceState h;
    if (cudaMemcpyAsync(&h, ctx->state, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DBP_ECUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess || cudaStreamSynchronize(ctx->copy_out) != cudaSuccess ||
        cudaStreamSynchronize(ctx->copy_in) != cudaSuccess)
        return DBP_ECUDA;
    if (delta_out) *delta_out = h.delta;
    if (nnz_out) *nnz_out = static_cast<long long>(h.nnz);
    return DBP_OK;
}

int dithered_linear_backward_host(dbp_ctx *ctx, const void *delta, const void *X, const void *W, int io,
                                  long long B, long long N, long long K, unsigned long long seed,
                                  float scale, float *dW, void *dX, float *db, unsigned flags,
                                  float *delta_out, long long *nnz_out) {
    if (!(scale > 0.f)) return DBP_EINVAL;
    ConvShape s{B, K, N, 1, 1, 1};
    return host_backward(ctx, delta, X, W, io, s, seed, scale, dW, dX, db, flags, delta_out, nnz_out);
}

int dithered_conv_backward_host(dbp_ctx *ctx, const void *delta, const void *X, const void *W, int io,
                                long long B, long long Cin, long long Cout, long long H, long long Wd,
                                int k, int stride, int pad, unsigned long long seed, float scale,
                                float *dW, void *dX, float *db, unsigned flags, float *delta_out,
                                long long *nnz_out) {
    if (!conv_form_supported(k, stride, pad)) return DBP_EUNSUPPORTED;
    if (stride == 2 && ((H & 1) || (Wd & 1))) return DBP_EUNSUPPORTED;
    if (!(scale > 0.f)) return DBP_EINVAL;
    ConvShape s{B, Cin, Cout, H, Wd, k};
    return host_backward(ctx, delta, X, W, io, s, seed, scale, dW, dX, db, flags, delta_out, nnz_out, stride);
}

int dbp_set_relu_mask(dbp_ctx *ctx, const uint8_t *mask) {
    if (!ctx) return DBP_EINVAL;
    ctx->next_mask = mask;
    return DBP_OK;
}

int dbp_relu_backward(dbp_ctx *ctx, const float *delta_a, const uint8_t *mask, float *delta_z, long long numel) {
    if (!ctx || !delta_a || !mask || !delta_z || numel <= 0) return DBP_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    KernelTimer t(ctx, DBP_K_GLUE);
    return launch_relu_backward(ctx, delta_a, mask, delta_z, numel);
}

int dbp_maxpool2x2_backward(dbp_ctx *ctx, const float *g, const int8_t *argmax, float *out, long long planes,
                            long long h, long long w) {
    if (!ctx || !g || !argmax || !out || planes <= 0 || h <= 0 || w <= 0) return DBP_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return DBP_ECUDA;
    KernelTimer t(ctx, DBP_K_GLUE);
    return launch_maxpool_backward(ctx, g, argmax, out, planes, h, w);
}

}  // extern "C"
