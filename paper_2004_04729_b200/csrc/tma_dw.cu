// Weight gradient of 1x1 convolutions on the tensor cores, operands brought in by TMA (Eq. (qdw)):
//   dW[co, ci] = Delta * sum_{b, p} q[b, co, p] * X[b, ci, p]
// The reduction index is the position, which is the contiguous index of both the bf16 code
// planes [b][co][pitch] and the activations [b][ci][HW], so both operands are K-major tiles of
// 64 positions of one image:
//   A = codes [128 co][64 p]   (one or two of them: MA accumulators share the activation tile)
//   B = X     [NT ci][64 p]
// The reduction over (image, 64-position chunk) is split over CTAs; a CTA accumulates its share in
// TMEM, scales it by Delta and has the copy engine add it into dW, which the layer's statistics
// kernel has cleared (the order of these additions, hence the last bits of dW, can differ from run
// to run). Warp 0 issues the copies, warp 1 the MMAs, warps 2-5 drain the accumulators at the end.
// Positions past the end of a plane read as zero.
#include "tc_common.cuh"

namespace dbp {

namespace {

using namespace tc;

constexpr int kATile = 128 * 128;                // 128 rows x 64 bf16
constexpr int kBMax = 256 * 128;
constexpr int kThreadsW = 192;
constexpr int kStageW = 32 * 128;                // one warp's staged 32 x 32 fp32 block

struct DwT {
    const float *delta_p;
    int Cin, Cout, HW;
    int cpi;                      // 64-position chunks per image
    long long nchunks;            // B * cpi
    int ci_tiles, nsplit;
    long long per_split;          // chunks per CTA
    int NT, NTp, MA, stages;      // ci tile, its accumulator stride (multiple of 32), accumulators
    int tmem_cols;
    int *err_flag;
    unsigned long long *stats;    // wait counters (may be null)
};

struct PipeW {
    unsigned long long full[4], empty[4], acc_full;
    unsigned tmem_base;
};

__global__ void __launch_bounds__(kThreadsW, 1)
tma_dw_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_x,
              const __grid_constant__ CUtensorMap map_dw, const DwT p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ PipeW pipe;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages;
    const int stage_bytes = p.MA * kATile + kBMax;

    // my work item: output tile (co group, ci tile) and a range of chunks
    const int split = blockIdx.x % p.nsplit;
    const int tile = blockIdx.x / p.nsplit;
    const int ci0 = (tile % p.ci_tiles) * p.NT;
    const int co0 = (tile / p.ci_tiles) * 128 * p.MA;
    const long long k0 = split * p.per_split;
    const long long k1 = k0 + p.per_split < p.nchunks ? k0 + p.per_split : p.nchunks;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&pipe.full[s], 1);
            mbar_init(&pipe.empty[s], 1);
        }
        mbar_init(&pipe.acc_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_x);
        tma_prefetch_desc(&map_dw);
    }
    if (warp == 1) tmem_alloc(&pipe.tmem_base, p.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = pipe.tmem_base;
    chain_wait();        // from here on the kernel reads what earlier kernels wrote
    chain_release();

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            unsigned parity = 1;
            long long b = k0 / p.cpi;
            int c = static_cast<int>(k0 - b * p.cpi);
            const unsigned bytes = static_cast<unsigned>(p.MA * kATile + p.NT * 128);
            long long waited = 0;
            for (long long k = k0; k < k1; ++k) {
                if (!mbar_wait_timed(&pipe.empty[s], parity, p.err_flag, waited)) break;
                unsigned char *st = smem + s * stage_bytes;
                mbar_expect_tx(&pipe.full[s], bytes);
                for (int a = 0; a < p.MA; ++a)
                    tma_load_3d(st + a * kATile, &map_q, c * 64, co0 + a * 128, static_cast<int>(b), &pipe.full[s]);
                tma_load_3d(st + p.MA * kATile, &map_x, c * 64, ci0, static_cast<int>(b), &pipe.full[s]);
                if (++c == p.cpi) { c = 0; ++b; }
                if (++s == S) { s = 0; parity ^= 1u; }
            }
            report_wait(p.stats, 3, waited);
        }
    } else if (warp == 1) {
        {   // the whole warp runs the loop (uniform control flow and operands); one elected lane issues
            const unsigned idesc = make_idesc(128, p.NT, false, false);
            int s = 0;
            unsigned parity = 0;
            bool ok = true;
            int c = static_cast<int>(k0 % p.cpi);
            long long wf = 0;
            const long long born = clock64();
            for (long long k = k0; k < k1; ++k) {
                ok = __all_sync(0xffffffffu, mbar_wait_timed(&pipe.full[s], parity, p.err_flag, wf));
                if (!ok) break;
                tc_fence_after();
                // the last chunk of a plane may hold fewer than 64 positions: skip the 16-position
                // slices that are entirely zero fill
                const int valid = p.HW - c * 64 < 64 ? p.HW - c * 64 : 64;
                const int nk = (valid + 15) >> 4;
                const unsigned a_addr = smem_u32(smem + s * stage_bytes);
                const unsigned long long bd = make_desc(a_addr + p.MA * kATile, 16, 1024);
                if (elect_one()) {
                    for (int a = 0; a < p.MA; ++a) {
                        const unsigned long long ad = make_desc(a_addr + a * kATile, 16, 1024);
                        for (int kk = 0; kk < nk; ++kk)       // 16 positions = 32 bytes further per MMA
                            mma_bf16(tmem_base + a * p.NTp, ad + 2 * kk, bd + 2 * kk, idesc, (k > k0 || kk > 0) ? 1u : 0u);
                    }
                    mma_commit(&pipe.empty[s]);
                }
                if (++c == p.cpi) c = 0;
                if (++s == S) { s = 0; parity ^= 1u; }
            }
            if (ok && elect_one()) mma_commit(&pipe.acc_full);
            if (lane == 0) {
                report_wait(p.stats, 1, wf);
                report_wait(p.stats, 6, clock64() - born);
                report_wait(p.stats, 7, 1);
            }
        }
    } else {
        // epilogue: TMEM lane = output channel, column = input channel. A warp's 32 x 32 block is scaled by
        // Delta and staged in shared memory as 128-byte rows (16-byte pieces XOR-swizzled by the row, the
        // layout the tensor map describes), then one lane asks the copy engine to add it into dW. The
        // operand ring is free by now: each warp cycles through four 4 KB blocks of it.
        const int q = warp & 3;
        unsigned char *stage0 = smem + (warp - 2) * 4 * kStageW;
        if (k1 > k0 && mbar_wait(&pipe.acc_full, 0, p.err_flag)) {
            tc_fence_after();
            const long long t_epi = clock64();
            const float delta = *p.delta_p;
            int n = 0;
            for (int a = 0; a < p.MA; ++a) {
                const int co_w = co0 + a * 128 + q * 32;                 // first output channel of this warp
#pragma unroll 1
                for (int c0 = 0; c0 < p.NT; c0 += 32, ++n) {
                    unsigned char *stage = stage0 + (n & 3) * kStageW;
                    if (n >= 4) {                                          // the engine must have read the block's last use
                        if (lane == 0) bulk_wait_read_but3();
                        __syncwarp();
                    }
                    unsigned v[32];
                    tmem_ld32(tmem_base + (static_cast<unsigned>(q * 32) << 16) + a * p.NTp + c0, v);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<float4 *>(stage + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                            make_float4(__uint_as_float(v[4 * j]) * delta, __uint_as_float(v[4 * j + 1]) * delta,
                                        __uint_as_float(v[4 * j + 2]) * delta, __uint_as_float(v[4 * j + 3]) * delta);
                    fence_async_proxy();
                    __syncwarp();
                    // rows past Cout and columns past Cin are skipped by the engine
                    if (lane == 0) {
                        if (co_w < p.Cout && ci0 + c0 < p.Cin) tma_reduce_add_2d(&map_dw, ci0 + c0, co_w, stage);
                        bulk_commit();                 // a group per block, issued or not: the wait above counts groups
                    }
                }
            }
            if (lane == 0) bulk_wait_read_all();
            if (threadIdx.x == 64) report_wait(p.stats, 5, clock64() - t_epi);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

}  // namespace

bool tma_dw_supported(const ConvShape &s, int io) {
    const long long HW = s.H * s.W;
    return io == DBP_BF16 && s.k == 1 && s.Cin % 8 == 0 && HW >= 16 && HW < (1ll << 30) &&
           s.B * ((HW + 63) / 64) >= 4;
}

int launch_tma_dw(dbp_ctx *ctx, const void *codes_bf16, const void *X, const float *delta_p,
                  const ConvShape &s, float *dW, int *err_flag) {
    const long long HW = s.H * s.W, pitch = tma_code_pitch(s);
    DwT p{};
    p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout); p.HW = static_cast<int>(HW);
    p.cpi = static_cast<int>((HW + 63) / 64);
    p.nchunks = s.B * p.cpi;
    p.NT = s.Cin >= 256 ? 256 : static_cast<int>((s.Cin + 15) / 16 * 16);
    p.NTp = (p.NT + 31) / 32 * 32;
    p.MA = s.Cout > 128 ? 2 : 1;
    p.stages = p.MA == 2 ? 3 : 4;
    p.tmem_cols = 32;
    while (p.tmem_cols < p.MA * p.NTp) p.tmem_cols *= 2;
    p.ci_tiles = static_cast<int>((s.Cin + p.NT - 1) / p.NT);
    const long long co_tiles = (s.Cout + 128 * p.MA - 1) / (128 * p.MA);
    const long long tiles = co_tiles * p.ci_tiles;
    long long per = 0;
    const long long nsplit = choose_split(tiles, p.nchunks, ctx->sm_count, &per);
    p.nsplit = static_cast<int>(nsplit);
    p.per_split = per;
    p.err_flag = err_flag;
    p.stats = ctx->wait_stats;
    p.delta_p = delta_p;
    int rc = DBP_OK;
    // activations whose planes do not start on 16-byte boundaries are first copied to padded planes
    const void *Xsrc = X;
    long long xpitch = HW;
    if (HW % 8 != 0) {
        xpitch = pitch;
        if ((rc = ws_reserve(ctx, ctx->x_padded, static_cast<size_t>(s.B) * s.Cin * xpitch * 2))) return rc;
        if ((rc = launch_pad_planes(ctx, X, ctx->x_padded.ptr, s.B * s.Cin, 1, static_cast<int>(HW), static_cast<int>(xpitch))))
            return rc;
        Xsrc = ctx->x_padded.ptr;
    }
    CUtensorMap map_q, map_x, map_dw;
    {
        const unsigned long long dims[2] = {static_cast<unsigned long long>(s.Cin), static_cast<unsigned long long>(s.Cout)};
        const unsigned long long str[1] = {static_cast<unsigned long long>(s.Cin) * 4};
        const unsigned box[2] = {32, 32};
        if (!encode_map_f32_sw128(&map_dw, dW, 2, dims, str, box)) return fail_cuda("tensor map of dW");
    }
    {
        const unsigned long long dims[3] = {static_cast<unsigned long long>(HW), static_cast<unsigned long long>(s.Cout),
                                            static_cast<unsigned long long>(s.B)};
        const unsigned long long str[2] = {static_cast<unsigned long long>(pitch) * 2,
                                           static_cast<unsigned long long>(pitch) * 2 * s.Cout};
        const unsigned box[3] = {64, 128, 1};
        if (!encode_map_bf16(&map_q, codes_bf16, 3, dims, str, box)) return DBP_ECUDA;
    }
    {
        const unsigned long long dims[3] = {static_cast<unsigned long long>(HW), static_cast<unsigned long long>(s.Cin),
                                            static_cast<unsigned long long>(s.B)};
        const unsigned long long str[2] = {static_cast<unsigned long long>(xpitch) * 2,
                                           static_cast<unsigned long long>(xpitch) * 2 * s.Cin};
        const unsigned box[3] = {64, static_cast<unsigned>(p.NT), 1};
        if (!encode_map_bf16(&map_x, Xsrc, 3, dims, str, box)) return DBP_ECUDA;
    }
    const size_t smem = static_cast<size_t>(p.stages) * (p.MA * kATile + kBMax) + 1024;       // >= 4 warps x 4 staging blocks
    if (cudaFuncSetAttribute(tma_dw_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return DBP_ECUDA;
    // dW has been cleared by this layer's statistics kernel
    return cuda_ok(launch_chained(tma_dw_kernel, dim3(static_cast<unsigned>(tiles * nsplit)), dim3(kThreadsW), smem,
                                  ctx->stream, map_q, map_x, map_dw, p));
}

}  // namespace dbp

namespace dbp {

namespace {

// Copies planes of H x W bf16 values into rows of Wp >= W values (Wp a multiple of 8), the extra
// columns zero, so that every row of every plane starts on a 16-byte boundary: the copy engine
// cannot address planes whose pitch is not a multiple of 16 bytes.
__global__ void __launch_bounds__(256)
pad_planes_kernel(const unsigned short *__restrict__ in, unsigned short *__restrict__ out, long long planes,
                  int H, int W, int Wp) {
    const int groups_per_row = Wp / 8;
    const long long ngroups = planes * H * groups_per_row;
    chain_wait();
    chain_release();
    for (long long g = blockIdx.x * 256ll + threadIdx.x; g < ngroups; g += gridDim.x * 256ll) {
        const long long row = g / groups_per_row;           // (plane, y)
        const int x0 = static_cast<int>(g - row * groups_per_row) * 8;
        const unsigned short *src = in + row * W + x0;
        unsigned short v[8];
        if ((W & 3) == 0 && x0 + 8 <= W) {          // rows start on 8-byte boundaries: two 8-byte loads
            const uint2 a = __ldg(reinterpret_cast<const uint2 *>(src)), b = __ldg(reinterpret_cast<const uint2 *>(src + 4));
            v[0] = static_cast<unsigned short>(a.x); v[1] = static_cast<unsigned short>(a.x >> 16);
            v[2] = static_cast<unsigned short>(a.y); v[3] = static_cast<unsigned short>(a.y >> 16);
            v[4] = static_cast<unsigned short>(b.x); v[5] = static_cast<unsigned short>(b.x >> 16);
            v[6] = static_cast<unsigned short>(b.y); v[7] = static_cast<unsigned short>(b.y >> 16);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = (x0 + j < W) ? __ldg(src + j) : static_cast<unsigned short>(0);
        }
        uint4 o;
        o.x = v[0] | (static_cast<unsigned>(v[1]) << 16);
        o.y = v[2] | (static_cast<unsigned>(v[3]) << 16);
        o.z = v[4] | (static_cast<unsigned>(v[5]) << 16);
        o.w = v[6] | (static_cast<unsigned>(v[7]) << 16);
        *reinterpret_cast<uint4 *>(out + row * Wp + x0) = o;
    }
}

}  // namespace

int launch_pad_planes(dbp_ctx *ctx, const void *in, void *out, long long planes, int H, int W, int Wp) {
    const long long ngroups = planes * H * (Wp / 8);
    long long blocks = (ngroups + 255) / 256;
    const long long cap = static_cast<long long>(ctx->sm_count) * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return cuda_ok(launch_chained(pad_planes_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, ctx->stream,
                                  static_cast<const unsigned short *>(in), static_cast<unsigned short *>(out), planes, H, W, Wp));
}

}  // namespace dbp
