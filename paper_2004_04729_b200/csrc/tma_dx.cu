// Input gradient of 1x1 convolutions on the tensor cores, operands brought in by TMA (Eq. (qda)):
//   dX[b, ci, p] = Delta * sum_co W[co, ci] * q[b, co, p]
// The quantizer has written the codes as bf16 planes [b][co][pitch], so both operands are plain
// tiled copies: a stage holds 64 output channels (the reduction index) of
//   A = W rows  [64 co][128 ci]          (M = input channels, MN-major, two 64-channel panels)
//   B = codes   [64 co][up to 256 p]     (N = positions, MN-major, one panel per 64-position chunk)
// A CTA is persistent: warp 0 issues the copies, warp 1 the MMAs, warps 2-9 drain an accumulator
// (scale by Delta, convert, store through a shared-memory staging block so that global stores are
// whole rows). TMEM holds two 256-column accumulators. With one accumulator per tile (128
// channels) tiles alternate between them, so the stores of one tile overlap the copies and MMAs of
// the next. With two per tile (256 channels; chosen for long reductions over many channels) both
// accumulators share the stage's code tile, which halves the code traffic per MMA.
// Positions are handled in chunks of 64 that never cross an image; a tile is up to four
// consecutive chunks (they may belong to two images). Rows past the tensor's edge are zero-filled
// by the copy engine.
#include "tc_common.cuh"

namespace dbp {

namespace tc {

namespace {
bool encode_map(CUtensorMap *map, CUtensorMapDataType type, CUtensorMapSwizzle swizzle, const void *base, int rank,
                const unsigned long long *dims, const unsigned long long *strides_bytes, const unsigned *box) {
    typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn fn = nullptr;
    if (fn == nullptr) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || sym == nullptr) {
            cudaGetLastError();
            return false;
        }
        fn = reinterpret_cast<EncodeFn>(sym);
    }
    cuuint64_t gdim[5], gstr[4];
    cuuint32_t bx[5], es[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bx[i] = box[i];
        es[i] = 1;
        if (i > 0) gstr[i - 1] = strides_bytes[i - 1];
    }
    return fn(map, type, static_cast<cuuint32_t>(rank), const_cast<void *>(base), gdim, gstr, bx, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
}  // namespace

bool encode_map_bf16(CUtensorMap *map, const void *base, int rank, const unsigned long long *dims,
                     const unsigned long long *strides_bytes, const unsigned *box) {
    return encode_map(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, base, rank, dims, strides_bytes, box);
}

bool encode_map_f32_sw128(CUtensorMap *map, const void *base, int rank, const unsigned long long *dims,
                          const unsigned long long *strides_bytes, const unsigned *box) {
    return encode_map(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, CU_TENSOR_MAP_SWIZZLE_128B, base, rank, dims, strides_bytes, box);
}

bool encode_map_f32_rows(CUtensorMap *map, const void *base, int rank, const unsigned long long *dims,
                         const unsigned long long *strides_bytes, const unsigned *box) {
    return encode_map(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, CU_TENSOR_MAP_SWIZZLE_NONE, base, rank, dims, strides_bytes, box);
}

}  // namespace tc

namespace {

using namespace tc;

constexpr int kStages = 4;                       // most stages (one accumulator); three with two
constexpr int kPanel = 64 * 128;                 // 64 k-rows x 128 bytes
constexpr int kABytes = 2 * kPanel;              // 128 input channels (one accumulator's weights)
constexpr int kNChunks = 4;                      // chunks of 64 positions per tile
constexpr int kBBytes = kNChunks * kPanel;
constexpr int kRing = kStages * (kABytes + kBBytes);   // bytes of the stage ring (3 x 64 KB = 4 x 48 KB)
constexpr int kEpiWarps = 8;                      // two per TMEM lane quarter: even and odd chunks of a tile
constexpr int kThreadsT = 64 + 32 * kEpiWarps;
constexpr int kAccCols = 256;
constexpr int kStageOut = 32 * 128;               // one warp's staged chunk: 32 channels x 64 positions, bf16

struct DxT {
    const float *delta_p;
    void *dX;                     // [B][Cin][HW], bf16 or fp32
    int dx_f32;
    int tma_out;                  // bf16 dX whose rows are multiples of 16 bytes: chunks leave through the copy engine
    int Cin, Cout, HW;
    int chunks_per_img;
    long long nchunks;            // B * chunks_per_img
    int ci_tiles, ksteps;
    int nct;                      // 64-position chunks per tile (4, or fewer when that gives too few tiles)
    int MA;                       // accumulators per tile: 1 (128 channels, two tiles in flight) or 2 (256 channels)
    long long ntiles;             // tiles are taken from the last one down: the quantizer has just written the codes front to
                                  // back, so the end of a tensor larger than the L2 is what is still there
    int *err_flag;
    unsigned long long *stats;    // wait counters (may be null)
};

struct PipeT {
    unsigned long long full[kStages], empty[kStages], acc_full[2], acc_empty[2];
    unsigned tmem_base;
};

__global__ void __launch_bounds__(kThreadsT, 1)
tma_dx_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_q,
              const __grid_constant__ CUtensorMap map_dx, const DxT p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ PipeT pipe;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // With two accumulators a tile is 256 channels: both share the stage's code tile, each has its
    // own weight tile, and the two TMEM accumulators belong to one tile (no second tile in
    // flight). With one accumulator tiles alternate between the two TMEM accumulators.
    const int MA = p.MA, S = MA == 2 ? 3 : 4;
    const int a_bytes = MA * kABytes, stage_bytes = a_bytes + kBBytes;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&pipe.full[s], 1);
            mbar_init(&pipe.empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&pipe.acc_full[a], 1);
            mbar_init(&pipe.acc_empty[a], kEpiWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&map_w);
        tma_prefetch_desc(&map_q);
        if (p.tma_out) tma_prefetch_desc(&map_dx);
    }
    if (warp == 1) tmem_alloc(&pipe.tmem_base, 2 * kAccCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = pipe.tmem_base;
    // everything above touched only this CTA's shared and tensor memory; what follows reads what
    // earlier kernels wrote
    chain_wait();
    chain_release();

    if (warp == 0) {
        {   // the whole warp runs the loop (uniform control flow and operands); one elected lane issues
            int s = 0;
            unsigned parity = 1;                 // a fresh barrier passes a wait on the previous phase
            bool ok = true;
            long long waited = 0;
            for (long long t = blockIdx.x; t < p.ntiles && ok; t += gridDim.x) {
                const long long tr = p.ntiles - 1 - t;            // last positions first: see DxT::ntiles
                const int ci0 = static_cast<int>(tr % p.ci_tiles) * 128 * MA;
                const long long g0 = (tr / p.ci_tiles) * p.nct;
                const int nch = static_cast<int>(p.nchunks - g0 < p.nct ? p.nchunks - g0 : p.nct);
                // the tile's chunks are consecutive: image and position of the first, then step and wrap
                const int b0 = static_cast<int>(g0 / p.chunks_per_img);
                const int c0 = static_cast<int>(g0 - static_cast<long long>(b0) * p.chunks_per_img);
                const unsigned tx = static_cast<unsigned>((2 * MA + nch) * kPanel);
                for (int ks = 0; ks < p.ksteps && ok; ++ks) {
                    ok = __all_sync(0xffffffffu, mbar_wait_timed(&pipe.empty[s], parity, p.err_flag, waited));
                    if (!ok) break;
                    if (elect_one()) {
                        unsigned char *st = smem + s * stage_bytes;
                        mbar_expect_tx(&pipe.full[s], tx);
                        for (int h = 0; h < 2 * MA; ++h)
                            tma_load_2d(st + h * kPanel, &map_w, ci0 + 64 * h, ks * 64, &pipe.full[s]);
                        st += a_bytes;
                        int b = b0, c = c0;
                        for (int i = 0; i < nch; ++i, st += kPanel) {
                            tma_load_3d(st, &map_q, c * 64, ks * 64, b, &pipe.full[s]);
                            if (++c == p.chunks_per_img) { c = 0; ++b; }
                        }
                    }
                    if (++s == S) { s = 0; parity ^= 1u; }
                }
            }
            if (lane == 0) report_wait(p.stats, 3, waited);
        }
    } else if (warp == 1) {
        {   // the whole warp runs the loop (uniform control flow and operands); one elected lane issues
            const unsigned idesc = make_idesc(128, 64 * p.nct, true, true);
            int s = 0;
            unsigned parity = 0;
            bool ok = true;
            long long it = 0;
            long long wf = 0, wa = 0;
            const long long born = clock64();
            for (long long t = blockIdx.x; t < p.ntiles && ok; t += gridDim.x, ++it) {
                // accumulator slot(s) of this tile and how often they have been used before
                const int slot0 = MA == 2 ? 0 : static_cast<int>(it & 1);
                const unsigned uses = static_cast<unsigned>(MA == 2 ? it : (it >> 1));
                for (int a = 0; a < MA && ok; ++a)
                    ok = __all_sync(0xffffffffu, mbar_wait_timed(&pipe.acc_empty[slot0 + a], (uses & 1u) ^ 1u, p.err_flag, wa));
                if (!ok) break;
                tc_fence_after();
                for (int ks = 0; ks < p.ksteps; ++ks) {
                    ok = __all_sync(0xffffffffu, mbar_wait_timed(&pipe.full[s], parity, p.err_flag, wf));
                    if (!ok) break;
                    tc_fence_after();
                    const unsigned a_addr = smem_u32(smem + s * stage_bytes);
                    const unsigned long long bd = make_desc(a_addr + a_bytes, kPanel, 1024);
                    if (elect_one()) {
                        for (int a = 0; a < MA; ++a) {
                            const unsigned long long ad = make_desc(a_addr + a * kABytes, kPanel, 1024);
                            const unsigned tmem_d = tmem_base + (slot0 + a) * kAccCols;
#pragma unroll
                            for (int k = 0; k < 4; ++k)      // 16 k-rows = 2048 bytes further per MMA
                                mma_bf16(tmem_d, ad + 128 * k, bd + 128 * k, idesc, (ks > 0 || k > 0) ? 1u : 0u);
                        }
                        mma_commit(&pipe.empty[s]);
                    }
                    if (++s == S) { s = 0; parity ^= 1u; }
                }
                if (ok && elect_one())
                    for (int a = 0; a < MA; ++a) mma_commit(&pipe.acc_full[slot0 + a]);
            }
            if (lane == 0) {
                report_wait(p.stats, 1, wf);
                report_wait(p.stats, 2, wa);
                report_wait(p.stats, 6, clock64() - born);
                report_wait(p.stats, 7, 1);
            }
        }
    } else {
        // epilogue: TMEM lane = input channel, column = position
        const int q = warp & 3;
        bool ok = true;
        long long it = 0;
        long long we = 0;
        const float delta = *p.delta_p;
        const int vw = (p.HW % 8 == 0) ? 8 : ((p.HW % 4 == 0) ? 4 : 1);
        unsigned char *stage = smem + kRing + (warp - 2) * kStageOut;
        const int part = (warp - 2) >> 2;          // which chunks of a tile this warp drains
        for (long long t = blockIdx.x; t < p.ntiles && ok; t += gridDim.x, ++it) {
          const int slot0 = MA == 2 ? 0 : static_cast<int>(it & 1);
          const unsigned uses = static_cast<unsigned>(MA == 2 ? it : (it >> 1));
          for (int am = 0; am < MA; ++am) {
            const int a = slot0 + am;
            const long long tr = p.ntiles - 1 - t;
            const int ci_w = (static_cast<int>(tr % p.ci_tiles) * MA + am) * 128 + q * 32;
            const int ci = ci_w + lane;
            const long long g0 = (tr / p.ci_tiles) * p.nct;
            const int nch = static_cast<int>(p.nchunks - g0 < p.nct ? p.nchunks - g0 : p.nct);
            ok = mbar_wait_timed(&pipe.acc_full[a], uses & 1u, p.err_flag, we);
            if (!ok) break;
            tc_fence_after();
            for (int c = part; c < nch; c += kEpiWarps / 4) {
                const long long b = (g0 + c) / p.chunks_per_img;
                const int p0 = static_cast<int>((g0 + c) % p.chunks_per_img) * 64;
                if (p.tma_out) {
                    // the chunk's 32 channels x 64 positions: both halves out of TMEM, scaled and rounded, into the
                    // staging block as swizzled 128-byte rows, then one tiled store (which skips what lies
                    // outside the tensor). The block is free again once the previous store has read it.
                    unsigned v0[32], v1[32];
                    const unsigned taddr = tmem_base + (static_cast<unsigned>(q * 32) << 16) + a * kAccCols + c * 64;
                    tmem_ld32(taddr, v0);
                    tmem_ld32(taddr + 32, v1);
                    if (lane == 0) bulk_wait_read_all();
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        unsigned w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v0[8 * j + 2 * i]) * delta,
                                                                           __uint_as_float(v0[8 * j + 2 * i + 1]) * delta);
                            w[i] = *reinterpret_cast<const unsigned *>(&h);
                        }
                        *reinterpret_cast<uint4 *>(stage + lane * 128 + ((j ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        unsigned w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v1[8 * j + 2 * i]) * delta,
                                                                           __uint_as_float(v1[8 * j + 2 * i + 1]) * delta);
                            w[i] = *reinterpret_cast<const unsigned *>(&h);
                        }
                        *reinterpret_cast<uint4 *>(stage + lane * 128 + (((4 + j) ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    fence_async_proxy();
                    __syncwarp();
                    if (lane == 0 && ci_w < p.Cin) {
                        tma_store_3d(&map_dx, p0, ci_w, static_cast<int>(b), stage);
                        bulk_commit();
                    }
                    continue;
                }
                const int nv = p.HW - p0 < 64 ? p.HW - p0 : 64;           // valid positions of the chunk
                const bool rows128 = nv == 64 && vw >= 4;                 // staged as swizzled 128-byte rows
#pragma unroll 1
                for (int half = 0; half < 2; ++half) {
                    const int pp = p0 + half * 32;
                    if (pp >= p.HW) break;                         // warp-uniform
                    unsigned v[32];
                    tmem_ld32(tmem_base + (static_cast<unsigned>(q * 32) << 16) + a * kAccCols + c * 64 + half * 32, v);
                    if (ci >= p.Cin && p.dx_f32) continue;
                    const long long o = (b * p.Cin + ci) * p.HW + pp;
                    const int nval = p.HW - pp < 32 ? p.HW - pp : 32;
                    if (p.dx_f32) {
                        float *dst = static_cast<float *>(p.dX) + o;
                        if (vw >= 4) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                if (j < nval)
                                    *reinterpret_cast<float4 *>(dst + j) =
                                        make_float4(__uint_as_float(v[j]) * delta, __uint_as_float(v[j + 1]) * delta,
                                                    __uint_as_float(v[j + 2]) * delta, __uint_as_float(v[j + 3]) * delta);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < nval) dst[j] = __uint_as_float(v[j]) * delta;
                        }
                    } else {
                        // bf16: my 32 values go to the warp's staging block, which holds the chunk
                        // as [32 channels][nv positions] (16-byte pieces XOR-swizzled by the row
                        // when a row is 128 bytes, packed rows otherwise)
                        unsigned w[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * j]) * delta,
                                                                           __uint_as_float(v[2 * j + 1]) * delta);
                            w[j] = *reinterpret_cast<const unsigned *>(&h);
                        }
                        if (rows128) {
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                *reinterpret_cast<uint4 *>(stage + lane * 128 + (((half * 4 + j) ^ (lane & 7)) << 4)) =
                                    make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                        } else {
                            unsigned short *row = reinterpret_cast<unsigned short *>(stage) + lane * nv + half * 32;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < nval) row[j] = static_cast<unsigned short>(w[j >> 1] >> (16 * (j & 1)));
                        }
                    }
                }
                if (!p.dx_f32) {
                    // staging block -> dX with lanes along the positions: full 128-byte rows, or, when
                    // the chunk is the whole plane, one contiguous run of 32 channels x HW positions
                    __syncwarp();
                    const int nrows = p.Cin - ci_w < 32 ? p.Cin - ci_w : 32;
                    __nv_bfloat16 *base = static_cast<__nv_bfloat16 *>(p.dX) + (b * p.Cin + ci_w) * p.HW + p0;
                    if (nrows > 0) {
                        if (rows128 && vw == 8) {
#pragma unroll
                            for (int r0 = 0; r0 < 32; r0 += 4) {
                                const int r = r0 + (lane >> 3), ch = lane & 7;
                                if (r < nrows)
                                    *reinterpret_cast<uint4 *>(base + static_cast<long long>(r) * p.HW + ch * 8) =
                                        *reinterpret_cast<const uint4 *>(stage + r * 128 + ((ch ^ (r & 7)) << 4));
                            }
                        } else if (rows128) {
#pragma unroll
                            for (int r0 = 0; r0 < 32; r0 += 2) {
                                const int r = r0 + (lane >> 4), pc = lane & 15;
                                if (r < nrows)
                                    *reinterpret_cast<uint2 *>(base + static_cast<long long>(r) * p.HW + pc * 4) =
                                        *reinterpret_cast<const uint2 *>(stage + r * 128 + (((pc >> 1) ^ (r & 7)) << 4) + (pc & 1) * 8);
                            }
                        } else if (p.chunks_per_img == 1) {
                            const int n16 = nrows * nv / 8;          // nrows is a multiple of 8: whole 16-byte pieces
                            for (int i = lane; i < n16; i += 32)
                                reinterpret_cast<uint4 *>(base)[i] = reinterpret_cast<const uint4 *>(stage)[i];
                        } else if (vw >= 4) {
                            const int per_row = nv / 4, n8 = nrows * per_row;
                            for (int i = lane; i < n8; i += 32) {
                                const int r = i / per_row, c4 = i - r * per_row;
                                *reinterpret_cast<uint2 *>(base + static_cast<long long>(r) * p.HW + c4 * 4) =
                                    reinterpret_cast<const uint2 *>(stage)[i];
                            }
                        } else {
                            const int n2 = nrows * nv;
                            for (int i = lane; i < n2; i += 32) {
                                const int r = i / nv, c1 = i - r * nv;
                                reinterpret_cast<unsigned short *>(base + static_cast<long long>(r) * p.HW)[c1] =
                                    reinterpret_cast<const unsigned short *>(stage)[i];
                            }
                        }
                    }
                    __syncwarp();
                }
            }
            tc_fence_before();
            warp_arrive(&pipe.acc_empty[a]);
          }
        }
        if (p.tma_out && lane == 0) bulk_wait_read_all();      // the staging block is read before the CTA goes
        if (threadIdx.x == 64) report_wait(p.stats, 5, we);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, 2 * kAccCols);
    }
}

}  // namespace

bool tma_dx_supported(const ConvShape &s, int io) {
    return io == DBP_BF16 && s.k == 1 && s.Cin % 8 == 0 && s.H * s.W >= 16 && s.H * s.W < (1ll << 30);
}

long long tma_code_pitch(const ConvShape &s) { return (s.H * s.W + 7) / 8 * 8; }

int launch_tma_dx(dbp_ctx *ctx, const void *codes_bf16, const void *W, const float *delta_p,
                  const ConvShape &s, void *dX, bool dx_bf16, int *err_flag) {
    const long long HW = s.H * s.W, pitch = tma_code_pitch(s);
    CUtensorMap map_w, map_q;
    {
        const unsigned long long dims[2] = {static_cast<unsigned long long>(s.Cin), static_cast<unsigned long long>(s.Cout)};
        const unsigned long long str[1] = {static_cast<unsigned long long>(s.Cin) * 2};
        const unsigned box[2] = {64, 64};
        if (!encode_map_bf16(&map_w, W, 2, dims, str, box)) return DBP_ECUDA;
    }
    {
        const unsigned long long dims[3] = {static_cast<unsigned long long>(HW), static_cast<unsigned long long>(s.Cout),
                                            static_cast<unsigned long long>(s.B)};
        const unsigned long long str[2] = {static_cast<unsigned long long>(pitch) * 2,
                                           static_cast<unsigned long long>(pitch) * 2 * s.Cout};
        const unsigned box[3] = {64, 64, 1};
        if (!encode_map_bf16(&map_q, codes_bf16, 3, dims, str, box)) return DBP_ECUDA;
    }
    DxT p{};
    p.delta_p = delta_p; p.dX = dX; p.dx_f32 = dx_bf16 ? 0 : 1;
    CUtensorMap map_dx = map_w;                  // a valid map when the store path is not used
    p.tma_out = (dx_bf16 && HW % 8 == 0) ? 1 : 0;
    if (p.tma_out) {
        const unsigned long long dims[3] = {static_cast<unsigned long long>(HW), static_cast<unsigned long long>(s.Cin),
                                            static_cast<unsigned long long>(s.B)};
        const unsigned long long str[2] = {static_cast<unsigned long long>(HW) * 2, static_cast<unsigned long long>(HW) * 2 * s.Cin};
        const unsigned box[3] = {64, 32, 1};
        if (!encode_map_bf16(&map_dx, dX, 3, dims, str, box)) return DBP_ECUDA;
    }
    p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout); p.HW = static_cast<int>(HW);
    p.chunks_per_img = static_cast<int>((HW + 63) / 64);
    p.nchunks = s.B * p.chunks_per_img;
    p.ksteps = static_cast<int>((s.Cout + 63) / 64);
    // Two accumulators halve the code traffic per MMA but leave half as many tiles and no second
    // tile in flight: worth it for long reductions that still fill the GPU. Few tiles: narrower ones.
    const long long ntile4 = (p.nchunks + kNChunks - 1) / kNChunks;
    p.MA = (s.Cin >= 256 && p.ksteps >= 4 && ntile4 * ((s.Cin + 255) / 256) >= (ctx->sm_count * 3) / 4) ? 2 : 1;
    p.ci_tiles = static_cast<int>((s.Cin + 128 * p.MA - 1) / (128 * p.MA));
    p.nct = kNChunks;
    while (p.nct > 1 && ((p.nchunks + p.nct - 1) / p.nct) * p.ci_tiles < (ctx->sm_count * 3) / 4) p.nct /= 2;
    p.ntiles = ((p.nchunks + p.nct - 1) / p.nct) * p.ci_tiles;
    p.err_flag = err_flag;
    p.stats = ctx->wait_stats;
    const size_t smem = static_cast<size_t>(kRing) + kEpiWarps * kStageOut + 1024;
    if (cudaFuncSetAttribute(tma_dx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return DBP_ECUDA;
    const long long grid = p.ntiles < ctx->sm_count ? p.ntiles : ctx->sm_count;
    return cuda_ok(launch_chained(tma_dx_kernel, dim3(static_cast<unsigned>(grid)), dim3(kThreadsT), smem, ctx->stream,
                                  map_w, map_q, map_dx, p));
}

}  // namespace dbp
