// Weight gradient of 3x3 convolutions (stride 1, pad 1) on the tensor cores, both operands brought
// in by tiled copies (Eq. (qdw), "analogous for convolutional layers"):
//   dW[co][ci][ky][kx] = Delta * sum_(b,j) X[b][ci][j] * q[b][co][j - (ky-1) W - (kx-1)]
// with j a position of the image (row-major), the code taken as zero outside the image and where
// the column x - (kx-1) leaves the row.
//
// The reduction index is the position. The activations lie [b][ci][position], so 64 consecutive
// positions of 128 input channels are one K-major tile (A, M = input channels). The quantizer has
// written the codes position-major, [b][position][co] in bf16, so a run of positions of 64 output
// channels is one MN-major panel (B, N = output channels), one 128-byte row per position, and a
// tap is only a different start row of that panel (the 128-byte swizzle is a function of the
// shared-memory address). The copy engine zero-fills the rows before the first and after the last
// position of the image, which is the padding above and below. Left/right padding cannot be a row
// offset: a CTA handles ONE kernel column kx, and one warp zeroes, in the freshly copied panel, the
// rows of image column 0 (kx = 0) or W-1 (kx = 2) before the MMAs read it.
//
// Per CTA: a range of segments (runs of up to 512 positions of one image, with a halo of W+1 rows
// on either side), an output tile of 128 input channels x 64 or 128 output channels, the three
// taps ky of its kx as three accumulators in tensor memory. With 64 output channels the taps ky = 1
// and ky = 0 share one MMA of N = 128: its second 64-column group starts W rows further on.
// Warp 0 copies code panels, warp 1 activation tiles, warp 2 issues the MMAs, warp 3 zeroes the
// masked rows, warps 4-7 stage the accumulators in shared memory and the copy engine adds them into a
// zero-initialised fp32 scratch [tap][co][ci] (the reduction over CTAs; the order of the additions,
// hence the last bits of dW, can differ from run to run). A second kernel scales by Delta, writes
// dW[co][ci][ky][kx] and puts the zeros back. Every wait is bounded.
#include "tc_common.cuh"

namespace dbp {

namespace {

using namespace tc;

constexpr int kThreadsW3 = 8 * 32;
constexpr int kXTile = 16384;             // [128 ci][64 positions] bf16
constexpr int kXS = 2;                    // 64-position stages per activation slot (one hand-over)
constexpr int kXSlot = kXS * kXTile;
constexpr int kMaxNX = 6;

struct Dw3T {
    int Cin, Cout, W, HW;
    int code_batch;               // images of the code tensor (the activations may hold two pieces of every image, one after the other)
    int SEG;                      // positions per segment (multiple of 64)
    int segs_per_img;
    long long nseg, per_split;
    int nsplit;
    int ci_tiles, co_tiles;
    int rows_box, nload;          // a panel is copied as nload boxes of rows_box rows
    int panel_bytes;              // multiple of 1024
    int nx;                       // activation slots in flight
    int stage_chunks;             // 32-column chunks of the accumulators that fit the shared memory at once
    int phase_tiles;              // > 0: a stride-2 layer on phase images, this many 128-channel tiles per phase (phase
                                  // ph = 2 py + px holds channels ph * 128 * phase_tiles ...). Only the taps with
                                  // ky in {1} (py = 0) or {0, 1} (py = 1), kx likewise, are wanted: the work items of
                                  // the other kernel columns do not exist and the other rows' MMAs are left out
    int *err_flag;
    unsigned long long *stats;    // wait counters (may be null)
};

struct PipeW3 {
    unsigned long long x_full[kMaxNX], x_empty[kMaxNX], q_full[2], q_ready[2], q_empty[2], acc;
    unsigned tmem_base;
};

// NP: 64-channel panels of the code operand (N = 64 NP output channels per tap)
template <int NP>
__global__ void __launch_bounds__(kThreadsW3, 1)
tc3_tma_dw_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_x,
                  const __grid_constant__ CUtensorMap map_acc, const Dw3T p) {
    constexpr int TCOLS = NP == 2 ? 512 : 256;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char *x_s = smem;                                   // nx activation slots
    unsigned char *q_s = x_s + p.nx * kXSlot;                    // 2 buffers x NP panels
    const int qbuf_bytes = NP * p.panel_bytes;
    __shared__ PipeW3 pipe;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // work item: (output tile, kernel column, range of segments)
    const int split = blockIdx.x % p.nsplit;
    int rest = blockIdx.x / p.nsplit;
    int kx, ci_t, co_t, live_lo = 0, live_hi = 3;       // rows ky in [live_lo, live_hi) are accumulated (NP == 2)
    int c_lo = 0, c_hi = (NP == 2 ? 384 : 192) / 32;    // 32-column chunks of the accumulators that are handed over
    if (p.phase_tiles > 0) {
        // per output-channel tile: the phases in order, one kernel column (kx = 1) per channel tile of a phase with
        // px = 0, two (kx = 0, 1) with px = 1
        const int tp = p.phase_tiles, per_co = 6 * tp;
        co_t = rest / per_co;
        int r = rest - co_t * per_co;
        const int py = r / (3 * tp);
        r -= py * 3 * tp;
        if (r < tp) { ci_t = 2 * py * tp + r; kx = 1; }
        else { r -= tp; ci_t = (2 * py + 1) * tp + (r >> 1); kx = r & 1; }
        // NP == 2: columns 0-127 are ky = 0, 128-255 ky = 1, 256-383 ky = 2; NP == 1: 0-63 ky = 2, 64-127 ky = 1, 128-191 ky = 0
        if (NP == 2) { live_lo = py ? 0 : 1; live_hi = 2; c_lo = 4 * live_lo; c_hi = 8; }
        else { c_lo = 2; c_hi = py ? 6 : 4; }
    } else {
        kx = rest % 3;
        rest /= 3;
        ci_t = rest % p.ci_tiles;
        co_t = rest / p.ci_tiles;
    }
    const int ci0 = ci_t * 128;
    const int co0 = co_t * 64 * NP;
    const long long g0 = split * p.per_split;
    const long long g1 = g0 + p.per_split < p.nseg ? g0 + p.per_split : p.nseg;
    const int halo = p.W + 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxNX; ++s) { mbar_init(&pipe.x_full[s], 1); mbar_init(&pipe.x_empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&pipe.q_full[s], 1); mbar_init(&pipe.q_ready[s], 1); mbar_init(&pipe.q_empty[s], 1); }
        mbar_init(&pipe.acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_x);
        tma_prefetch_desc(&map_acc);
    }
    if (warp == 2) tmem_alloc(&pipe.tmem_base, TCOLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = pipe.tmem_base;
    chain_wait();        // from here on the kernel reads what earlier kernels wrote
    chain_release();

    // segment g: image, first position, number of 64-position stages
    auto seg_of = [&](long long g, int &b, int &u0, int &ns) {
        b = static_cast<int>(g / p.segs_per_img);
        u0 = static_cast<int>(g - static_cast<long long>(b) * p.segs_per_img) * p.SEG;
        const int left = p.HW - u0;
        ns = ((left < p.SEG ? left : p.SEG) + 63) >> 6;
    };
    // The activation stages of this CTA are consecutive 64-position blocks of consecutive images; a
    // slot holds kXS consecutive blocks of one image. A new slot starts at the CTA's first stage, at
    // the first block of an image, and after kXS stages (copy and MMA threads follow the same rule).

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            const unsigned tx = static_cast<unsigned>(NP * p.nload * p.rows_box * 128);
            int sg = 0;
            long long waited = 0;
            for (long long g = g0; g < g1 && ok; ++g, ++sg) {
                int b, u0, ns;
                seg_of(g, b, u0, ns);
                const int buf = sg & 1;
                ok = mbar_wait_timed(&pipe.q_empty[buf], ((sg >> 1) & 1) ^ 1, p.err_flag, waited);
                if (!ok) break;
                unsigned char *dst = q_s + buf * qbuf_bytes;
                mbar_expect_tx(&pipe.q_full[buf], tx);
#pragma unroll
                for (int pn = 0; pn < NP; ++pn)
                    for (int l = 0; l < p.nload; ++l)
                        tma_load_3d(dst + pn * p.panel_bytes + l * p.rows_box * 128, &map_q, co0 + 64 * pn,
                                    u0 - halo + l * p.rows_box, b % p.code_batch, &pipe.q_full[buf]);
            }
            report_wait(p.stats, 3, waited);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            int s = 0, j = kXS;                    // j: stages already in the current slot
            unsigned parity = 1;
            long long waited = 0;
            for (long long g = g0; g < g1 && ok; ++g) {
                int b, u0, ns;
                seg_of(g, b, u0, ns);
                for (int k = 0; k < ns; ++k) {
                    const int blk = (u0 >> 6) + k;
                    if (j == kXS || blk == 0) {
                        ok = mbar_wait_timed(&pipe.x_empty[s], parity, p.err_flag, waited);
                        if (!ok) break;
                        unsigned char *dst = x_s + s * kXSlot;
                        mbar_expect_tx(&pipe.x_full[s], kXSlot);
                        // positions past the image's end read as zero (a block past its end is all zero)
#pragma unroll
                        for (int i = 0; i < kXS; ++i)
                            tma_load_3d(dst + i * kXTile, &map_x, (blk + i) * 64, ci0, b, &pipe.x_full[s]);
                        if (++s == p.nx) { s = 0; parity ^= 1u; }
                        j = 0;
                    }
                    ++j;
                }
            }
            report_wait(p.stats, 4, waited);
        }
    } else if (warp == 2) {
        {   // the whole warp runs the loop (uniform control flow and operands); one elected lane issues
            // tap ky reads the panel from row (2 - ky) W + (2 - kx) on. NP == 2: one MMA of N = 128 per tap
            // (accumulator columns 128 ky ...). NP == 1: the three taps share ONE MMA of N = 192 whose
            // 64-column groups start W rows apart (columns 0-63: ky = 2, 64-127: ky = 1, 128-191: ky = 0):
            // an MMA instruction takes about a hundred clocks to issue however narrow it is.
            constexpr unsigned idesc128 = make_idesc(128, 128, false, true), idesc192 = make_idesc(128, 192, false, true);
            const unsigned r0 = static_cast<unsigned>((2 * p.W + 2 - kx) * 8), r1 = static_cast<unsigned>((p.W + 2 - kx) * 8),
                           r2 = static_cast<unsigned>((2 - kx) * 8);     // start rows in 16-byte units
            bool ok = true;
            int slot = -1, j = kXS, sg = 0;
            unsigned xpar = 0;
            unsigned acc_on = 0u;
            long long wq = 0, wx = 0;
            const long long born = clock64();
            for (long long g = g0; g < g1 && ok; ++g, ++sg) {
                int b, u0, ns;
                seg_of(g, b, u0, ns);
                const int buf = sg & 1;
                ok = __all_sync(0xffffffffu, mbar_wait_timed(&pipe.q_ready[buf], (sg >> 1) & 1, p.err_flag, wq));
                if (!ok) break;
                tc_fence_after();
                const unsigned q_addr = smem_u32(q_s + buf * qbuf_bytes);
                const unsigned long long bA = NP == 2 ? make_desc(q_addr, p.panel_bytes, 1024) + r0
                                                      : make_desc(q_addr, p.W * 128, 1024) + r2;
                const unsigned long long bB = make_desc(q_addr, p.panel_bytes, 1024) + r1;     // NP == 2 only
                const unsigned long long bC = make_desc(q_addr, p.panel_bytes, 1024) + r2;     // NP == 2 only
                for (int k = 0; k < ns && ok; ++k) {
                    const int blk = (u0 >> 6) + k;
                    if (j == kXS || blk == 0) {
                        if (slot >= 0 && elect_one()) mma_commit(&pipe.x_empty[slot]);
                        if (++slot == p.nx) { slot = 0; xpar ^= 1u; }
                        ok = __all_sync(0xffffffffu, mbar_wait_timed(&pipe.x_full[slot], xpar, p.err_flag, wx));
                        if (!ok) break;
                        tc_fence_after();
                        j = 0;
                    }
                    // the last stage of an image may hold fewer than 64 positions: skip the 16-position
                    // slices that are entirely zero fill
                    const int left = p.HW - (u0 + 64 * k);
                    const int nk = left >= 64 ? 4 : (left + 15) >> 4;
                    const unsigned long long ad = make_desc(smem_u32(x_s + slot * kXSlot + j * kXTile), 16, 1024);
                    const unsigned radv = static_cast<unsigned>(64 * k * 8);
                    if (elect_one())
                    for (int kk = 0; kk < nk; ++kk) {
                        const unsigned adv = radv + kk * 128;                 // 16 rows = 2048 bytes
                        if (NP == 2) {
                            if (live_lo == 0) mma_bf16(tmem_base, ad + 2 * kk, bA + adv, idesc128, acc_on);
                            mma_bf16(tmem_base + 128, ad + 2 * kk, bB + adv, idesc128, acc_on);
                            if (live_hi == 3) mma_bf16(tmem_base + 256, ad + 2 * kk, bC + adv, idesc128, acc_on);
                        } else {
                            mma_bf16(tmem_base, ad + 2 * kk, bA + adv, idesc192, acc_on);
                        }
                        acc_on = 1u;
                    }
                    acc_on = 1u;
                    ++j;
                }
                if (ok && elect_one()) mma_commit(&pipe.q_empty[buf]);
            }
            if (ok && slot >= 0 && elect_one()) mma_commit(&pipe.x_empty[slot]);
            if (ok && g1 > g0 && elect_one()) mma_commit(&pipe.acc);
            if (lane == 0) {
                report_wait(p.stats, 0, wq);
                report_wait(p.stats, 1, wx);
                report_wait(p.stats, 6, clock64() - born);
                report_wait(p.stats, 7, 1);
            }
        }
    } else if (warp == 3) {
        // masked rows: image column 0 for kx = 0, W-1 for kx = 2 (generic-proxy writes, then a proxy
        // fence so that the tensor core sees them)
        bool ok = true;
        int sg = 0;
        const int zc = kx == 0 ? 0 : p.W - 1;
        const int rows_total = p.nload * p.rows_box;
        for (long long g = g0; g < g1 && ok; ++g, ++sg) {
            int b, u0, ns;
            seg_of(g, b, u0, ns);
            const int buf = sg & 1;
            ok = mbar_wait(&pipe.q_full[buf], (sg >> 1) & 1, p.err_flag);
            if (!ok) break;
            if (kx != 1) {
                unsigned char *qb = q_s + buf * qbuf_bytes;
                const int i_lo = u0 - halo;                       // image position of panel row 0
                // first image position >= max(i_lo, 0) in column zc
                const int start = i_lo > 0 ? i_lo : 0;
                int i = start + ((zc - start % p.W) + p.W) % p.W;
                const int sub = lane >> 3, chunk = lane & 7;      // four rows x eight 16-byte pieces per pass
                i += sub * p.W;
                for (; i < p.HW && i - i_lo < rows_total; i += 4 * p.W) {
                    const int r = i - i_lo;
#pragma unroll
                    for (int pn = 0; pn < NP; ++pn)
                        *reinterpret_cast<uint4 *>(qb + pn * p.panel_bytes + r * 128 + chunk * 16) = make_uint4(0u, 0u, 0u, 0u);
                }
                fence_async_proxy();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&pipe.q_ready[buf]);
        }
    } else {
        // epilogue: TMEM lane = input channel, column = (tap, output channel). Every buffer of the
        // pipeline is free by now, so the accumulators are staged there as plain fp32 rows
        // [column][128 ci] and one thread hands them to the copy engine, which adds them into the
        // scratch [tap][co][ci] (rows of 512 bytes, 32 columns per request).
        const int q = warp & 3, et = threadIdx.x - 128;
        bool ok = g1 > g0 && mbar_wait(&pipe.acc, 0, p.err_flag);
        {   // the same decision in all 128 threads (they meet at barriers below)
            unsigned r;
            asm volatile(
                "{\n\t.reg .pred p, q;\n\t"
                "setp.ne.b32 p, %1, 0;\n\t"
                "bar.red.and.pred q, 1, 128, p;\n\t"
                "selp.b32 %0, 1, 0, q;\n\t}"
                : "=r"(r) : "r"(ok ? 1u : 0u) : "memory");
            ok = r != 0;
        }
        if (ok) {
            tc_fence_after();
            const long long t_epi = clock64();
            const int nchunks = c_hi;                  // only the rows the layer wants are handed over
            float *stg = reinterpret_cast<float *>(smem);
            for (int c0 = c_lo; c0 < nchunks; c0 += p.stage_chunks) {
                const int nb = nchunks - c0 < p.stage_chunks ? nchunks - c0 : p.stage_chunks;
                for (int i = 0; i < nb; ++i) {
                    unsigned v[32];
                    tmem_ld32(tmem_base + (static_cast<unsigned>(q * 32) << 16) + (c0 + i) * 32, v);
                    float *dst = stg + i * 4096 + q * 32 + lane;
#pragma unroll
                    for (int j = 0; j < 32; ++j) dst[j * 128] = __uint_as_float(v[j]);
                }
                fence_async_proxy();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (et == 0) {
                    for (int i = 0; i < nb; ++i) {
                        const int c = c0 + i;
                        int ky, col0;                           // tap and first output channel of these 32 columns
                        if (NP == 2) { ky = c >> 2; col0 = (c & 3) * 32; }     // columns 0-127: ky = 0, 128-255: ky = 1, ...
                        else { ky = 2 - (c >> 1); col0 = (c & 1) * 32; }       // columns 0-63: ky = 2, 64-127: ky = 1, 128-191: ky = 0
                        // columns past Cout hold exact zeros (their codes were zero fill): adding them is harmless
                        tma_reduce_add_2d(&map_acc, ci0, (ky * 3 + kx) * p.Cout + co0 + col0, stg + i * 4096);
                    }
                    bulk_commit();
                    bulk_wait_read_all();
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
            if (et == 0) report_wait(p.stats, 5, clock64() - t_epi);     // how long handing over the sums took
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        __syncwarp();
        tmem_dealloc(tmem_base, TCOLS);
    }
}

// dW[co][ci][tap] = Delta * acc[tap][co][cip]; the scratch goes back to zero for the next call. The scratch
// rows hold cin_pad >= Cin channels (activations whose channel count is no multiple of 8 were padded).
// A block takes 256 consecutive (co, cip) pairs, one per thread: nine coalesced reads (and the zeros written
// back), a transposition through shared memory (row pitch 9 words: no bank conflicts either way), and the
// results leave as one contiguous run.
__global__ void __launch_bounds__(256)
tc3_dw_finish_kernel(float *__restrict__ acc, const float *__restrict__ delta_p, float *__restrict__ dW, long long pairs,
                     int cin, int cin_pad) {
    __shared__ float t_s[256 * 9];
    chain_wait();
    chain_release();
    const float delta = *delta_p;
    for (long long i0 = blockIdx.x * 256ll; i0 < pairs; i0 += gridDim.x * 256ll) {
        const long long i = i0 + threadIdx.x;
        if (i < pairs) {
            float v[9];
#pragma unroll
            for (int t = 0; t < 9; ++t) v[t] = __ldcg(acc + t * pairs + i);
#pragma unroll
            for (int t = 0; t < 9; ++t) {
                __stcg(acc + t * pairs + i, 0.f);
                t_s[threadIdx.x * 9 + t] = v[t] * delta;
            }
        }
        __syncthreads();
        const long long left = pairs - i0;
        const int np = static_cast<int>(left < 256 ? left : 256);
        if (cin == cin_pad) {
            for (int k = threadIdx.x; k < np * 9; k += 256) dW[i0 * 9 + k] = t_s[k];
        } else {
            for (int k = threadIdx.x; k < np * 9; k += 256) {
                const long long pr = i0 + k / 9;
                const long long co = pr / cin_pad;
                const int ci = static_cast<int>(pr - co * cin_pad);
                if (ci < cin) dW[(co * cin + ci) * 9 + k % 9] = t_s[k];
            }
        }
        __syncthreads();
    }
}

// The same for a stride-2 layer run on phase images (scratch rows of 4 cin channels, phase ph = 2 py + px at channels
// ph * cin ...): the strided layer's tap (ky, kx) of (co, ci) is tap (ty, tx) of channel ph * cin + ci with
// ky = 0 -> (py, ty) = (1, 0), 1 -> (0, 1), 2 -> (1, 1), kx likewise; the other scratch entries were never touched.
// dW[co][ci][ky][kx] is written directly, one (co, ci) pair per thread.
__global__ void __launch_bounds__(256)
tc3_dw_finish_phases_kernel(float *__restrict__ acc, const float *__restrict__ delta_p, float *__restrict__ dW, int cout, int cin) {
    __shared__ float t_s[256 * 9];
    chain_wait();
    chain_release();
    const float delta = *delta_p;
    const long long pairs = static_cast<long long>(cout) * cin, pairs4 = 4 * pairs;
    for (long long i0 = blockIdx.x * 256ll; i0 < pairs; i0 += gridDim.x * 256ll) {
        const long long i = i0 + threadIdx.x;
        if (i < pairs) {
            const long long co = i / cin, ci = i - co * cin;
            float *base = acc + co * 4 * cin + ci;
            float v[9];
#pragma unroll
            for (int t = 0; t < 9; ++t) {
                const int ky = t / 3, kx = t % 3;
                const int ph = (ky != 1) * 2 + (kx != 1), tp = (ky == 0 ? 0 : 1) * 3 + (kx == 0 ? 0 : 1);
                v[t] = __ldcg(base + tp * pairs4 + static_cast<long long>(ph) * cin);
            }
#pragma unroll
            for (int t = 0; t < 9; ++t) {
                const int ky = t / 3, kx = t % 3;
                const int ph = (ky != 1) * 2 + (kx != 1), tp = (ky == 0 ? 0 : 1) * 3 + (kx == 0 ? 0 : 1);
                __stcg(base + tp * pairs4 + static_cast<long long>(ph) * cin, 0.f);
                t_s[threadIdx.x * 9 + t] = v[t] * delta;
            }
        }
        __syncthreads();
        const long long left = pairs - i0;
        const int np = static_cast<int>(left < 256 ? left : 256);
        for (int k = threadIdx.x; k < np * 9; k += 256) dW[i0 * 9 + k] = t_s[k];
        __syncthreads();
    }
}

// fp32 activations [B][Cin][HW] -> two bf16 tensors [B][cin_pad][pitch], one after the other: the values rounded
// to bf16 and what that rounding left over, rounded again (the two pieces add up to the fp32 value to within
// 2^-18 of it). Rows are padded to `pitch` (a multiple of 8) and channels to cin_pad (a multiple of 8) with zeros.
// A thread takes eight consecutive positions of one plane: two 16-byte loads where the plane allows it, one 16-byte
// store per piece.
__global__ void __launch_bounds__(256)
x_split_kernel(const float *__restrict__ X, __nv_bfloat16 *__restrict__ out, long long B, int Cin, int cin_pad, int HW, int pitch) {
    chain_wait();
    chain_release();
    const int gpp = pitch / 8;                                   // groups of eight positions per plane
    const long long planes = B * cin_pad, ngroups = planes * gpp;
    const long long n = planes * pitch;
    const bool vec = (HW % 4 == 0);
    for (long long gi = blockIdx.x * 256ll + threadIdx.x; gi < ngroups; gi += gridDim.x * 256ll) {
        long long pl;
        int gq;
        if ((ngroups >> 31) == 0) {                              // 32-bit divisions cost a fraction of 64-bit ones
            const unsigned u = static_cast<unsigned>(gi);
            pl = u / static_cast<unsigned>(gpp);
            gq = static_cast<int>(u - static_cast<unsigned>(pl) * static_cast<unsigned>(gpp));
        } else {
            pl = gi / gpp;
            gq = static_cast<int>(gi - pl * gpp);
        }
        const long long b = pl / cin_pad;
        const int ci = static_cast<int>(pl - b * cin_pad);
        const int pp0 = gq * 8;
        float x[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (ci < Cin && pp0 < HW) {
            const float *src = X + (b * Cin + ci) * HW + pp0;
            if (vec) {
                const float4 v0 = __ldg(reinterpret_cast<const float4 *>(src));
                x[0] = v0.x; x[1] = v0.y; x[2] = v0.z; x[3] = v0.w;
                if (pp0 + 4 < HW) {
                    const float4 v1 = __ldg(reinterpret_cast<const float4 *>(src + 4));
                    x[4] = v1.x; x[5] = v1.y; x[6] = v1.z; x[7] = v1.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (pp0 + i < HW) x[i] = __ldg(src + i);
            }
        }
        unsigned h[4], l[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 hh = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
            const float2 hf = __bfloat1622float2(hh);
            const __nv_bfloat162 ll = __floats2bfloat162_rn(x[2 * i] - hf.x, x[2 * i + 1] - hf.y);
            h[i] = *reinterpret_cast<const unsigned *>(&hh);
            l[i] = *reinterpret_cast<const unsigned *>(&ll);
        }
        const long long o = pl * pitch + pp0;
        *reinterpret_cast<uint4 *>(out + o) = make_uint4(h[0], h[1], h[2], h[3]);
        *reinterpret_cast<uint4 *>(out + n + o) = make_uint4(l[0], l[1], l[2], l[3]);
    }
}

// The same for tiny planes stacked into tall images (one row of zeros after every image): out is
// [2][B / G][cin_pad][pitch] with G (H + 1) W positions per tall image; position q of tall image t is position
// q % ((H + 1) W) of image t G + q / ((H + 1) W), or zero in the extra row and in the padding.
__global__ void __launch_bounds__(256)
x_split_stacked_kernel(const float *__restrict__ X, __nv_bfloat16 *__restrict__ out, long long Bt, int G, int Cin, int cin_pad,
                       int HW, int W, int pitch) {
    chain_wait();
    chain_release();
    const long long n = Bt * cin_pad * pitch;
    const int per_img = HW + W;
    for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += gridDim.x * 256ll) {
        const long long pl = i / pitch;
        const int q = static_cast<int>(i - pl * pitch);
        const long long t = pl / cin_pad;
        const int ci = static_cast<int>(pl - t * cin_pad);
        const int g = q / per_img, r = q - g * per_img;
        __nv_bfloat16 hi = __float2bfloat16_rn(0.f), lo = hi;
        if (g < G && r < HW && ci < Cin) {
            const float x = __ldg(X + ((t * G + g) * Cin + ci) * HW + r);
            hi = __float2bfloat16_rn(x);
            lo = __float2bfloat16_rn(x - __bfloat162float(hi));
        }
        out[i] = hi;
        out[n + i] = lo;
    }
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

}  // namespace

// DBP_EUNSUPPORTED: the shape does not fit (the caller uses another kernel)
int tc3_stack_images(const ConvShape &s, int io) {
    const long long HW = s.H * s.W, per_img = HW + s.W;
    if (io != DBP_F32 || s.k != 3 || HW >= 64 || per_img > 64 || s.B < 2) return 0;
    // the largest divisor of the batch whose tall image stays within one segment of the kernel
    for (long long g = s.B; g >= 2; --g)
        if (s.B % g == 0 && g * per_img <= 320) return static_cast<int>(g);
    return 0;
}

// stack_g > 0: `s` describes the tall images (B / G of them, G (H + 1) rows) and the codes are the stacked copy;
// real_h is the height of one image
int launch_tc3_tma_dw(dbp_ctx *ctx, const void *codes_nhwc, const void *X, int io, const float *delta_p,
                      const ConvShape &s, float *dW, int *err_flag, int stack_g, int real_h) {
    if (!tc3_tma_dw_supported(s, io)) return DBP_EUNSUPPORTED;
    if (stack_g > 0 && io != DBP_F32) return DBP_EINVAL;
    const int pieces = io == DBP_F32 ? 2 : 1;
    // fp32 activations are re-written anyway (split into two bf16 pieces): their channels are padded to a
    // multiple of 8 on the way, so any Cin works there
    const long long cin_pad = io == DBP_F32 ? (s.Cin + 7) / 8 * 8 : s.Cin;
    const long long HW = s.H * s.W;
    Dw3T p{};
    p.Cin = static_cast<int>(cin_pad); p.Cout = static_cast<int>(s.Cout); p.W = static_cast<int>(s.W); p.HW = static_cast<int>(HW);
    p.err_flag = err_flag;
    p.stats = ctx->wait_stats;
    const int NP = s.Cout > 64 ? 2 : 1;
    p.ci_tiles = static_cast<int>((cin_pad + 127) / 128);
    p.co_tiles = static_cast<int>((s.Cout + 64 * NP - 1) / (64 * NP));
    // the longest segment whose two code buffers fit beside at least three activation slots
    const size_t budget = 227 * 1024 - 2048;
    const int seg_cap = static_cast<int>(HW < 512 ? (HW + 63) / 64 * 64 : 512);
    size_t smem = 0;
    for (int seg = seg_cap; seg >= 64; seg -= 64) {
        const int rows = seg + 2 * (p.W + 1);
        const int nload = (rows + 255) / 256, rows_box = (rows + nload - 1) / nload;
        const int panel = round_up(nload * rows_box * 128, 1024);
        const size_t fixed = 2 * static_cast<size_t>(NP) * panel + 1024;
        if (fixed + 3 * kXSlot > budget) continue;
        p.SEG = seg; p.nload = nload; p.rows_box = rows_box; p.panel_bytes = panel;
        p.nx = static_cast<int>((budget - fixed) / kXSlot);
        if (p.nx > kMaxNX) p.nx = kMaxNX;
        smem = fixed + static_cast<size_t>(p.nx) * kXSlot;
        break;
    }
    if (smem == 0) return DBP_EUNSUPPORTED;
    p.segs_per_img = (p.HW + p.SEG - 1) / p.SEG;
    p.code_batch = static_cast<int>(s.B);
    p.nseg = s.B * pieces * p.segs_per_img;
    // a stride-2 layer on phase images whose phases are whole channel tiles: 6 of the 12 (phase, kernel column)
    // pairs carry taps of the strided layer
    p.phase_tiles = (ctx->phase_cin > 0 && ctx->phase_cin % 128 == 0 && cin_pad == 4ll * ctx->phase_cin && stack_g == 0)
                        ? ctx->phase_cin / 128 : 0;
    const long long tiles = p.phase_tiles > 0 ? static_cast<long long>(p.co_tiles) * 6 * p.phase_tiles
                                              : static_cast<long long>(p.ci_tiles) * p.co_tiles * 3;
    const long long nsplit = choose_split(tiles, p.nseg, ctx->sm_count, &p.per_split);
    p.nsplit = static_cast<int>(nsplit);
    if (tiles * nsplit >= (1ll << 31)) return DBP_EUNSUPPORTED;
    // fp32 scratch [9][Cout][Cin]: zero whenever no call is in flight
    const size_t pairs = static_cast<size_t>(s.Cout) * cin_pad;
    const size_t had = ctx->dw_acc.bytes;
    int rc = ws_reserve(ctx, ctx->dw_acc, pairs * 9 * sizeof(float));
    if (rc) return rc;
    if (ctx->dw_acc.bytes != had || !ctx->dw_acc_clean) {
        if (cudaMemsetAsync(ctx->dw_acc.ptr, 0, ctx->dw_acc.bytes, ctx->stream) != cudaSuccess) return fail_cuda("clearing the dW scratch");
        ctx->dw_acc_clean = true;
    }
    float *acc = static_cast<float *>(ctx->dw_acc.ptr);
    p.stage_chunks = static_cast<int>((smem - 1024) / 16384);
    // fp32 activations are split into two bf16 pieces (as if the batch were twice as long); bf16 ones whose
    // planes do not start on 16-byte boundaries are first copied to padded planes
    const void *Xsrc = X;
    long long xpitch = HW;
    if (io == DBP_F32) {
        xpitch = (HW + 7) / 8 * 8;
        const long long planes = s.B * cin_pad;
        if ((rc = ws_reserve(ctx, ctx->x_padded, static_cast<size_t>(planes) * xpitch * 2 * 2))) return rc;
        long long blocks = (planes * (xpitch / 8) + 255) / 256;
        if (blocks > ctx->sm_count * 16) blocks = ctx->sm_count * 16;
        if (stack_g > 0) {
            blocks = (planes * xpitch + 255) / 256;
            if (blocks > ctx->sm_count * 16) blocks = ctx->sm_count * 16;
            rc = cuda_ok(launch_chained(x_split_stacked_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, ctx->stream,
                                        static_cast<const float *>(X), static_cast<__nv_bfloat16 *>(ctx->x_padded.ptr), s.B, stack_g,
                                        static_cast<int>(s.Cin), static_cast<int>(cin_pad), static_cast<int>(real_h * s.W),
                                        static_cast<int>(s.W), static_cast<int>(xpitch)));
        } else {
            rc = cuda_ok(launch_chained(x_split_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, ctx->stream,
                                        static_cast<const float *>(X), static_cast<__nv_bfloat16 *>(ctx->x_padded.ptr), s.B,
                                        static_cast<int>(s.Cin), static_cast<int>(cin_pad), static_cast<int>(HW), static_cast<int>(xpitch)));
        }
        if (rc) return rc;
        Xsrc = ctx->x_padded.ptr;
    } else if (HW % 8 != 0) {
        xpitch = (HW + 7) / 8 * 8;
        if ((rc = ws_reserve(ctx, ctx->x_padded, static_cast<size_t>(s.B) * s.Cin * xpitch * 2))) return rc;
        if ((rc = launch_pad_planes(ctx, X, ctx->x_padded.ptr, s.B * s.Cin, 1, static_cast<int>(HW), static_cast<int>(xpitch))))
            return rc;
        Xsrc = ctx->x_padded.ptr;
    }
    CUtensorMap map_q, map_x, map_acc;
    {
        const unsigned long long dims[2] = {static_cast<unsigned long long>(cin_pad), static_cast<unsigned long long>(s.Cout) * 9};
        const unsigned long long str[1] = {static_cast<unsigned long long>(cin_pad) * 4};
        const unsigned box[2] = {128, 32};
        if (!encode_map_f32_rows(&map_acc, acc, 2, dims, str, box)) return fail_cuda("tensor map of the dW scratch");
    }
    {
        const unsigned long long dims[3] = {static_cast<unsigned long long>(s.Cout), static_cast<unsigned long long>(HW),
                                            static_cast<unsigned long long>(s.B)};
        const unsigned long long str[2] = {static_cast<unsigned long long>(s.Cout) * 2,
                                           static_cast<unsigned long long>(s.Cout) * 2 * HW};
        const unsigned box[3] = {64, static_cast<unsigned>(p.rows_box), 1};
        if (!encode_map_bf16(&map_q, codes_nhwc, 3, dims, str, box)) return fail_cuda("tensor map of the code panels");
    }
    {
        const unsigned long long dims[3] = {static_cast<unsigned long long>(HW), static_cast<unsigned long long>(cin_pad),
                                            static_cast<unsigned long long>(s.B) * pieces};
        const unsigned long long str[2] = {static_cast<unsigned long long>(xpitch) * 2,
                                           static_cast<unsigned long long>(xpitch) * 2 * cin_pad};
        const unsigned box[3] = {64, 128, 1};
        if (!encode_map_bf16(&map_x, Xsrc, 3, dims, str, box)) return fail_cuda("tensor map of the activations");
    }
    auto kern = NP == 2 ? tc3_tma_dw_kernel<2> : tc3_tma_dw_kernel<1>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return fail_cuda("shared memory size");
    if ((rc = cuda_ok(launch_chained(kern, dim3(static_cast<unsigned>(tiles * nsplit)), dim3(kThreadsW3), smem,
                                     ctx->stream, map_q, map_x, map_acc, p))))
        return rc;
    if (p.phase_tiles > 0 && ctx->phase_dw_out != nullptr) {
        // the strided layer's own weight gradient, straight from the scratch
        long long blocks = (static_cast<long long>(pairs / 4) + 255) / 256;
        if (blocks > ctx->sm_count * 16) blocks = ctx->sm_count * 16;
        ctx->phase_dw_done = true;
        return cuda_ok(launch_chained(tc3_dw_finish_phases_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, ctx->stream,
                                      acc, delta_p, ctx->phase_dw_out, static_cast<int>(s.Cout), ctx->phase_cin));
    }
    long long blocks = (static_cast<long long>(pairs) + 255) / 256;
    if (blocks > ctx->sm_count * 16) blocks = ctx->sm_count * 16;
    return cuda_ok(launch_chained(tc3_dw_finish_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, ctx->stream, acc,
                                  delta_p, dW, static_cast<long long>(pairs), static_cast<int>(s.Cin), static_cast<int>(cin_pad)));
}

}  // namespace dbp
