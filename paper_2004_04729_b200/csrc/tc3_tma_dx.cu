// Input gradient of 3x3 convolutions (stride 1, pad 1) on the tensor cores, both operands brought
// in by tiled copies (Eq. (qda), "analogous for convolutional layers"):
//   dX[b][ci][y][x] = Delta * sum_(co,ky,kx) q[b][co][y+1-ky][x+1-kx] * W[co][ci][ky][kx]
//
// The quantizer has written the codes position-major, [b][y][x][co] in bf16, so a patch of
// (Ht+2) x (W+2) positions x 64 output channels is ONE 4-D tiled copy whose out-of-image rows and
// columns the copy engine fills with zeros: the convolution's zero padding costs nothing. In
// shared memory the patch is a K-major operand, one 128-byte row of 64 channels per position,
// rows numbered r = yy * (W+2) + xx. The output position (y, x) of the patch is accumulator column
// n = (y-y0) * (W+2) + x, and the code a tap (ky, kx) needs for it sits in row
// n + (2-ky) * (W+2) + (2-kx): a tap is only a different start row of the same operand (the 128-byte
// swizzle is a function of the shared-memory address, so a descriptor may start at any row). The
// two columns per image row that belong to the halo (x = W, W+1) are computed and thrown away.
// Small images (the whole image in one patch) are taken several at a time along the same row space.
//
//   A = weights of one tap [64 co][128 ci]  (M = input channels, MN-major; from W re-laid as [co][tap][ci])
//   B = code patch         [rows][64 co]    (N = up to 256 patch positions, K-major)
//   K = (64-channel block of co) x (nine taps), four MMAs of 16 channels each
//
// A CTA is persistent over (patch, 128-channel block of ci) tiles. Warp 0 copies code patches,
// warp 1 copies weight tiles, warp 2 issues the MMAs into one of two accumulators in tensor memory,
// warps 4-19 drain the other one: scale by Delta, convert, compact the valid columns into a
// shared staging block [ci][positions] and write whole runs of consecutive positions per channel.
// Every wait is bounded.
#include "tc_common.cuh"

namespace dbp {

namespace {

using namespace tc;

constexpr int kThreadsX = 20 * 32;               // copy, copy, MMA, spare, sixteen epilogue warps
constexpr int kWPanel = 8192;                    // [64 co][64 ci] bf16
constexpr int kMaxQ = 2;                         // code patches in flight
constexpr int kMaxW = 18;                        // weight slots (ring, or all of them when they stay resident)
constexpr int kAccCols = 256;
constexpr int kEpiThreads = 512;

struct Dx3T {
    const float *delta_p;
    void *dX;
    int dx_f32;
    int B, Cin, Cout, H, W, Wp;
    int Ht;                       // image rows per patch
    int nb;                       // images per patch (> 1 only when Ht == H)
    int tiles_y;                  // patches per image (nb == 1)
    int img_rows;                 // (Ht + 2) * Wp: patch rows per image
    int N;                        // accumulator columns in use (multiple of 16)
    int q_bytes;                  // bytes of one patch buffer (multiple of 1024)
    int q_tx;                     // bytes one patch copy delivers
    int ncb;                      // 64-channel blocks of co
    int ci_tiles;
    long long pos_tiles, ntiles;
    int a_panels;                 // 64-channel panels of ci per weight tile (1 or 2)
    int ntaps;                    // 9, or 18 for fp32 weights split into two bf16 pieces (taps 9-17: the low pieces)
    int es;                       // bytes per element of dX (2 or 4)
    int G;                        // taps per weight slot (one hand-over): 9, 3 or 1
    int w_slot;                   // bytes of a weight slot: G * a_panels * 8 KB
    int nq, nw;                   // ring sizes
    int resident;                 // the weights of all taps and co blocks stay in shared memory (one ci block)
    int run;                      // Ht * W: staged positions per image
    int pitch;                    // bytes per channel row of the staging block (an odd number of words)
    int pairs;                    // W even: columns are staged two at a time
    int phase_cin;                // > 0: the layer is a stride-2 layer on phase images (channel block ph * phase_cin ...
                                  // holds phase ph = 2 py + px); a phase's weights are zero outside the taps
                                  // ky in {1} (py = 0) or {0, 1} (py = 1), kx likewise, and those taps are skipped
    int *err_flag;
    unsigned long long *stats;    // wait counters (may be null)
};

struct PipeX {
    unsigned long long q_full[kMaxQ], q_empty[kMaxQ], w_full[kMaxW], w_empty[kMaxW], acc_full[2], acc_empty[2];
    unsigned tmem_base;
};

__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, int c0, int c1, int c2, int c3,
                                            unsigned long long *bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// Barrier over the epilogue threads that also tells every one of them whether all of them are
// still fine: a thread whose bounded wait ran out arrives like the others, so nobody is left waiting.
__device__ __forceinline__ bool epilogue_all(bool mine) {
    unsigned r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, %2, p;\n\t"
        "selp.b32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"(mine ? 1u : 0u), "n"(kEpiThreads) : "memory");
    return r != 0;
}

__global__ void __launch_bounds__(kThreadsX, 1)
tc3_tma_dx_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_w, const Dx3T p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char *q_s = smem;                                   // nq code patches
    unsigned char *w_s = q_s + p.nq * p.q_bytes;                 // nw weight slots
    short *s_off = reinterpret_cast<short *>(w_s + p.nw * p.w_slot);   // column -> staged position (or -1), 256 entries
    unsigned char *stage = reinterpret_cast<unsigned char *>(s_off) + 512;   // [128 ci][pitch]
    __shared__ PipeX pipe;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxQ; ++s) { mbar_init(&pipe.q_full[s], 1); mbar_init(&pipe.q_empty[s], 1); }
        for (int s = 0; s < kMaxW; ++s) { mbar_init(&pipe.w_full[s], 1); mbar_init(&pipe.w_empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&pipe.acc_full[a], 1); mbar_init(&pipe.acc_empty[a], kEpiThreads / 32); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_w);
    }
    if (warp == 2) tmem_alloc(&pipe.tmem_base, 2 * kAccCols);
    // which accumulator columns hold an output, and where it goes in a channel's staged run
    if (threadIdx.x >= 128 && threadIdx.x < 384) {
        const int n = threadIdx.x - 128;
        const int img = n / p.img_rows, rem = n - img * p.img_rows;
        const int yy = rem / p.Wp, xx = rem - yy * p.Wp;
        s_off[n] = (n < p.N && img < p.nb && yy < p.Ht && xx < p.W) ? static_cast<short>(img * p.run + yy * p.W + xx) : static_cast<short>(-1);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = pipe.tmem_base;
    // everything above touched only this CTA's shared and tensor memory
    chain_wait();
    chain_release();

    // tile t -> (patch, ci block); patch -> first image and first image row
    auto tile_of = [&](long long t, int &ci0, int &b0, int &y0) {
        const long long pt = t / p.ci_tiles;
        ci0 = static_cast<int>(t - pt * p.ci_tiles) * 128;
        if (p.nb == 1) {
            b0 = static_cast<int>(pt / p.tiles_y);
            y0 = static_cast<int>(pt - static_cast<long long>(b0) * p.tiles_y) * p.Ht;
        } else {
            b0 = static_cast<int>(pt) * p.nb;
            y0 = 0;
        }
    };
    const int slots_per_cb = p.ntaps / p.G;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            unsigned parity = 1;                   // a fresh barrier passes a wait on the previous phase
            bool ok = true;
            long long waited = 0;
            for (long long t = blockIdx.x; t < p.ntiles && ok; t += gridDim.x) {
                int ci0, b0, y0;
                tile_of(t, ci0, b0, y0);
                for (int c = 0; c < p.ncb && ok; ++c) {
                    ok = mbar_wait_timed(&pipe.q_empty[s], parity, p.err_flag, waited);
                    if (!ok) break;
                    mbar_expect_tx(&pipe.q_full[s], static_cast<unsigned>(p.q_tx));
                    tma_load_4d(q_s + s * p.q_bytes, &map_q, c * 64, -1, y0 - 1, b0, &pipe.q_full[s]);
                    if (++s == p.nq) { s = 0; parity ^= 1u; }
                }
            }
            report_wait(p.stats, 3, waited);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int s = 0;
            unsigned parity = 1;
            bool ok = true;
            const unsigned w_tx = static_cast<unsigned>(p.w_slot);
            long long waited = 0;
            for (long long t = blockIdx.x; t < p.ntiles && ok; t += gridDim.x) {
                int ci0, b0, y0;
                tile_of(t, ci0, b0, y0);
                for (int c = 0; c < p.ncb && ok; ++c)
                    for (int g = 0; g < slots_per_cb; ++g) {
                        if (!p.resident) {
                            ok = mbar_wait_timed(&pipe.w_empty[s], parity, p.err_flag, waited);
                            if (!ok) break;
                        }
                        mbar_expect_tx(&pipe.w_full[s], w_tx);
                        // one arrival for the whole slot: the taps' panels are separate copies under one barrier
                        unsigned char *dst = w_s + s * p.w_slot;
                        for (int gg = 0; gg < p.G; ++gg)
                            for (int h = 0; h < p.a_panels; ++h, dst += kWPanel)
                                tma_load_3d(dst, &map_w, ci0 + 64 * h, g * p.G + gg, c * 64, &pipe.w_full[s]);
                        if (++s == p.nw) { s = 0; parity ^= 1u; }
                    }
                if (p.resident) break;             // one ci block: every tile uses the same weights (all slots are loaded now)
            }
            report_wait(p.stats, 4, waited);
        }
    } else if (warp == 2) {
        {   // the whole warp runs the loop (uniform control flow and operands); one elected lane issues
            const unsigned idesc = make_idesc(128, p.N, true, false);
            // start row of tap (ky, kx) inside the patch is (2 - ky) Wp + (2 - kx); as a descriptor offset
            // (16-byte units, 8 per row) it starts at tap_first and moves by -8, -8, +16 - 8 Wp, ...
            const int tap_first = (2 * p.Wp + 2) * 8, tap_wrap = (2 - p.Wp) * 8;
            const unsigned a_tap = static_cast<unsigned>(p.a_panels * kWPanel) >> 4;     // one tap further inside a slot
            int qs = 0, ws = 0;
            unsigned qpar = 0, wpar = 0;
            bool ok = true;
            long long it = 0;
            long long wq = 0, ww = 0, wa = 0;
            const long long born = clock64();
            for (long long t = blockIdx.x; t < p.ntiles && ok; t += gridDim.x, ++it) {
                const int slot = static_cast<int>(it & 1);
                const unsigned uses = static_cast<unsigned>(it >> 1);
                ok = __all_sync(0xffffffffu, mbar_wait_timed(&pipe.acc_empty[slot], (uses & 1u) ^ 1u, p.err_flag, wa));
                if (!ok) break;
                tc_fence_after();
                const unsigned tmem_d = tmem_base + slot * kAccCols;
                unsigned acc_on = 0u;
                int live_y = 7, live_x = 7;                // bit t: taps with coordinate t carry non-zero weights
                if (p.phase_cin > 0) {
                    const int ph = static_cast<int>(t % p.ci_tiles) * 128 / p.phase_cin;
                    live_y = (ph & 2) ? 3 : 2;
                    live_x = (ph & 1) ? 3 : 2;
                }
                if (p.resident) { ws = 0; wpar = 0; }      // completed barriers stay passable on parity 0
                for (int c = 0; c < p.ncb && ok; ++c) {
                    ok = __all_sync(0xffffffffu, mbar_wait_timed(&pipe.q_full[qs], qpar, p.err_flag, wq));
                    if (!ok) break;
                    tc_fence_after();
                    const unsigned long long bd0 = make_desc(smem_u32(q_s + qs * p.q_bytes), 16, 1024);
                    int toff = tap_first, kx = 0, ky = 0;
                    for (int g = 0; g < slots_per_cb && ok; ++g) {
                        ok = __all_sync(0xffffffffu, mbar_wait_timed(&pipe.w_full[ws], wpar, p.err_flag, ww));
                        if (!ok) break;
                        tc_fence_after();
                        // with one panel of ci (Cin <= 64) the upper 64 rows of the MMA re-read the same panel (their
                        // results are never stored) instead of whatever follows the slot
                        unsigned long long ad = make_desc(smem_u32(w_s + ws * p.w_slot), p.a_panels == 2 ? kWPanel : 0, 1024);
                        for (int gg = 0; gg < p.G; ++gg, ad += a_tap) {
                            const unsigned long long bd = bd0 + static_cast<unsigned>(toff);
                            const bool live = ((live_y >> ky) & 1) && ((live_x >> kx) & 1);
                            if (kx == 2) {
                                kx = 0;
                                toff += tap_wrap;
                                if (++ky == 3) { ky = 0; toff = tap_first; }      // the second piece's taps start over
                            } else {
                                ++kx;
                                toff -= 8;
                            }
                            if (!live) continue;
                            if (elect_one()) {
#pragma unroll
                                for (int k = 0; k < 4; ++k)   // 16 co: 16 rows of A (2048 bytes), 32 bytes along a row of B
                                    mma_bf16(tmem_d, ad + 128 * k, bd + 2 * k, idesc, k ? 1u : acc_on);
                            }
                            acc_on = 1u;
                        }
                        if (!p.resident && elect_one()) mma_commit(&pipe.w_empty[ws]);
                        if (++ws == p.nw) { ws = 0; wpar ^= 1u; }
                    }
                    if (ok && elect_one()) mma_commit(&pipe.q_empty[qs]);
                    if (++qs == p.nq) { qs = 0; qpar ^= 1u; }
                }
                if (ok && elect_one()) mma_commit(&pipe.acc_full[slot]);
            }
            if (lane == 0) {
                report_wait(p.stats, 0, wq);
                report_wait(p.stats, 1, ww);
                report_wait(p.stats, 2, wa);
                report_wait(p.stats, 6, clock64() - born);
                report_wait(p.stats, 7, 1);
            }
        }
    } else if (warp >= 4) {
        // epilogue: TMEM lane = input channel, column = patch position. Warp (q, part): lane quarter q,
        // one quarter of the 32-column chunks.
        const int ew = warp - 4, q = ew & 3, part = ew >> 2;
        const int et = threadIdx.x - 128;                           // 0 .. 511
        const float delta = *p.delta_p;
        const int nchunk = (p.N + 31) >> 5, ch_lo = (nchunk * part + 3) >> 2, ch_hi = (nchunk * (part + 1) + 3) >> 2;
        const int HW = p.H * p.W;
        bool ok = true;
        long long it = 0;
        long long we = 0;
        for (long long t = blockIdx.x; t < p.ntiles; t += gridDim.x, ++it) {
            const int slot = static_cast<int>(it & 1);
            const unsigned uses = static_cast<unsigned>(it >> 1);
            int ci0, b0, y0;
            tile_of(t, ci0, b0, y0);
            ok = epilogue_all(mbar_wait_timed(&pipe.acc_full[slot], uses & 1u, p.err_flag, we));
            if (!ok) break;                                          // the same decision in every epilogue thread
            tc_fence_after();
            const int ci_l = q * 32 + lane, ci = ci0 + ci_l;
            const int rows_valid = p.H - y0 < p.Ht ? p.H - y0 : p.Ht;
            // ---- phase A: accumulator -> staging block (rows of bf16 or fp32 values per channel)
            if (ci0 + q * 32 < p.Cin) {                              // warp-uniform: some of my 32 channels exist
                unsigned char *row = stage + ci_l * p.pitch;
                for (int chn = ch_lo; chn < ch_hi; ++chn) {
                    unsigned v[32];
                    tmem_ld32(tmem_base + (static_cast<unsigned>(q * 32) << 16) + slot * kAccCols + chn * 32, v);
                    const short *off = s_off + chn * 32;
                    // the 32 table entries of the chunk as four 16-byte loads
                    const uint4 *tp = reinterpret_cast<const uint4 *>(off);
                    const uint4 t0 = tp[0], t1 = tp[1], t2 = tp[2], t3 = tp[3];
                    const unsigned tw[16] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w,
                                             t2.x, t2.y, t2.z, t2.w, t3.x, t3.y, t3.z, t3.w};
                    if (p.es == 4) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int o = static_cast<int>(static_cast<short>((tw[j >> 1] >> (16 * (j & 1))) & 0xffffu));
                            if (o >= 0) *reinterpret_cast<float *>(row + 4 * o) = __uint_as_float(v[j]) * delta;
                        }
                    } else if (p.pairs) {
                        // entry 2i tells where columns 2i, 2i+1 go
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int o = static_cast<int>(static_cast<short>(tw[i] & 0xffffu));
                            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * i]) * delta, __uint_as_float(v[2 * i + 1]) * delta);
                            if (o >= 0) *reinterpret_cast<unsigned *>(row + 2 * o) = *reinterpret_cast<const unsigned *>(&h);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int o = static_cast<int>(static_cast<short>((tw[j >> 1] >> (16 * (j & 1))) & 0xffffu));
                            if (o >= 0) *reinterpret_cast<__nv_bfloat16 *>(row + 2 * o) = __float2bfloat16_rn(__uint_as_float(v[j]) * delta);
                        }
                    }
                }
            }
            // the accumulator is free once every epilogue warp has read its part
            tc_fence_before();
            warp_arrive(&pipe.acc_empty[slot]);
            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
            // ---- phase B: staging block -> dX, runs of consecutive positions per (image, channel)
            {
                const int ncv = p.Cin - ci0 < 128 ? p.Cin - ci0 : 128;
                const int len = rows_valid * p.W;                    // elements per run
                unsigned char *dst0 = static_cast<unsigned char *>(p.dX);
                const bool words = p.es == 4 || p.pairs;             // whole 32-bit words
                const int nwords = p.es == 4 ? len : len >> 1;
                for (int img = 0; img < p.nb && b0 + img < p.B; ++img) {
                    for (int r = et >> 5; r < ncv; r += kEpiThreads / 32) {
                        const unsigned char *src = stage + r * p.pitch + p.es * img * p.run;
                        unsigned char *dst = dst0 + ((static_cast<long long>(b0 + img) * p.Cin + ci0 + r) * HW + y0 * p.W) * p.es;
                        if (words) {
                            for (int i = lane; i < nwords; i += 32)
                                reinterpret_cast<unsigned *>(dst)[i] = reinterpret_cast<const unsigned *>(src)[i];
                        } else {
                            for (int i = lane; i < len; i += 32)
                                reinterpret_cast<unsigned short *>(dst)[i] = reinterpret_cast<const unsigned short *>(src)[i];
                        }
                    }
                }
            }
            // the staging block is rewritten by the next tile only after everyone is done reading it
            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
        }
        if (et == 0) report_wait(p.stats, 5, we);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        __syncwarp();
        tmem_dealloc(tmem_base, 2 * kAccCols);
    }
}

// weights [Cout][Cin][3][3] -> [Cout][9][Cin] (the tap's [co][ci] matrix with ci contiguous)
__global__ void __launch_bounds__(256)
w_taps_bf16_kernel(const unsigned short *__restrict__ W, unsigned short *__restrict__ out, long long Cout, long long Cin) {
    chain_wait();
    chain_release();
    const long long n = Cout * Cin * 9;
    for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += gridDim.x * 256ll) {
        const long long ci = i % Cin, t = (i / Cin) % 9, co = i / (Cin * 9);
        out[i] = __ldg(W + (co * Cin + ci) * 9 + t);
    }
}

// fp32 weights -> [Cout][18][Cin] bf16: taps 0-8 hold the values rounded to bf16, taps 9-17 what that
// rounding left over, rounded to bf16 again. The sum of the two pieces differs from the fp32 value by
// at most 2^-18 of it, and a code times a piece is exact in the fp32 accumulator.
__global__ void __launch_bounds__(256)
w_taps_split_kernel(const float *__restrict__ W, __nv_bfloat16 *__restrict__ out, long long Cout, long long Cin) {
    chain_wait();
    chain_release();
    const long long n = Cout * Cin * 9;
    for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += gridDim.x * 256ll) {
        const long long ci = i % Cin, t = (i / Cin) % 9, co = i / (Cin * 9);
        const float w = __ldg(W + (co * Cin + ci) * 9 + t);
        const __nv_bfloat16 hi = __float2bfloat16_rn(w);
        const __nv_bfloat16 lo = __float2bfloat16_rn(w - __bfloat162float(hi));
        out[(co * 18 + t) * Cin + ci] = hi;
        out[(co * 18 + 9 + t) * Cin + ci] = lo;
    }
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

}  // namespace

// Shapes the TMA-fed 3x3 kernels take: channel counts that keep every row of the position-major
// codes, of the re-laid weights and of the activations on 16-byte boundaries. fp32 operands are
// split into two bf16 pieces each (the codes are exact in bf16), so they take the same kernels.
bool tc3_tma_supported(const ConvShape &s, int io) {
    return (io == DBP_BF16 || io == DBP_F32) && s.k == 3 && s.Cin % 8 == 0 && s.Cout % 8 == 0 && s.W >= 1 && s.W <= 62 &&
           s.H <= 4096 && s.B * s.H * s.W < (1ll << 30);
}

// The weight-gradient kernel alone also takes fp32 layers whose input channel count is no multiple of 8 (a
// network's first layer): its activations are re-written channel-padded anyway.
bool tc3_tma_dw_supported(const ConvShape &s, int io) {
    if (tc3_tma_supported(s, io)) return true;
    ConvShape t = s;
    t.Cin = (s.Cin + 7) / 8 * 8;
    return io == DBP_F32 && tc3_tma_supported(t, io);
}

// DBP_EUNSUPPORTED: the shape does not fit (the caller uses another kernel)
int launch_tc3_tma_dx(dbp_ctx *ctx, const void *codes_nhwc, const void *W, int io, const float *delta_p,
                      const ConvShape &s, void *dX, bool dx_bf16, int *err_flag, bool weights_ready) {
    if (!tc3_tma_supported(s, io)) return DBP_EUNSUPPORTED;
    Dx3T p{};
    p.delta_p = delta_p; p.dX = dX; p.dx_f32 = dx_bf16 ? 0 : 1;
    p.es = dx_bf16 ? 2 : 4;
    p.ntaps = io == DBP_F32 ? 18 : 9;
    p.B = static_cast<int>(s.B); p.Cin = static_cast<int>(s.Cin); p.Cout = static_cast<int>(s.Cout);
    p.H = static_cast<int>(s.H); p.W = static_cast<int>(s.W); p.Wp = p.W + 2;
    p.err_flag = err_flag;
    p.stats = ctx->wait_stats;
    p.phase_cin = (ctx->phase_cin > 0 && ctx->phase_cin % 128 == 0 && s.Cin == 4ll * ctx->phase_cin) ? ctx->phase_cin : 0;
    p.ncb = (p.Cout + 63) / 64;
    p.ci_tiles = (p.Cin + 127) / 128;
    p.a_panels = p.Cin <= 64 ? 1 : 2;
    const size_t tap_bytes = static_cast<size_t>(p.a_panels) * kWPanel;
    const size_t budget = 227 * 1024 - 2048;
    // patch geometry: the cheapest of the candidates by (waves of one CTA per SM) x (columns per tile;
    // a narrow MMA takes as long to issue as one of about 200 columns takes to run). A candidate must
    // leave room for its two patch buffers, its staging block and at least three weight taps.
    const int sms = ctx->sm_count;
    int best_ht = 0, best_nb = 1;
    double best_cost = 1e300;
    auto patch_bytes = [&](int ht, int nb, int n) {
        const int img_rows = (ht + 2) * p.Wp, rows_read = n + 2 * p.Wp + 2;
        return round_up((rows_read > img_rows * nb ? rows_read : img_rows * nb) * 128, 1024);
    };
    auto stage_pitch = [&](int ht, int nb) {
        int pitch = round_up(nb * ht * p.W * p.es, 4);
        if ((pitch / 4) % 2 == 0) pitch += 4;      // an odd number of words: see below
        return pitch;
    };
    auto consider = [&](int ht, int nb) {
        const int img_rows = (ht + 2) * p.Wp;
        const int last = (nb - 1) * img_rows + (ht - 1) * p.Wp + p.W - 1;     // last column that holds an output
        const int n = round_up(last + 1, 16);
        if (n > 256 || img_rows * nb > 1024) return;
        if (2 * static_cast<size_t>(patch_bytes(ht, nb, n)) + 128 * static_cast<size_t>(stage_pitch(ht, nb)) + 1536 + 3 * tap_bytes > budget) return;
        const long long tiles = nb == 1 ? static_cast<long long>(p.B) * ((p.H + ht - 1) / ht) : (p.B + nb - 1) / nb;
        const long long waves = (tiles * p.ci_tiles + sms - 1) / sms;
        const double cost = static_cast<double>(waves) * ((n < 208 ? 208 : n) + 64);      // an MMA takes >= ~100 clocks to issue
        if (cost < best_cost) { best_cost = cost; best_ht = ht; best_nb = nb; }
    };
    for (int ht = 1; ht <= p.H; ++ht) consider(ht, 1);
    for (int nb = 2; nb <= 16 && nb <= p.B; ++nb) consider(p.H, nb);
    if (best_ht == 0) return DBP_EUNSUPPORTED;
    p.Ht = best_ht; p.nb = best_nb;
    p.tiles_y = (p.H + p.Ht - 1) / p.Ht;
    p.img_rows = (p.Ht + 2) * p.Wp;
    p.N = round_up((p.nb - 1) * p.img_rows + (p.Ht - 1) * p.Wp + p.W, 16);
    p.pos_tiles = p.nb == 1 ? static_cast<long long>(p.B) * p.tiles_y : (p.B + p.nb - 1) / p.nb;
    p.ntiles = p.pos_tiles * p.ci_tiles;
    p.q_tx = p.img_rows * p.nb * 128;
    // the last tap of the last column reads row N - 1 + 2 Wp + 2; rows past the copied patch hold
    // stale data, which only reaches columns that are never stored
    p.q_bytes = patch_bytes(p.Ht, p.nb, p.N);
    p.run = p.Ht * p.W;
    // an odd number of 32-bit words per row: the 32 channels of a warp hit 32 different banks when
    // they stage the same position
    p.pitch = stage_pitch(p.Ht, p.nb);
    p.pairs = p.W % 2 == 0 ? 1 : 0;
    const size_t stage_bytes = static_cast<size_t>(128) * p.pitch;
    // Weights: a slot holds G taps and is handed over with one barrier (the hand-over, not the copy
    // instruction, is what costs time). With one ci block and room for all taps of all co blocks they
    // are loaded once and stay; otherwise they stream through a ring of slots.
    p.nq = kMaxQ;
    const size_t fixed = static_cast<size_t>(p.nq) * p.q_bytes + stage_bytes + 512 + 1024;
    const size_t room = budget - fixed;
    const int slots_all = p.ncb * (p.ntaps / 9);
    if (p.ci_tiles == 1 && slots_all <= kMaxW && static_cast<size_t>(slots_all) * 9 * tap_bytes <= room) {
        p.resident = 1; p.G = 9; p.nw = slots_all;
    } else if (room >= 2 * 3 * tap_bytes) {
        p.resident = 0; p.G = 3; p.nw = static_cast<int>(room / (3 * tap_bytes));
    } else {
        p.resident = 0; p.G = 1; p.nw = static_cast<int>(room / tap_bytes);
    }
    if (p.nw > kMaxW) p.nw = kMaxW;
    p.w_slot = static_cast<int>(p.G * tap_bytes);
    const size_t smem = fixed + static_cast<size_t>(p.nw) * p.w_slot;

    // re-laid weights
    const size_t wb = sizeof(__nv_bfloat16) * static_cast<size_t>(s.Cout) * s.Cin * p.ntaps;
    int rc = ws_reserve(ctx, ctx->w_taps, wb);
    if (rc) return rc;
    if (!weights_ready) {
        long long blocks = (static_cast<long long>(s.Cout) * s.Cin * 9 + 255) / 256;
        if (blocks > sms * 8) blocks = sms * 8;
        if (io == DBP_F32)
            rc = cuda_ok(launch_chained(w_taps_split_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, ctx->stream,
                                        static_cast<const float *>(W), static_cast<__nv_bfloat16 *>(ctx->w_taps.ptr), s.Cout, s.Cin));
        else
            rc = cuda_ok(launch_chained(w_taps_bf16_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, ctx->stream,
                                        static_cast<const unsigned short *>(W), static_cast<unsigned short *>(ctx->w_taps.ptr),
                                        s.Cout, s.Cin));
        if (rc) return rc;
    }
    CUtensorMap map_q, map_w;
    {
        const unsigned long long dims[4] = {static_cast<unsigned long long>(s.Cout), static_cast<unsigned long long>(s.W),
                                            static_cast<unsigned long long>(s.H), static_cast<unsigned long long>(s.B)};
        const unsigned long long str[3] = {static_cast<unsigned long long>(s.Cout) * 2,
                                           static_cast<unsigned long long>(s.Cout) * 2 * s.W,
                                           static_cast<unsigned long long>(s.Cout) * 2 * s.W * s.H};
        const unsigned box[4] = {64, static_cast<unsigned>(p.Wp), static_cast<unsigned>(p.Ht + 2), static_cast<unsigned>(p.nb)};
        if (!encode_map_bf16(&map_q, codes_nhwc, 4, dims, str, box)) return fail_cuda("tensor map of the code patches");
    }
    {
        const unsigned long long dims[3] = {static_cast<unsigned long long>(s.Cin), static_cast<unsigned long long>(p.ntaps),
                                            static_cast<unsigned long long>(s.Cout)};
        const unsigned long long str[2] = {static_cast<unsigned long long>(s.Cin) * 2,
                                           static_cast<unsigned long long>(s.Cin) * 2 * p.ntaps};
        const unsigned box[3] = {64, 1, 64};
        if (!encode_map_bf16(&map_w, ctx->w_taps.ptr, 3, dims, str, box)) return fail_cuda("tensor map of the weights");
    }
    if (cudaFuncSetAttribute(tc3_tma_dx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return fail_cuda("shared memory size");
    const long long grid = p.ntiles < sms ? p.ntiles : sms;
    return cuda_ok(launch_chained(tc3_tma_dx_kernel, dim3(static_cast<unsigned>(grid)), dim3(kThreadsX), smem, ctx->stream,
                                  map_q, map_w, p));
}

}  // namespace dbp
