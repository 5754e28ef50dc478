// tcgen05 / mbarrier / cp.async wrappers shared by the tensor-core kernels (inline PTX for sm_100a).
#pragma once

#include "dbp_internal.cuh"

namespace dbp {
namespace tc {

constexpr long long kWaitCycles = 1000000000ll;     // a wait gives up after this many SM clocks

__device__ __forceinline__ unsigned smem_u32(const void *p) {
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(unsigned long long *bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One arrival for a whole warp: 256 threads arriving one by one on the same barrier word are
// 256 serialized shared-memory atomics per hand-over; after __syncwarp the lanes' earlier
// writes (and proxy fences) are ordered before lane 0's arrival.
__device__ __forceinline__ void warp_arrive(unsigned long long *bar) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}
// cp.async groups: a thread closes a group after the copies of one stage and later waits until
// at most `pending` newer groups are still in flight
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_pending(int pending) {
    switch (pending) {
        case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;   // fewer pending is always safe
    }
}
// arrival that fires when this thread's earlier cp.async copies have landed
__device__ __forceinline__ void mbar_arrive_on_cp_async(unsigned long long *bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Waits for the phase with the given parity. try_wait suspends the thread in hardware until the
// phase completes or a short system time limit passes, so a waiter wakes as soon as the barrier
// flips (a test_wait/nanosleep poll adds its sleep to every hand-over). Returns false, with the
// error flag set, when the phase did not complete within about half a second.
__device__ __forceinline__ bool mbar_try(unsigned addr, unsigned parity) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred P1;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 P1, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, P1;\n\t}"
        : "=r"(done) : "r"(addr), "r"(parity) : "memory");
    return done != 0;
}
__device__ __forceinline__ bool mbar_test(unsigned addr, unsigned parity) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred P1;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 P1, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, P1;\n\t}"
        : "=r"(done) : "r"(addr), "r"(parity) : "memory");
    return done != 0;
}
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, unsigned parity, int *err_flag,
                                          long long budget = kWaitCycles) {
    const unsigned addr = smem_u32(bar);
    if (mbar_test(addr, parity)) return true;
    const long long t0 = clock64();
    do {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_test(addr, parity)) return true;
    } while (clock64() - t0 <= budget);
    atomicExch(err_flag, 1);
    return false;
}
// The same wait, with the SM clocks it took added to `waited` (a measurement aid: the single
// threads that issue copies and MMAs report where they stood still).
__device__ __forceinline__ bool mbar_wait_timed(unsigned long long *bar, unsigned parity, int *err_flag, long long &waited) {
    if (mbar_test(smem_u32(bar), parity)) return true;
    const long long t0 = clock64();
    const bool ok = mbar_wait(bar, parity, err_flag);
    waited += clock64() - t0;
    return ok;
}
__device__ __forceinline__ void report_wait(unsigned long long *stats, int slot, long long cycles) {
    if (stats != nullptr && cycles > 0) atomicAdd(stats + slot, static_cast<unsigned long long>(cycles));
}
// One lane of a converged warp: lets a whole warp run a loop with warp-uniform control flow and
// operands (so that descriptor arithmetic can stay in uniform registers) while a single thread
// issues the copy, MMA or commit.
__device__ __forceinline__ bool elect_one() {
    unsigned pred;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(unsigned *dst_smem, int ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
}
__device__ __forceinline__ void tmem_dealloc(unsigned taddr, int ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols));
}
__device__ __forceinline__ void mma_bf16(unsigned tmem_d, unsigned long long adesc, unsigned long long bdesc,
                                         unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(unsigned long long *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(unsigned taddr, unsigned (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc, bool valid) {
    const int n = valid ? 16 : 0;   // src-size 0: the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(n) : "memory");
}

// 4- or 8-byte asynchronous copy (zero-filled when !valid); both addresses aligned to the size
template <int BYTES>
__device__ __forceinline__ void cp_async_small(void *smem_dst, const void *gsrc, bool valid) {
    static_assert(BYTES == 4 || BYTES == 8, "cp.async.ca copies 4, 8 or 16 bytes");
    const int n = valid ? BYTES : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;" ::"r"(smem_u32(smem_dst)), "l"(gsrc), "n"(BYTES), "r"(n) : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1; lbo/sbo in bytes.
// K-major operand: rows of 64 K-elements, 8-row groups sbo apart (lbo unused).
// MN-major operand: rows (one per k) of 64 MN-elements, 8-row groups sbo apart, 64-element
// MN groups lbo apart.
__device__ __forceinline__ unsigned long long make_desc(unsigned smem_addr, unsigned lbo, unsigned sbo) {
    unsigned long long d = 0;
    d |= static_cast<unsigned long long>((smem_addr & 0x3ffffu) >> 4);
    d |= static_cast<unsigned long long>((lbo >> 4) & 0x3fffu) << 16;
    d |= static_cast<unsigned long long>((sbo >> 4) & 0x3fffu) << 32;
    d |= 1ull << 46;     // version
    d |= 2ull << 61;     // SWIZZLE_128B
    return d;
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16.
__host__ __device__ constexpr unsigned make_idesc(int M, int N, bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (a_mn_major ? (1u << 15) : 0u) | (b_mn_major ? (1u << 16) : 0u) |
           (static_cast<unsigned>(N >> 3) << 17) | (static_cast<unsigned>(M >> 4) << 24);
}

// byte offset of 16-byte chunk `chunk` (0..7) of row `row` inside a 128-byte-swizzled panel
__device__ __forceinline__ unsigned swz(unsigned row, unsigned chunk) { return row * 128u + ((chunk ^ (row & 7u)) << 4); }

// four int8 codes packed in a word -> two words of packed bf16 (exact).
// byte ^ 0x80 = code + 128 as an unsigned byte; 0x4B0000xx read as a float is 2^23 + xx, so
// subtracting 2^23 + 128 leaves the code as a float whose top 16 bits are its bf16 pattern.
__device__ __forceinline__ void codes4_to_bf16(unsigned w, unsigned &lo, unsigned &hi) {
    const unsigned x = w ^ 0x80808080u;
    const float f0 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7650)) - 8388736.0f;
    const float f1 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7651)) - 8388736.0f;
    const float f2 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7652)) - 8388736.0f;
    const float f3 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7653)) - 8388736.0f;
    lo = __byte_perm(__float_as_uint(f0), __float_as_uint(f1), 0x7632);
    hi = __byte_perm(__float_as_uint(f2), __float_as_uint(f3), 0x7632);
}
// eight int8 codes (two words) -> eight bf16 (one 16-byte chunk)
__device__ __forceinline__ uint4 expand8(uint2 c) {
    uint4 o;
    codes4_to_bf16(c.x, o.x, o.y);
    codes4_to_bf16(c.y, o.z, o.w);
    return o;
}
__device__ __forceinline__ unsigned short code_to_bf16(int c) {
    return static_cast<unsigned short>(__float_as_uint(static_cast<float>(c)) >> 16);
}


}  // namespace tc
}  // namespace dbp

// ---------------------------------------------------------------- TMA (bulk tensor copies)
#include <cuda.h>

namespace dbp {
namespace tc {

// Arms a barrier with the byte count of the bulk copies that will complete on it (one arrival).
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Tiled loads of this GPU's own memory into this CTA's shared memory; completion is counted in
// bytes on `bar`. The innermost coordinate times the element size must be a multiple of 16.
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, unsigned long long *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int c0, int c1, int c2, unsigned long long *bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// Host: a bf16 tensor map with 128-byte swizzle. dims/box are in elements (innermost first),
// strides in bytes for dimensions 1.. (multiples of 16); the box's innermost extent is 64
// elements (128 bytes). Out-of-range elements read as zero. Returns false when the driver entry
// point is missing or rejects the description.
bool encode_map_bf16(CUtensorMap *map, const void *base, int rank, const unsigned long long *dims,
                     const unsigned long long *strides_bytes, const unsigned *box);
// Host: an fp32 tensor map without swizzle (a box lands / leaves as plain rows of box[0] floats);
// used for reductions into global memory.
bool encode_map_f32_rows(CUtensorMap *map, const void *base, int rank, const unsigned long long *dims,
                         const unsigned long long *strides_bytes, const unsigned *box);

// The same with 128-byte swizzle: the box's innermost extent is 32 floats.
bool encode_map_f32_sw128(CUtensorMap *map, const void *base, int rank, const unsigned long long *dims,
                          const unsigned long long *strides_bytes, const unsigned *box);

// Adds a box of fp32 values in shared memory (plain rows, or swizzled as the tensor map says) into global memory through the copy
// engine: the additions happen at the L2 with whole-line requests. Elements outside the tensor are
// skipped. The issuing thread closes a group after its reductions and waits until the engine has
// read the shared memory before that memory is reused (or the CTA exits).
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap *map, int c0, int c1, const void *src) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(smem_u32(src)) : "memory");
}
// Stores a box from shared memory (laid out as the tensor map's swizzle says) into global memory;
// the part of the box outside the tensor is not written. Group and wait rules as for the reduction.
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, int c0, int c1, int c2, const void *src) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(src)) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// all but the three most recent groups of this thread have been read
__device__ __forceinline__ void bulk_wait_read_but3() { asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory"); }

}  // namespace tc
}  // namespace dbp
