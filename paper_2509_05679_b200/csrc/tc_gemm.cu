// Tensor-core kernels for sm_100a: implicit-GEMM convolution / linear layers on tcgen05.mma with
// accumulators in tensor memory, operands staged in shared memory by TMA (cp.async.bulk.tensor,
// 128-byte swizzle), a 3-4 stage mbarrier pipeline, and warp-specialised roles:
//   warp 0 : TMA producer (the whole warp runs the loop, one elected lane issues the copies)
//   warp 1 : tensor-memory allocation, MMA issue (same scheme), deallocation
//   warps 2-5 (or 2-9) : epilogue (tcgen05.ld -> registers -> bf16 tile in shared memory -> TMA store)
//
// Two kernels:
//   km_kernel  (forward and input-gradient): D[pixel][c_out] = sum_{tap, c} A[pixel + tap][c] * B[c_out][tap, c]
//              A is an NHWC activation read through a 4-D tensor map (one box per filter tap, shifted by
//              the tap; out-of-bounds elements are zero-filled, which is the padding), B a K-major weight
//              matrix.  Both operands are K-major in shared memory.
//   wg_kernel  (weight gradient): D[(tap, c_in)][c_out] = sum_{pixel} X[pixel + tap][c_in] * dY[pixel][c_out]
//              The contraction runs over pixels = worker x batch x H x W, so the average over workers is
//              part of the contraction.  Both operands are MN-major in shared memory (channel contiguous).
//              Split over pixels across CTAs; partial sums are reduced in a fixed order by a second kernel.
// Every wait on an mbarrier is bounded; a wait that gives up sets an error word and the CTA leaves
// through the common exit (tensor memory is always released).
#include "tc_gemm.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cstdio>
#include <cstring>

namespace fdg {
namespace tc {

typedef __nv_bfloat16 bf16;

constexpr int BLOCK_M = 128;      // rows of an accumulator tile (= tensor-memory lanes)
constexpr int BLOCK_K = 64;       // bf16 elements per 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 192;
constexpr long long WAIT_CYCLES = 4000000000LL;   // ~2 s at 2 GHz
constexpr unsigned EPI_SLEEP_NS = 200;            // pause between polls of a long wait (epilogue warps)

// ------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok;
}
// Bounded wait: false (and *err set) if the phase did not complete within WAIT_CYCLES.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* err, int code) {
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > WAIT_CYCLES) { atomicCAS(err, 0, code); return false; }
    }
    return true;
}
// The same for whole warps that wait long (the epilogue warps wait for a tile's MMAs): sleeping between polls keeps
// them out of the issue slots and the barrier unit that the single producer and MMA threads depend on.
__device__ __forceinline__ bool mbar_wait_sleep(uint64_t* bar, uint32_t parity, int* err, int code) {
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        __nanosleep(EPI_SLEEP_NS);
        if (clock64() - t0 > WAIT_CYCLES) { atomicCAS(err, 0, code); return false; }
    }
    return true;
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* tm, uint64_t* bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, uint64_t* bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* tm) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// the mbarrier receives one arrival when all previously issued MMAs of this thread have completed
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// ---- forms that take 32-bit shared-memory addresses.  The TMA-producer and MMA-issuer loops run in ONE thread each, so
// every instruction in them is on the critical path (measured: a k-block of four 128x256x16 MMAs is 512 cycles of
// tensor-pipe work, and a loop body that rebuilt descriptors and divided by the stage count took about 900): the
// loops keep running addresses and phases and add constants to descriptor words instead.
__device__ __forceinline__ bool mbar_wait_a(uint32_t bar, uint32_t parity, int* err, int code) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
    long long t0 = clock64();
    for (;;) {
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if (clock64() - t0 > WAIT_CYCLES) { atomicCAS(err, 0, code); return false; }
    }
}
__device__ __forceinline__ void mbar_expect_tx_a(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_4d_a(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_2d_a(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// descriptors given as (low word, shared high word): only the address field in the low word changes between MMAs
template <bool PAIR>
__device__ __forceinline__ void umma_bf16_w(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t accumulate) {
    if (PAIR)
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                     "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}"
                     ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
                     ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate) : "memory");
}
template <bool PAIR>
__device__ __forceinline__ void umma_commit_a(uint32_t bar) {
    if (PAIR)
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(bar), "h"((uint16_t)3) : "memory");
    else
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// One lane of a converged warp.  The producer and MMA loops are executed by all 32 lanes, so that loop state stays
// warp-uniform, and only the asynchronous instructions themselves sit behind this predicate.
__device__ __forceinline__ uint32_t elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred P1;\n\t.reg .b32 dummy;\n\telect.sync dummy|P1, 0xffffffff;\n\tselp.u32 %0, 1, 0, P1;\n\t}" : "=r"(pred));
    return pred;
}
// shared -> global tile store (bulk async group of the issuing thread)
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* tm, uint32_t src, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(tm), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ---- CTA pairs (cluster of two, tcgen05 cta_group::2): one MMA of 256 rows, each CTA holds its 128 rows of A and of
// the accumulator and half of B's rows, so every SM reads only half of B from its shared memory.
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
// address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank)); return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA loads whose completion is signalled on an mbarrier of either CTA of the pair (`bar` is a cluster address)
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// executed by the same warp of both CTAs of the pair
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// issued by one thread of the pair's first CTA; descriptors address the same offsets in both CTAs' shared memory
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// one arrival on the mbarrier at this offset in BOTH CTAs once all MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((uint16_t)3) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns -> 32 registers per thread (thread = lane)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// the same without the wait: two of these fetch 64 columns, then tmem_ld_wait()
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t* v) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
//   K-major operand  [rows][64 bf16]: 8-row groups are `sbo` bytes apart (1024); lbo unused.
//   MN-major operand [k rows][64 bf16 of the M/N axis]: groups of 8 k-rows are `sbo` bytes apart (1024),
//                    consecutive 64-element chunks of the M/N axis are `lbo` bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor for kind::f16: fp32 accumulator, bf16 A and B, dense.
__device__ __forceinline__ uint32_t make_idesc(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ uint8_t* align1024(uint8_t* p) {
    return (uint8_t*)(((uintptr_t)p + 1023) & ~(uintptr_t)1023);
}

// ------------------------------------------------------------------------------------------ forward / dgrad
// Persistent: one CTA per SM walks over output tiles (column tile fastest, so CTAs running side by side
// read the same activation tile through L2).  Two accumulator buffers in tensor memory let the MMA warp
// start the next tile while the epilogue warps drain the previous one.  The epilogue stages each
// 32-column slice through shared memory so that a warp's global stores cover whole rows.
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
constexpr int EPI_SLICE = 64;                     // accumulator columns an epilogue warp handles at a time
constexpr int EPI_BUF_BYTES = 32 * EPI_SLICE * 2; // one staged slice: 32 rows x 64 bf16 = 32 rows of 128 bytes (128-byte swizzle)

// One 64-column slice of a warp's 32 accumulator rows (v: this lane's row): bias / ReLU / accumulation into the stored
// gradient, rounding to bf16, the staged copy in shared memory (stg: one EPI_BUF_BYTES buffer), the store (a TMA store of
// the box at (cx, cw, chh, cn) of tmO, or row by row through rowptr), and the per-column sums for a following batch-norm.
// bias, rowptr and stat_dst already point at the slice's first column (or are null).
__device__ __forceinline__ void epi_slice(uint32_t (&v)[EPI_SLICE], const float* bias, int epi, unsigned long long rowptr, unsigned vmask, bool ok,
                                          bool tma_out, const CUtensorMap* tmO, int cx, int cw, int chh, int cn, uint32_t stg, int lane,
                                          float* stat_dst) {
    const uint32_t swz = (uint32_t)(lane & 7);
    if (bias) {
#pragma unroll
        for (int j = 0; j < EPI_SLICE; j += 4) {
            const float4 bb = __ldg((const float4*)(bias + j));
            v[j] = __float_as_uint(__uint_as_float(v[j]) + bb.x); v[j + 1] = __float_as_uint(__uint_as_float(v[j + 1]) + bb.y);
            v[j + 2] = __float_as_uint(__uint_as_float(v[j + 2]) + bb.z); v[j + 3] = __float_as_uint(__uint_as_float(v[j + 3]) + bb.w);
        }
    }
    if (epi & EPI_RELU) {
#pragma unroll
        for (int j = 0; j < EPI_SLICE; ++j) v[j] = __float_as_uint(fmaxf(__uint_as_float(v[j]), 0.f));
    }
    if ((epi & EPI_ACCUM) && rowptr) {
        // add the gradient already stored for this row (rounded once, after the addition)
        const uint4* o = (const uint4*)((const bf16*)rowptr);
#pragma unroll
        for (int g = 0; g < EPI_SLICE / 8; ++g) {
            const uint4 old = o[g];
            const uint32_t w4[4] = {old.x, old.y, old.z, old.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[8 * g + 2 * j] = __float_as_uint(__uint_as_float(v[8 * g + 2 * j]) + __uint_as_float(w4[j] << 16));
                v[8 * g + 2 * j + 1] = __float_as_uint(__uint_as_float(v[8 * g + 2 * j + 1]) + __uint_as_float(w4[j] & 0xffff0000u));
            }
        }
    }
    // the staging buffer used two slices ago must have been read by its TMA store (the elected lane issued it)
    if (tma_out) { if (elect_one()) bulk_wait_read<1>(); }
    __syncwarp();
    // row `lane`, 16-byte chunk g goes to chunk position g ^ (lane % 8): the 128-byte swizzle of the store's tensor map
#pragma unroll
    for (int g = 0; g < EPI_SLICE / 8; ++g) {
        uint32_t pk[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const __nv_bfloat162 t = __floats2bfloat162_rn(__uint_as_float(v[8 * g + 2 * j]), __uint_as_float(v[8 * g + 2 * j + 1]));
            pk[j] = *(const uint32_t*)&t;
        }
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + (((uint32_t)g ^ swz) << 4)),
                     "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
    }
    if (tma_out) {
        fence_proxy_async();
        __syncwarp();
        if (elect_one()) {
            tma_store_4d(tmO, stg, cx, cw, chh, cn);
            bulk_commit();
        }
    } else {
        __syncwarp();
        // 8 lanes cover one row's 128 bytes, 4 rows per pass
#pragma unroll
        for (int pass = 0; pass < 8; ++pass) {
            const int r = pass * 4 + (lane >> 3);
            const uint32_t g = (uint32_t)(lane & 7);
            const unsigned long long rp = __shfl_sync(0xffffffffu, rowptr, r);
            uint4 t;
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(t.x), "=r"(t.y), "=r"(t.z), "=r"(t.w)
                         : "r"(stg + r * 128 + ((g ^ (uint32_t)(r & 7)) << 4)) : "memory");
            if (rp && ok) *(uint4*)((bf16*)rp + g * 8) = t;
        }
    }
    if (stat_dst) {
        // batch-norm statistics of the layer's output, fused: this lane sums columns 2*lane and 2*lane+1 of the
        // slice over the warp's valid rows, from the values as stored
        float s1a = 0.f, s2a = 0.f, s1b = 0.f, s2b = 0.f;
        const uint32_t cbase = stg + (uint32_t)(lane & 3) * 4, cg = (uint32_t)(lane >> 2);
#pragma unroll 8
        for (int r = 0; r < 32; ++r) {
            uint32_t t;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(t) : "r"(cbase + r * 128 + ((cg ^ (uint32_t)(r & 7)) << 4)) : "memory");
            if ((vmask >> r) & 1u) {
                const float x0 = __uint_as_float(t << 16), x1 = __uint_as_float(t & 0xffff0000u);
                s1a += x0; s2a = fmaf(x0, x0, s2a); s1b += x1; s2b = fmaf(x1, x1, s2b);
            }
        }
        *(float4*)(stat_dst + 4 * lane) = make_float4(s1a, s2a, s1b, s2b);
    }
}


// EPI_WARPS = 4 or 8: with 8, two warps share each quarter of the tensor-memory lanes and take alternate 64-column slices.
// PAIR: launched as clusters of two CTAs.  A pair computes two neighbouring pixel tiles against the same column tile
// with one 256-row MMA per step, issued by the pair's first CTA; each CTA loads its own pixel tile and half of the
// weight rows, drains its own half of the accumulator, and the tmem_empty / full barriers of the first CTA collect
// both CTAs' arrivals.  The number of pixel tiles must be even.
// KSUB: 64-wide K sub-blocks per pipeline stage; a tile's last stage may hold fewer.
// MIN_CTAS: CTAs per SM the register allocation must allow.
//
// Epilogue.  A warp owns 32 rows (pixels) of the tile.  Per 64-column slice it reads the accumulator, applies
// bias / ReLU / accumulation into the old gradient, rounds to bf16 and writes the 32 x 64 block into a swizzled
// staging buffer (two per warp).  If the launch has an output tensor map (p.tma_out) one elected lane hands the
// block to a TMA store, whose box is exactly the warp's 32 pixels x 64 channels; otherwise the warp copies the
// block out row by row (strided outputs of a stride-2 input gradient, partial tiles).  When a batch-norm follows, the
// per-channel sum and sum of squares over the warp's rows are taken from the staged (rounded) values.
//
// ROWS (3x3, stride 1, a tile = whole rows of one image): a stage holds the tile's rows plus one row above and below
// for ONE horizontal shift and one 64-channel chunk; the three vertical taps read it through descriptors that start
// 0, 1 or 2 image rows into the stage (a multiple of 1024 bytes, so the swizzle pattern is unchanged), against three
// weight tiles.  The activation is fetched three times instead of nine.  RESIDENT: the whole weight matrix (all taps
// and chunks of this CTA's rows) is loaded once and stays in shared memory; stages then hold activations only.
constexpr int ROWS_A_BYTES = 24 * 1024;           // room for 128 + 2 * 32 pixels of 128 bytes
template <int N_TILE, int STAGES, int EPI_WARPS, bool PAIR, int KSUB, int MIN_CTAS, bool ROWS, int RES_KB>
__global__ void __launch_bounds__(64 + 32 * EPI_WARPS, MIN_CTAS)
km_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmO, KmParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    constexpr bool RESIDENT = RES_KB > 0;
    constexpr int B_ROWS = PAIR ? N_TILE / 2 : N_TILE;
    constexpr int A_BYTES = BLOCK_M * BLOCK_K * 2, B_BYTES = B_ROWS * BLOCK_K * 2, SUB_BYTES = A_BYTES + B_BYTES;
    constexpr int STAGE_BYTES = ROWS ? ROWS_A_BYTES + (RESIDENT ? 0 : 3 * B_BYTES) : KSUB * SUB_BYTES;
    constexpr int RES_BYTES = RES_KB * 1024;
    constexpr int EPI_BYTES = EPI_WARPS * 2 * EPI_BUF_BYTES;
    constexpr int COL_STEP = EPI_SLICE * (EPI_WARPS / 4);
    constexpr uint32_t TMEM_COLS = 2 * N_TILE;
    uint8_t* wres = smem + STAGES * STAGE_BYTES;                 // resident weights: [tap][chunk][B_ROWS x 64]
    uint8_t* epi_smem = wres + RES_BYTES;
    uint64_t* full = (uint64_t*)(epi_smem + EPI_BYTES);
    uint64_t* empty = full + STAGES;
    uint64_t* tmem_full = empty + STAGES;        // [2]
    uint64_t* tmem_empty = tmem_full + 2;        // [2]
    uint64_t* wres_bar = tmem_empty + 2;
    uint32_t* tmem_slot = (uint32_t*)(wres_bar + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_rank() : 0u;
    const int walker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, walkers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int tiles_m = p.tiles_w * p.tiles_h * p.tiles_n / (PAIR ? 2 : 1);     // pixel tiles, or pairs of them
    const int tiles_c = p.Cn / N_TILE;
    const int per_cls = tiles_m * tiles_c;
    const int total = per_cls * p.ncls;                 // tile index = (class, pixel tile (pair), column tile), column tile fastest

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmA); tma_prefetch_desc(&tmB);
        if (p.tma_out) tma_prefetch_desc(&tmO);
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], PAIR ? 2 * EPI_WARPS : EPI_WARPS); }
        mbar_init(wres_bar, 1);
        fence_barrier_init();
    }
    __syncwarp();
    if (warp == 1) { if (PAIR) tmem_alloc_pair(tmem_slot, TMEM_COLS); else tmem_alloc(tmem_slot, TMEM_COLS); }
    tc_fence_before();
    if (PAIR) cluster_sync_all(); else __syncthreads();       // the pair's barriers are initialised before either CTA signals one
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---- producer (all lanes walk the loop; one elected lane issues)
        bool ok = true;
        const uint32_t smem0 = smem_u32(smem), full_l0 = smem_u32(full), empty0 = smem_u32(empty);
        const uint32_t full_s0 = PAIR ? map_to_cta(full_l0, 0) : full_l0;      // where loads signal: the pair's first CTA
        // stage cursor: destination, barriers, and the parity waited for on `empty` (a fresh barrier
        // passes a wait for parity 1, so the first round finds every stage free)
        uint32_t st = 0, ph = 1, dst = smem0, fb = full_s0, fl = full_l0, eb = empty0;
        if (RESIDENT) {
            // every tap and chunk of this CTA's weight rows, once (a single column tile: Cn == N_TILE)
            const int nblk = p.ntaps * p.kchunks;
            if (elect_one()) {
                mbar_expect_tx_a(smem_u32(wres_bar), nblk * B_BYTES);
                for (int t = 0; t < p.ntaps; ++t)
                    for (int kc = 0; kc < p.kchunks; ++kc)
                        tma_load_2d_a(smem_u32(wres) + (t * p.kchunks + kc) * B_BYTES, &tmB, smem_u32(wres_bar), p.koff[t] + kc * BLOCK_K,
                                      PAIR ? (int)rank * B_ROWS : 0);
            }
            __syncwarp();
        }
        int ktab[9];                                   // rows mode: weight column of (shift, vertical tap), chunk 0
#pragma unroll
        for (int i = 0; i < 9; ++i) ktab[i] = ROWS ? p.koff[p.rows_tap[i]] : 0;
        const uint32_t a_bytes = ROWS ? (uint32_t)(p.Ht + 2) * p.Wt * 128u : 0u;
        for (int tile = walker; tile < total && ok; tile += walkers) {
            const int cls = tile / per_cls, tl = tile - cls * per_cls;
            int tm = tl / tiles_c; const int co0 = (tl - tm * tiles_c) * N_TILE;
            if (PAIR) tm = 2 * tm + (int)rank;
            const int tw = tm % p.tiles_w; tm /= p.tiles_w;
            const int th = tm % p.tiles_h; const int tn = tm / p.tiles_h;
            const int w0 = tw * p.Wt * p.xs, h0 = th * p.Ht * p.xs, n0 = p.n_base + tn * p.Nt;
            const int brow = co0 + (PAIR ? (int)rank * B_ROWS : 0);
            if (ROWS) {
                for (int kc = 0; kc < p.kchunks && ok; ++kc) {
#pragma unroll
                    for (int dwi = 0; dwi < 3; ++dwi) {
                        if (!mbar_wait_a(eb, ph, p.err, 1)) { ok = false; break; }
                        if (elect_one()) {
                            if (!PAIR || rank == 0) mbar_expect_tx_a(fl, (PAIR ? 2 : 1) * (a_bytes + (RESIDENT ? 0 : 3 * B_BYTES)));
                            if (PAIR) tma_load_4d_pair(dst, &tmA, fb, kc * BLOCK_K, dwi - 1, h0 - 1, n0);
                            else tma_load_4d_a(dst, &tmA, fb, kc * BLOCK_K, dwi - 1, h0 - 1, n0);
                            if (!RESIDENT) {
#pragma unroll
                                for (int dhi = 0; dhi < 3; ++dhi) {
                                    const int kcol = ktab[dwi * 3 + dhi] + kc * BLOCK_K;
                                    if (PAIR) tma_load_2d_pair(dst + ROWS_A_BYTES + dhi * B_BYTES, &tmB, fb, kcol, brow);
                                    else tma_load_2d_a(dst + ROWS_A_BYTES + dhi * B_BYTES, &tmB, fb, kcol, brow);
                                }
                            }
                        }
                        __syncwarp();
                        if (++st == STAGES) { st = 0; ph ^= 1u; dst = smem0; fb = full_s0; fl = full_l0; eb = empty0; }
                        else { dst += STAGE_BYTES; fb += 8; fl += 8; eb += 8; }
                    }
                }
                continue;
            }
            const int tap_end = p.cls_tap0[cls + 1];
            int left = (tap_end - p.cls_tap0[cls]) * p.kchunks;      // sub-blocks of this tile still to load
            int sub = 0;                                               // sub-block slot inside the current stage
            for (int tap = p.cls_tap0[cls]; tap < tap_end && ok; ++tap) {
                const int cw = w0 + p.dw[tap], chh = h0 + p.dh[tap], kcol = p.koff[tap];
                for (int kc = 0; kc < p.kchunks; ++kc) {
                    if (sub == 0 && !mbar_wait_a(eb, ph, p.err, 1)) { ok = false; break; }
                    const uint32_t da = dst + sub * SUB_BYTES;
                    if (elect_one()) {
                        if (sub == 0) {
                            // the stage's loads (both CTAs' for a pair) complete on one barrier that expects all their bytes
                            const int cnt = left < KSUB ? left : KSUB;
                            if (!PAIR || rank == 0) mbar_expect_tx_a(fl, (PAIR ? 2 : 1) * cnt * SUB_BYTES);
                        }
                        if (PAIR) {
                            tma_load_4d_pair(da, &tmA, fb, kc * BLOCK_K, cw, chh, n0);
                            tma_load_2d_pair(da + A_BYTES, &tmB, fb, kcol + kc * BLOCK_K, brow);
                        } else {
                            tma_load_4d_a(da, &tmA, fb, kc * BLOCK_K, cw, chh, n0);
                            tma_load_2d_a(da + A_BYTES, &tmB, fb, kcol + kc * BLOCK_K, brow);
                        }
                    }
                    __syncwarp();
                    --left;
                    if (++sub == KSUB || left == 0) {
                        sub = 0;
                        if (++st == STAGES) { st = 0; ph ^= 1u; dst = smem0; fb = full_s0; fl = full_l0; eb = empty0; }
                        else { dst += STAGE_BYTES; fb += 8; fl += 8; eb += 8; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issue (first CTA of a pair only; the elected lane is the same one every time, so the commits
        // track the MMAs it issued)
        if (rank == 0) {
            const uint32_t idesc = make_idesc(PAIR ? 2 * BLOCK_M : BLOCK_M, N_TILE, 0, 0);
            const uint64_t dconst = make_desc(0, 16, 1024);                     // address field left empty
            const uint32_t d_hi = (uint32_t)(dconst >> 32), d_lo = (uint32_t)dconst;
            const uint32_t a16_0 = smem_u32(smem) >> 4, full0 = smem_u32(full), empty0 = smem_u32(empty);
            uint32_t st = 0, ph = 0, a16 = a16_0, fb = full0, eb = empty0;
            int ti = 0;
            bool ok = true;
            const uint32_t row16 = ROWS ? (uint32_t)p.Wt * 128u >> 4 : 0u;      // one image row of a rows-mode stage, in descriptor address units
            uint32_t btab[9];                                                  // resident weights: descriptor word of (shift, vertical tap), chunk 0
#pragma unroll
            for (int i = 0; i < 9; ++i) btab[i] = RESIDENT ? d_lo + (smem_u32(wres) >> 4) + (uint32_t)(p.rows_tap[i] * p.kchunks * (B_BYTES >> 4)) : 0u;
            for (int tile = walker; tile < total && ok; tile += walkers, ++ti) {
                const int buf = ti & 1, use = ti >> 1;
                const int cls = tile / per_cls;
                const int num_kb = (p.cls_tap0[cls + 1] - p.cls_tap0[cls]) * p.kchunks;
                if (use > 0 && !mbar_wait(&tmem_empty[buf], (use - 1) & 1, p.err, 7)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d = tmem_base + buf * N_TILE;
                uint32_t acc = 0;
                if (ROWS) {
                    if (RESIDENT && ti == 0 && !mbar_wait(wres_bar, 0, p.err, 8)) { ok = false; break; }
                    // one stage = one (chunk, horizontal shift); the loop over shifts is unrolled and every table
                    // look-up happens before the tile loop, because the tensor pipe drains while this warp computes
                    for (int kc = 0; kc < p.kchunks && ok; ++kc) {
#pragma unroll
                        for (int dwi = 0; dwi < 3; ++dwi) {
                            if (!mbar_wait_a(fb, ph, p.err, 2)) { ok = false; break; }
                            tc_fence_after();
                            const uint32_t a_lo = d_lo + a16;
                            if (elect_one()) {
#pragma unroll
                                for (int dhi = 0; dhi < 3; ++dhi) {
                                    const uint32_t b_lo = RESIDENT ? btab[dwi * 3 + dhi] + (uint32_t)kc * (B_BYTES >> 4)
                                                                   : a_lo + (uint32_t)((ROWS_A_BYTES + dhi * B_BYTES) >> 4);
#pragma unroll
                                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                                        umma_bf16_w<PAIR>(d, a_lo + dhi * row16 + 2 * k, b_lo + 2 * k, d_hi, idesc, (dhi == 0 && k == 0) ? acc : 1u);
                                }
                                umma_commit_a<PAIR>(eb);
                                if (dwi == 2 && kc == p.kchunks - 1) umma_commit_a<PAIR>(smem_u32(&tmem_full[buf]));
                            }
                            __syncwarp();
                            acc = 1;
                            if (++st == STAGES) { st = 0; ph ^= 1u; a16 = a16_0; fb = full0; eb = empty0; }
                            else { a16 += STAGE_BYTES >> 4; fb += 8; eb += 8; }
                        }
                    }
                } else
                for (int left = num_kb; left > 0; left -= KSUB) {
                    if (!mbar_wait_a(fb, ph, p.err, 2)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_lo = d_lo + a16, b_lo = a_lo + (A_BYTES >> 4);
                    if (elect_one()) {
#pragma unroll
                        for (int j = 0; j < KSUB; ++j) {
                            if (j < left) {
#pragma unroll
                                for (int k = 0; k < BLOCK_K / UMMA_K; ++k)        // 16 columns of K = 32 bytes = 2 address units
                                    umma_bf16_w<PAIR>(d, a_lo + j * (SUB_BYTES >> 4) + 2 * k, b_lo + j * (SUB_BYTES >> 4) + 2 * k, d_hi, idesc,
                                                      (j == 0 && k == 0) ? acc : 1u);
                            }
                        }
                        umma_commit_a<PAIR>(eb);
                        // the tile's last stage: arrives once every MMA of this tile has finished (in both CTAs of a pair)
                        if (left <= KSUB) umma_commit_a<PAIR>(smem_u32(&tmem_full[buf]));
                    }
                    __syncwarp();
                    acc = 1;
                    if (++st == STAGES) { st = 0; ph ^= 1u; a16 = a16_0; fb = full0; eb = empty0; }
                    else { a16 += STAGE_BYTES >> 4; fb += 8; eb += 8; }
                }
            }
        }
    } else {
        // ---- epilogue: warp q = warp % 4 owns tensor-memory lanes 32q .. 32q+31 (= tile rows)
        const int q = warp & 3, half = (warp - 2) >> 2;
        const uint32_t stg0 = smem_u32(epi_smem + (warp - 2) * 2 * EPI_BUF_BYTES);
        uint32_t sbuf = 0;
        int ti = 0;
        bool ok = true;
        const bool tma_out = p.tma_out != 0;
        const uint32_t tmem_empty0 = PAIR ? map_to_cta(smem_u32(&tmem_empty[0]), 0) : 0u;
        // this lane's row of the tile, and the first row of the warp, as (pixel column, pixel row, sample) inside the tile
        const int row = q * 32 + lane;
        const int pw = row % p.Wt, ph = (row / p.Wt) % p.Ht, pn = row / (p.Wt * p.Ht);
        const int bw0 = (q * 32) % p.Wt, bh0 = ((q * 32) / p.Wt) % p.Ht, bn0 = (q * 32) / (p.Wt * p.Ht);
        for (int tile = walker; tile < total && ok; tile += walkers, ++ti) {
            const int buf = ti & 1, use = ti >> 1;
            const int cls = tile / per_cls, tl = tile - cls * per_cls;
            int tm = tl / tiles_c; const int co0 = (tl - tm * tiles_c) * N_TILE;
            if (PAIR) tm = 2 * tm + (int)rank;
            const int tmi = tm + (p.n_base / p.Nt) * (p.tiles_h * p.tiles_w);      // tile index within the whole tensor
            const int tw = tm % p.tiles_w; tm /= p.tiles_w;
            const int th = tm % p.tiles_h; const int tn = tm / p.tiles_h;
            // this lane's row of the tile -> output address (0 = row outside the tensor)
            const int n = p.n_base + tn * p.Nt + pn, h = th * p.Ht + ph, w = tw * p.Wt + pw;
            const bool valid = n < p.N && h < p.Hd && w < p.Wd;
            const unsigned long long rowptr = valid ? (unsigned long long)((bf16*)p.out + (((size_t)n * p.Ho + (h * p.os + p.cls_oph[cls])) * p.Wo +
                                                                                                (w * p.os + p.cls_opw[cls])) * p.Co + co0) : 0ull;
            const unsigned vmask = __ballot_sync(0xffffffffu, rowptr != 0ull);
            ok = mbar_wait_sleep(&tmem_full[buf], use & 1, p.err, 3);
            tc_fence_after();
#pragma unroll 1
            for (int c = half * EPI_SLICE; c < N_TILE; c += COL_STEP) {
                uint32_t v[EPI_SLICE];
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * N_TILE + c;
                tmem_ld32_nowait(taddr, v);
                tmem_ld32_nowait(taddr + 32, v + 32);
                tmem_ld_wait();
                if (c + COL_STEP >= N_TILE) {      // this warp's last read of the accumulator: hand the buffer back to the MMA warp
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) { if (PAIR) mbar_arrive_cluster(tmem_empty0 + 8 * buf); else mbar_arrive(&tmem_empty[buf]); }
                }
                epi_slice(v, p.bias ? p.bias + co0 + c : nullptr, p.epi, rowptr ? rowptr + 2ull * c : 0ull, vmask, ok, tma_out, &tmO, co0 + c,
                          tw * p.Wt + bw0, th * p.Ht + bh0, p.n_base + tn * p.Nt + bn0, stg0 + sbuf * EPI_BUF_BYTES, lane,
                          p.stat_part ? p.stat_part + (((size_t)tmi * 4 + q) * p.Cn + co0 + c) * 2 : nullptr);
                sbuf ^= 1u;
            }
        }
        // the staging buffers must outlive the stores that read them
        if (tma_out) { if (elect_one()) bulk_wait_all(); }
        __syncwarp();
    }
    tc_fence_before();
    __syncwarp();
    if (PAIR) cluster_sync_all(); else __syncthreads();       // neither CTA of a pair leaves while the other may still signal it
    if (warp == 1) { tc_fence_after(); if (PAIR) tmem_dealloc_pair(tmem_base, TMEM_COLS); else tmem_dealloc(tmem_base, TMEM_COLS); }
}

// ------------------------------------------------------------------------------------------ weight gradient
// Tile: rows = two 64-row blocks of the (tap, c_in chunk) axis, columns = N_TILE output channels.
// blockIdx.x = row-block pair, blockIdx.y = column tile, blockIdx.z = pixel split.
template <int N_TILE, int STAGES>
__global__ void __launch_bounds__(NUM_THREADS, 1)
wg_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmDY, WgParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    constexpr int BOX_BYTES = 64 * 64 * 2;                 // 64 pixels x 64 channels
    constexpr int A_BYTES = 2 * BOX_BYTES, B_BYTES = (N_TILE / 64) * BOX_BYTES, STAGE_BYTES = A_BYTES + B_BYTES;
    uint64_t* full = (uint64_t*)(smem + STAGES * STAGE_BYTES);
    uint64_t* empty = full + STAGES;
    uint64_t* accum_bar = empty + STAGES;
    uint32_t* tmem_slot = (uint32_t*)(accum_bar + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rb0 = blockIdx.x * 2;
    const int rb1 = min(rb0 + 1, p.row_blocks - 1);       // an odd count: the last tile's upper half repeats a block and is not stored
    const int co0 = blockIdx.y * N_TILE;
    const int pt_begin = blockIdx.z * p.ptiles_per_split;
    const int pt_end = min(p.ptiles, pt_begin + p.ptiles_per_split);
    const int num_kb = pt_end - pt_begin;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmDY);
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(accum_bar, 1);
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(tmem_slot, N_TILE < 32 ? 32 : N_TILE);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---- producer: all lanes walk the loop, one elected lane issues
        const int tap0 = rb0 / p.kchunks, cc0 = (rb0 - tap0 * p.kchunks) * 64;
        const int tap1 = rb1 / p.kchunks, cc1 = (rb1 - tap1 * p.kchunks) * 64;
        const int dw0 = p.dw[tap0], dh0 = p.dh[tap0], dw1 = p.dw[tap1], dh1 = p.dh[tap1];
        const uint32_t smem0 = smem_u32(smem), full0 = smem_u32(full), empty0 = smem_u32(empty);
        uint32_t st = 0, ph = 1, dst = smem0, fb = full0, eb = empty0;
        // pixel-tile cursor (tw fastest, then th, then tn), advanced without divisions
        int pt = pt_begin;
        int tw = pt % p.tiles_w; pt /= p.tiles_w;
        int th = pt % p.tiles_h; int tn = pt / p.tiles_h;
        const int wstep = p.Wt * p.xs, hstep = p.Ht * p.xs;
        for (int kb = 0; kb < num_kb; ++kb) {
            if (!mbar_wait_a(eb, ph, p.err, 4)) break;
            const int w0 = tw * p.Wt, h0 = th * p.Ht, n0 = p.n_base + tn * p.Nt;
            const int xw = tw * wstep, xh = th * hstep;
            if (elect_one()) {
                mbar_expect_tx_a(fb, STAGE_BYTES);
                tma_load_4d_a(dst, &tmX, fb, cc0, xw + dw0, xh + dh0, n0);
                tma_load_4d_a(dst + BOX_BYTES, &tmX, fb, cc1, xw + dw1, xh + dh1, n0);
#pragma unroll
                for (int j = 0; j < N_TILE / 64; ++j)
                    tma_load_4d_a(dst + A_BYTES + j * BOX_BYTES, &tmDY, fb, co0 + j * 64, w0, h0, n0);
            }
            __syncwarp();
            if (++tw == p.tiles_w) { tw = 0; if (++th == p.tiles_h) { th = 0; ++tn; } }
            if (++st == STAGES) { st = 0; ph ^= 1u; dst = smem0; fb = full0; eb = empty0; }
            else { dst += STAGE_BYTES; fb += 8; eb += 8; }
        }
    } else if (warp == 1) {
        // ---- MMA issue (the elected lane is the same one every time, so the commits track the MMAs it issued)
        const uint32_t idesc = make_idesc(BLOCK_M, N_TILE, 1, 1);
        const uint64_t dconst = make_desc(0, BOX_BYTES, 1024);
        const uint32_t d_hi = (uint32_t)(dconst >> 32), d_lo = (uint32_t)dconst;
        const uint32_t a16_0 = smem_u32(smem) >> 4, full0 = smem_u32(full), empty0 = smem_u32(empty);
        uint32_t st = 0, ph = 0, a16 = a16_0, fb = full0, eb = empty0, acc = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
            if (!mbar_wait_a(fb, ph, p.err, 5)) break;
            tc_fence_after();
            const uint32_t a_lo = d_lo + a16, b_lo = a_lo + (A_BYTES >> 4);
            if (elect_one()) {
#pragma unroll
                for (int k = 0; k < 64 / UMMA_K; ++k)      // 16 pixels = 16 rows of 128 bytes per MMA = 128 address units
                    umma_bf16_w<false>(tmem_base, a_lo + k * (UMMA_K * 128 >> 4), b_lo + k * (UMMA_K * 128 >> 4), d_hi, idesc, k == 0 ? acc : 1u);
                umma_commit_a<false>(eb);
                if (kb == num_kb - 1) umma_commit(accum_bar);
            }
            __syncwarp();
            acc = 1;
            if (++st == STAGES) { st = 0; ph ^= 1u; a16 = a16_0; fb = full0; eb = empty0; }
            else { a16 += STAGE_BYTES >> 4; fb += 8; eb += 8; }
        }
    } else {
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const bool ok = num_kb > 0 ? mbar_wait_sleep(accum_bar, 0, p.err, 6) : true;
        tc_fence_after();
        const int rb = rb0 + (row >> 6);
        const bool valid = ok && rb < p.row_blocks;
        // partial[z][row-block][64][c_out]
        float* out = p.partial + (((size_t)blockIdx.z * p.row_blocks + rb) * 64 + (row & 63)) * p.Co + co0;
#pragma unroll 1
        for (int c = 0; c < N_TILE; c += 32) {
            uint32_t v[32];
            if (num_kb > 0) tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + c, v);
            else {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = 0u;
            }
            if (!valid) continue;
            uint4* o4 = (uint4*)(out + c);
#pragma unroll
            for (int g = 0; g < 8; ++g) o4[g] = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, N_TILE < 32 ? 32 : N_TILE); }
}

// ------------------------------------------------------------------------------------------ weight gradient, rows mode
// 3x3, stride 1, pad 1, with a contraction step of 128 pixels = whole rows of one or two images (W >= 8).  A stage holds
// NX sub-tiles of x, each the step's rows plus one above and one below for one (horizontal shift, 64-channel chunk),
// and the step's dy.  The three vertical taps of a sub-tile are views that start 0, 1 or 2 image rows into it, so one
// fetch of x serves three taps, and dy is fetched once for all 3 * NX (tap, chunk) row blocks the CTA accumulates:
// row blocks 2g and 2g+1 form the two 64-row halves of accumulator g (the descriptor's leading-dimension offset is
// the distance between the two views).  NX = 3: the three shifts of a 64-channel input (all nine taps in one CTA);
// NX = 2: one shift, two chunks (blockIdx.x = shift + 3 * chunk pair).
struct Wg2Params {
    int W, Ht, Nt, tiles_h, tiles_n;          // contraction step = W x Ht x Nt = 128 pixels
    int ptiles, ptiles_per_split, n_base;
    int kchunks, row_blocks, Co;
    float* partial;                           // [splits][row_blocks * 64][Co]
    int* err;
};
template <int N_TILE, int NX, int XSUB_KB, int STAGES>
__global__ void __launch_bounds__(NUM_THREADS, 1)
wg2_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmDY, Wg2Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    constexpr int XSUB = XSUB_KB * 1024, DYBOX = 128 * 128, NB = N_TILE / 64;
    constexpr int STAGE_BYTES = NX * XSUB + NB * DYBOX;
    constexpr int RB = 3 * NX, G = (RB + 1) / 2;
    constexpr uint32_t TMEM_COLS = 512;
    static_assert(G * N_TILE <= 512, "tensor memory");
    uint64_t* full = (uint64_t*)(smem + STAGES * STAGE_BYTES);
    uint64_t* empty = full + STAGES;
    uint64_t* accum_bar = empty + STAGES;
    uint32_t* tmem_slot = (uint32_t*)(accum_bar + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int dw_fixed = NX == 3 ? 0 : (int)blockIdx.x % 3, chunk0 = NX == 3 ? 0 : 2 * ((int)blockIdx.x / 3);
    const int co0 = blockIdx.y * N_TILE;
    const int pt_begin = blockIdx.z * p.ptiles_per_split;
    const int pt_end = min(p.ptiles, pt_begin + p.ptiles_per_split);
    const int num_kb = pt_end - pt_begin;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmDY);
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(accum_bar, 1);
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t xsub_bytes = (uint32_t)(p.Ht + 2) * p.W * p.Nt * 128u;

    if (warp == 0) {
        const uint32_t smem0 = smem_u32(smem), full0 = smem_u32(full), empty0 = smem_u32(empty);
        uint32_t st = 0, ph = 1, dst = smem0, fb = full0, eb = empty0;
        int th = pt_begin % p.tiles_h, tn = pt_begin / p.tiles_h;
        for (int kb = 0; kb < num_kb; ++kb) {
            if (!mbar_wait_a(eb, ph, p.err, 4)) break;
            const int h0 = th * p.Ht, n0 = p.n_base + tn * p.Nt;
            if (elect_one()) {
                mbar_expect_tx_a(fb, NX * xsub_bytes + NB * DYBOX);
#pragma unroll
                for (int sx = 0; sx < NX; ++sx)
                    tma_load_4d_a(dst + sx * XSUB, &tmX, fb, (NX == 3 ? 0 : chunk0 + sx) * 64, (NX == 3 ? sx : dw_fixed) - 1, h0 - 1, n0);
#pragma unroll
                for (int j = 0; j < NB; ++j) tma_load_4d_a(dst + NX * XSUB + j * DYBOX, &tmDY, fb, co0 + j * 64, 0, h0, n0);
            }
            __syncwarp();
            if (++th == p.tiles_h) { th = 0; ++tn; }
            if (++st == STAGES) { st = 0; ph ^= 1u; dst = smem0; fb = full0; eb = empty0; }
            else { dst += STAGE_BYTES; fb += 8; eb += 8; }
        }
    } else if (warp == 1) {
        const uint32_t idesc = make_idesc(BLOCK_M, N_TILE, 1, 1);
        const uint32_t d_hi = (uint32_t)(make_desc(0, 0, 1024) >> 32);
        const uint32_t row16 = (uint32_t)p.W * 128u >> 4;                   // one image row, in descriptor address units
        // low descriptor word of accumulator g's x operand, without the stage address: view of row block 2g, and the
        // distance to the view of row block 2g+1 as the leading-dimension offset
        uint32_t xlo[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int ra = 2 * g, rb = 2 * g + 1 < RB ? 2 * g + 1 : 2 * g;
            const uint32_t oa = (uint32_t)(ra / 3) * (XSUB >> 4) + (uint32_t)(ra % 3) * row16;
            const uint32_t ob = (uint32_t)(rb / 3) * (XSUB >> 4) + (uint32_t)(rb % 3) * row16;
            xlo[g] = oa | ((ob - oa) << 16);
        }
        const uint32_t dylo = (uint32_t)((NX * XSUB) >> 4) | ((uint32_t)(DYBOX >> 4) << 16);
        // x rows of the step's 16-pixel slices (the sub-tile keeps two extra rows per image)
        uint32_t koff[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int pix = 16 * k, ni = pix / (p.W * p.Ht), hi = (pix / p.W) % p.Ht, wi = pix % p.W;
            koff[k] = (uint32_t)((ni * (p.Ht + 2) + hi) * p.W + wi) * 8u;
        }
        const uint32_t a16_0 = smem_u32(smem) >> 4, full0 = smem_u32(full), empty0 = smem_u32(empty);
        uint32_t st = 0, ph = 0, a16 = a16_0, fb = full0, eb = empty0, acc = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
            if (!mbar_wait_a(fb, ph, p.err, 5)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int g = 0; g < G; ++g) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                                     "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
                                     ::"r"(tmem_base + g * N_TILE), "r"(xlo[g] + a16 + koff[k]), "r"(dylo + a16 + (uint32_t)k * 128u), "r"(d_hi), "r"(idesc),
                                       "r"(k == 0 ? acc : 1u) : "memory");
                    }
                }
                umma_commit_a<false>(eb);
                if (kb == num_kb - 1) umma_commit(accum_bar);
            }
            __syncwarp();
            acc = 1;
            if (++st == STAGES) { st = 0; ph ^= 1u; a16 = a16_0; fb = full0; eb = empty0; }
            else { a16 += STAGE_BYTES >> 4; fb += 8; eb += 8; }
        }
    } else {
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const bool ok = num_kb > 0 ? mbar_wait_sleep(accum_bar, 0, p.err, 6) : true;
        tc_fence_after();
#pragma unroll 1
        for (int g = 0; g < G; ++g) {
            const int rb = 2 * g + (row >> 6);                       // local row block -> (sub-tile, vertical tap)
            const bool valid = ok && rb < RB;
            const int sx = rb / 3, dhi = rb % 3;
            const int dwi = NX == 3 ? sx : dw_fixed, chunk = NX == 3 ? 0 : chunk0 + sx;
            const int grb = (dhi * 3 + dwi) * p.kchunks + chunk;     // row block of the whole matrix: (tap, chunk)
            float* out = p.partial + (((size_t)blockIdx.z * p.row_blocks + grb) * 64 + (row & 63)) * p.Co + co0;
#pragma unroll 1
            for (int c = 0; c < N_TILE; c += 32) {
                uint32_t v[32];
                if (num_kb > 0) tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + g * N_TILE + c, v);
                else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                if (!valid) continue;
                uint4* o4 = (uint4*)(out + c);
#pragma unroll
                for (int gq = 0; gq < 8; ++gq) o4[gq] = make_uint4(v[4 * gq], v[4 * gq + 1], v[4 * gq + 2], v[4 * gq + 3]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, TMEM_COLS); }
}

// ------------------------------------------------------------------------------------------ first layer, weight gradient
// 3x3, stride 1, pad 1, 3 input channels (K = 27 of the weight matrix's columns).  The 27 columns of the im2col
// matrix are built in shared memory: the producer fetches the step's image rows (plus one above and below) as raw
// rows of W * 3 elements, four builder warps write one 128-byte line per pixel, [pixel][k] with k = (row tap, column tap,
// channel), zero beyond 27, in the 128-byte-swizzled layout the MMA reads (MN-major: M = k, contraction = pixels).
// D[k][c_out] accumulates over all steps of the CTA in tensor memory; rows 64..127 of the accumulator repeat rows 0..63
// (leading-dimension offset 0) and are dropped.  Partials per CTA, reduced in a fixed order by stem_wg_reduce_kernel.
struct StemWgParams {
    int W, Ht, tiles_h;                 // contraction step = W x Ht = 128 pixels of one image
    int steps, steps_per_cta;           // steps = N * tiles_h
    float* partial;                     // [Co / 64][CTAs][64 k][64 c_out]
    int* err;
};
constexpr int STEM_RAW_BYTES = 2048;    // room for (Ht + 2) raw rows of W * 3 bf16
template <int STAGES>
__global__ void __launch_bounds__(NUM_THREADS, 1)
stem_wg_kernel(const __grid_constant__ CUtensorMap tmRaw, const __grid_constant__ CUtensorMap tmDY, StemWgParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    constexpr int TILE = 128 * 128;                                  // im2col tile and dy tile: 128 pixels x 128 bytes
    uint8_t* im = smem;                                              // [STAGES][TILE]
    uint8_t* dyt = smem + STAGES * TILE;                             // [STAGES][TILE]
    uint8_t* raw = smem + 2 * STAGES * TILE;                         // [STAGES][STEM_RAW_BYTES]
    uint64_t* tma_full = (uint64_t*)(raw + STAGES * STEM_RAW_BYTES);
    uint64_t* im_full = tma_full + STAGES;
    uint64_t* empty = im_full + STAGES;
    uint64_t* accum_bar = empty + STAGES;
    uint32_t* tmem_slot = (uint32_t*)(accum_bar + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int co0 = blockIdx.y * 64;
    const int s_begin = blockIdx.x * p.steps_per_cta;
    const int s_end = min(p.steps, s_begin + p.steps_per_cta);
    const int num_kb = s_end > s_begin ? s_end - s_begin : 0;
    const uint32_t raw_bytes = (uint32_t)(p.Ht + 2) * p.W * 6u;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmRaw); tma_prefetch_desc(&tmDY);
        for (int s = 0; s < STAGES; ++s) { mbar_init(&tma_full[s], 1); mbar_init(&im_full[s], 4); mbar_init(&empty[s], 1); }
        mbar_init(accum_bar, 1);
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(tmem_slot, 64);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        uint32_t st = 0, ph = 1;
        int th = s_begin % p.tiles_h, n = s_begin / p.tiles_h;
        for (int kb = 0; kb < num_kb; ++kb) {
            if (!mbar_wait(&empty[st], ph, p.err, 11)) break;
            if (elect_one()) {
                const uint32_t bar = smem_u32(&tma_full[st]);
                mbar_expect_tx_a(bar, raw_bytes + TILE);
                asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                             ::"r"(smem_u32(raw + st * STEM_RAW_BYTES)), "l"(&tmRaw), "r"(bar), "r"(0), "r"(th * p.Ht - 1), "r"(n) : "memory");
                tma_load_4d_a(smem_u32(dyt + st * TILE), &tmDY, bar, co0, 0, th * p.Ht, n);
            }
            __syncwarp();
            if (++th == p.tiles_h) { th = 0; ++n; }
            if (++st == STAGES) { st = 0; ph ^= 1u; }
        }
    } else if (warp == 1) {
        const uint32_t idesc = make_idesc(BLOCK_M, 64, 1, 1);
        const uint64_t dA = make_desc(0, 0, 1024), dB = make_desc(0, TILE, 1024);
        const uint32_t d_hi = (uint32_t)(dA >> 32), a_lo0 = (uint32_t)dA, b_lo0 = (uint32_t)dB;
        uint32_t st = 0, ph = 0, acc = 0;
        for (int kb = 0; kb < num_kb; ++kb) {
            if (!mbar_wait(&tma_full[st], ph, p.err, 12)) break;      // dy has landed
            if (!mbar_wait(&im_full[st], ph, p.err, 13)) break;       // the im2col lines are written
            tc_fence_after();
            const uint32_t a_lo = a_lo0 + (smem_u32(im + st * TILE) >> 4), b_lo = b_lo0 + (smem_u32(dyt + st * TILE) >> 4);
            if (elect_one()) {
#pragma unroll
                for (int k = 0; k < 8; ++k)               // 16 pixels = 16 lines of 128 bytes per MMA
                    umma_bf16_w<false>(tmem_base, a_lo + k * 128, b_lo + k * 128, d_hi, idesc, k == 0 ? acc : 1u);
                umma_commit(&empty[st]);
                if (kb == num_kb - 1) umma_commit(accum_bar);
            }
            __syncwarp();
            acc = 1;
            if (++st == STAGES) { st = 0; ph ^= 1u; }
        }
    } else {
        // ---- builders: thread = one pixel of the step
        const int pix = (warp - 2) * 32 + lane;
        const int r = pix / p.W, c = pix - r * p.W;
        const bool left = c > 0, right = c < p.W - 1;
        const uint32_t line = (uint32_t)pix * 128u, swz = (uint32_t)(pix & 7);
        uint32_t st = 0, ph = 0;
        bool ok = true;
        // columns 32..63 of every line are never written below: clear them once (their accumulator rows are dropped)
        for (int s2 = 0; s2 < STAGES; ++s2)
#pragma unroll
            for (int ch = 4; ch < 8; ++ch)
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(smem_u32(im + s2 * TILE) + line + (((uint32_t)ch ^ swz) << 4)), "r"(0u) : "memory");
        for (int kb = 0; kb < num_kb && ok; ++kb) {
            ok = mbar_wait(&tma_full[st], ph, p.err, 14);
            const uint32_t rb = smem_u32(raw + st * STEM_RAW_BYTES) + (uint32_t)(r * p.W + c - 1) * 6u;
            uint32_t h[28];
#pragma unroll
            for (int dr = 0; dr < 3; ++dr) {
#pragma unroll
                for (int j = 0; j < 9; ++j) {
                    uint32_t v = 0;
                    const bool in = j < 3 ? left : (j < 6 ? true : right);
                    if (in) { uint16_t t; asm volatile("ld.shared.u16 %0, [%1];" : "=h"(t) : "r"(rb + (uint32_t)(dr * p.W * 6 + 2 * j)) : "memory"); v = t; }
                    h[dr * 9 + j] = v;
                }
            }
            h[27] = 0;
            const uint32_t dst = smem_u32(im + st * TILE) + line;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                uint32_t w4[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) { const int i = 8 * ch + 2 * j; w4[j] = i + 1 < 28 ? (h[i] | (h[i + 1] << 16)) : 0u; }
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (((uint32_t)ch ^ swz) << 4)), "r"(w4[0]), "r"(w4[1]), "r"(w4[2]), "r"(w4[3]) : "memory");
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&im_full[st]);
            if (++st == STAGES) { st = 0; ph ^= 1u; }
        }
        // ---- epilogue: accumulator rows 0..63 (warps of lane quarters 0 and 1) are the im2col columns k
        const int q = warp & 3;
        if (q < 2) {
            const bool done = num_kb > 0 ? mbar_wait_sleep(accum_bar, 0, p.err, 15) : true;
            tc_fence_after();
            const int k = q * 32 + lane;
            float* out = p.partial + (((size_t)blockIdx.y * gridDim.x + blockIdx.x) * 64 + k) * 64;
#pragma unroll 1
            for (int cc = 0; cc < 64; cc += 32) {
                uint32_t v[32];
                if (num_kb > 0) tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + cc, v);
                else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                if (!done || k >= 27) continue;
                uint4* o4 = (uint4*)(out + cc);
#pragma unroll
                for (int g = 0; g < 8; ++g) o4[g] = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 64); }
}

// dw[co][k] = sum over CTAs (ascending) of partial[co / 64][cta][k][co % 64], k < 27
__global__ void stem_wg_reduce_kernel(const float* __restrict__ partial, float* __restrict__ dw, int ctas, int Co, bool accum) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= Co * 27) return;
    const int k = i / Co, co = i - k * Co;                 // consecutive threads: consecutive c_out (coalesced reads)
    const float* ptr = partial + ((size_t)(co >> 6) * ctas * 64 + k) * 64 + (co & 63);
    float s = 0.f;
#pragma unroll 4
    for (int b = 0; b < ctas; ++b) s += ptr[(size_t)b * 64 * 64];
    float* d = dw + (size_t)co * 27 + k;
    *d = accum ? *d + s : s;
}

// ------------------------------------------------------------------------------------------ first layer, forward
// Same im2col lines as stem_wg_kernel, read K-major this time: D[pixel][c_out] = lines[pixel][k] * W[c_out][k], k < 32
// (two MMAs per 128-pixel tile).  The 64 x 27 weight tile is written once per CTA.  Warps: 0 producer of raw rows,
// 1 MMA issue, 2-5 epilogue (the one of km_kernel: bf16 tile, TMA store, batch-norm sums), 6-9 line builders.
struct StemFwParams {
    int W, Ht, tiles_h, tiles;          // tile = W x Ht = 128 pixels of one image; tiles = N * tiles_h
    int Co, epi;
    const bf16* w;                      // [Co][27]
    const float* bias;                  // or nullptr
    float* stat_part;                   // or nullptr: [tile * 4 + warp][Co][2]
    int* err;
};
template <int STAGES>
__global__ void __launch_bounds__(320, 2)
stem_fw_kernel(const __grid_constant__ CUtensorMap tmRaw, const __grid_constant__ CUtensorMap tmO, StemFwParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    constexpr int TILE = 128 * 128;
    uint8_t* im = smem;                                              // [STAGES][TILE]
    uint8_t* wt = smem + STAGES * TILE;                              // [64 c_out][128 bytes]
    uint8_t* epi_smem = wt + 64 * 128;                               // [4 warps][2][EPI_BUF_BYTES]
    uint8_t* raw = epi_smem + 4 * 2 * EPI_BUF_BYTES;                 // [STAGES][STEM_RAW_BYTES]
    uint64_t* raw_full = (uint64_t*)(raw + STAGES * STEM_RAW_BYTES);
    uint64_t* im_full = raw_full + STAGES;
    uint64_t* empty = im_full + STAGES;
    uint64_t* tmem_full = empty + STAGES;                            // [2]
    uint64_t* tmem_empty = tmem_full + 2;                            // [2]
    uint64_t* wt_bar = tmem_empty + 2;
    uint32_t* tmem_slot = (uint32_t*)(wt_bar + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int co0 = blockIdx.y * 64;
    const uint32_t raw_bytes = (uint32_t)(p.Ht + 2) * p.W * 6u;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmRaw); tma_prefetch_desc(&tmO);
        for (int s = 0; s < STAGES; ++s) { mbar_init(&raw_full[s], 1); mbar_init(&im_full[s], 4); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], 4); }
        mbar_init(wt_bar, 4);
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(tmem_slot, 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        uint32_t st = 0, ph = 1;
        for (int tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
            if (!mbar_wait(&empty[st], ph, p.err, 21)) break;
            const int n = tile / p.tiles_h, th = tile - n * p.tiles_h;
            if (elect_one()) {
                const uint32_t bar = smem_u32(&raw_full[st]);
                mbar_expect_tx_a(bar, raw_bytes);
                asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                             ::"r"(smem_u32(raw + st * STEM_RAW_BYTES)), "l"(&tmRaw), "r"(bar), "r"(0), "r"(th * p.Ht - 1), "r"(n) : "memory");
            }
            __syncwarp();
            if (++st == STAGES) { st = 0; ph ^= 1u; }
        }
    } else if (warp == 1) {
        const uint32_t idesc = make_idesc(BLOCK_M, 64, 0, 0);
        const uint64_t dK = make_desc(0, 16, 1024);
        const uint32_t d_hi = (uint32_t)(dK >> 32), d_lo = (uint32_t)dK;
        const uint32_t b_lo = d_lo + (smem_u32(wt) >> 4);
        uint32_t st = 0, ph = 0;
        int ti = 0;
        bool ok = mbar_wait(wt_bar, 0, p.err, 22);
        for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x, ++ti) {
            const int buf = ti & 1, use = ti >> 1;
            if (use > 0 && !mbar_wait(&tmem_empty[buf], (use - 1) & 1, p.err, 23)) break;
            if (!mbar_wait(&im_full[st], ph, p.err, 24)) break;
            tc_fence_after();
            const uint32_t a_lo = d_lo + (smem_u32(im + st * TILE) >> 4);
            if (elect_one()) {
                umma_bf16_w<false>(tmem_base + buf * 64, a_lo, b_lo, d_hi, idesc, 0u);
                umma_bf16_w<false>(tmem_base + buf * 64, a_lo + 2, b_lo + 2, d_hi, idesc, 1u);
                umma_commit(&empty[st]);
                umma_commit(&tmem_full[buf]);
            }
            __syncwarp();
            if (++st == STAGES) { st = 0; ph ^= 1u; }
        }
    } else if (warp >= 6) {
        // ---- builders: thread = one pixel of the tile; first the weight tile (threads 0..63: one c_out row each)
        const int pix = (warp - 6) * 32 + lane;
        const uint32_t line = (uint32_t)pix * 128u, swz = (uint32_t)(pix & 7);
        if (pix < 64) {
            const bf16* wr = p.w + (size_t)(co0 + pix) * 27;
            uint32_t h[28];
#pragma unroll
            for (int j = 0; j < 27; ++j) h[j] = (uint32_t)__bfloat16_as_ushort(wr[j]);
            h[27] = 0;
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                uint32_t w4[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) { const int i = 8 * ch + 2 * j; w4[j] = i + 1 < 28 ? (h[i] | (h[i + 1] << 16)) : 0u; }
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(wt) + line + (((uint32_t)ch ^ swz) << 4)), "r"(w4[0]), "r"(w4[1]), "r"(w4[2]), "r"(w4[3]) : "memory");
            }
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(wt_bar);
        const int r = pix / p.W, c = pix - r * p.W;
        const bool left = c > 0, right = c < p.W - 1;
        uint32_t st = 0, ph = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x) {
            ok = mbar_wait(&raw_full[st], ph, p.err, 25);
            const uint32_t rb = smem_u32(raw + st * STEM_RAW_BYTES) + (uint32_t)(r * p.W + c - 1) * 6u;
            uint32_t h[28];
#pragma unroll
            for (int dr = 0; dr < 3; ++dr) {
#pragma unroll
                for (int j = 0; j < 9; ++j) {
                    uint32_t v = 0;
                    const bool in = j < 3 ? left : (j < 6 ? true : right);
                    if (in) { uint16_t t; asm volatile("ld.shared.u16 %0, [%1];" : "=h"(t) : "r"(rb + (uint32_t)(dr * p.W * 6 + 2 * j)) : "memory"); v = t; }
                    h[dr * 9 + j] = v;
                }
            }
            h[27] = 0;
            const uint32_t dst = smem_u32(im + st * TILE) + line;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                uint32_t w4[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) { const int i = 8 * ch + 2 * j; w4[j] = i + 1 < 28 ? (h[i] | (h[i + 1] << 16)) : 0u; }
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (((uint32_t)ch ^ swz) << 4)), "r"(w4[0]), "r"(w4[1]), "r"(w4[2]), "r"(w4[3]) : "memory");
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&im_full[st]);
            if (++st == STAGES) { st = 0; ph ^= 1u; }
        }
    } else {
        // ---- epilogue: warp q = warp % 4 owns tensor-memory lanes 32q .. 32q+31 = 32 consecutive pixels of the tile
        const int q = warp & 3;
        const uint32_t stg0 = smem_u32(epi_smem + (warp - 2) * 2 * EPI_BUF_BYTES);
        uint32_t sbuf = 0;
        int ti = 0;
        bool ok = true;
        const int bw0 = (q * 32) % p.W, bh0 = (q * 32) / p.W;
        for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x, ++ti) {
            const int buf = ti & 1, use = ti >> 1;
            const int n = tile / p.tiles_h, th = tile - n * p.tiles_h;
            ok = mbar_wait_sleep(&tmem_full[buf], use & 1, p.err, 26);
            tc_fence_after();
            uint32_t v[EPI_SLICE];
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * 64;
            tmem_ld32_nowait(taddr, v);
            tmem_ld32_nowait(taddr + 32, v + 32);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tmem_empty[buf]);
            epi_slice(v, p.bias ? p.bias + co0 : nullptr, p.epi, 0ull, 0xffffffffu, ok, true, &tmO, co0, bw0, th * p.Ht + bh0, n,
                      stg0 + sbuf * EPI_BUF_BYTES, lane, p.stat_part ? p.stat_part + (((size_t)tile * 4 + q) * p.Co + co0) * 2 : nullptr);
            sbuf ^= 1u;
        }
        if (elect_one()) bulk_wait_all();
        __syncwarp();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 128); }
}

// dW[co][tap][ci] = sum_z partial[z][(tap, cc)][ci % 64][co], z ascending.  A CTA of 256 threads (it fits beside a
// resident tensor-core CTA of another stream) transposes a tile of 8 rows x 32 columns: many small CTAs, because a layer
// has few output elements (36 864 for 64 -> 64) and many partial matrices (up to 147), so the kernel lives on the number of
// loads in flight; a thread owns one element and keeps 16 independent loads in flight along z.
__global__ void __launch_bounds__(256) wg_reduce_kernel(const float* __restrict__ partial, float* __restrict__ dw, int splits, int row_blocks, int Co,
                                                        bool accum) {
    __shared__ float t[8][33];
    const int R = row_blocks * 64;                       // = taps * Cin
    const int r0 = blockIdx.x * 8, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x, ty = threadIdx.y;        // 32 x 8
    const unsigned zs = (unsigned)R * Co;                // one partial matrix (< 2^32 elements)
    const float* p = partial + (size_t)(r0 + ty) * Co + c0 + tx;
    float s = 0.f;
    int z = 0;
    for (; z + 16 <= splits; z += 16, p += (size_t)16 * zs) {
        float v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = __ldg(p + j * zs);
#pragma unroll
        for (int j = 0; j < 16; ++j) s += v[j];
    }
    for (; z < splits; ++z, p += zs) s += __ldg(p);
    t[ty][tx] = s;
    __syncthreads();
    const int tid = ty * 32 + tx, c = tid >> 3, r = tid & 7;      // 8 consecutive threads write 8 consecutive elements of a row of dW
    float* d = dw + (size_t)(c0 + c) * R + r0 + r;
    *d = accum ? *d + t[r][c] : t[r][c];
}

// One launch per module and step: the update of Eq. dl_update for ALL of the module's parameters.
//   * weight matrices of tensor-core layers, in 32 x 32 tiles: w -= lr g on the fp32 master, the bf16 copy W[co][tap][ci] of
//     the next version and its tap-flipped transpose Wt[ci][taps-1-tap][co] for the input-gradient kernel;
//   * everything else (matrices of other layers, biases, gamma, beta), 4 values per thread: w -= lr g, the storage copy.
// has_grad == 0 (no backward batch yet): w(t+1) = w(t), only the copies are written.
// (Summing the weight-gradient partials here as well was measured slower: that reduction then sits in the module's chain
// in front of its next forward pass instead of running beside the backward pass on the weight-gradient stream.)
// 256 threads and few registers per CTA: the CTAs fit beside a resident tensor-core CTA of another module, so the
// update does not wait for a persistent kernel to drain (with 1024-thread CTAs it did, and the step took 4 % longer).
__global__ void __launch_bounds__(256) update_module_kernel(UpdTable tb, float* __restrict__ master, const float* __restrict__ grad,
                                                            bf16* __restrict__ wcopy, bf16* __restrict__ wtcopy, float* __restrict__ small_copy, float lr,
                                                            int has_grad) {
    __shared__ bf16 t[32][34];
    const int tx = threadIdx.x, ty = threadIdx.y;          // 32 x 8
    int b = blockIdx.x;
    if (b < tb.total_tiles) {
        int oi = 0;
        while (oi + 1 < tb.nops && b >= tb.ops[oi + 1].tile0) ++oi;
        const UpdOp o = tb.ops[oi];
        b -= o.tile0;
        const int R = o.taps * o.Ci, tiles_c = o.Co / 32;
        const int r0 = (b / tiles_c) * 32, c0 = (b % tiles_c) * 32;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = ty + 8 * i;                          // row c0 + c of W, columns r0 + tx
            const size_t idx = o.w_off + (size_t)(c0 + c) * R + r0 + tx;
            float w = master[idx];
            if (has_grad) { w = fmaf(-lr, grad[idx], w); master[idx] = w; }
            const bf16 wb = __float2bfloat16_rn(w);
            wcopy[idx] = wb;
            t[c][tx] = wb;                                     // [c][r]
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = r0 + ty + 8 * i, tap = r / o.Ci, ci = r - tap * o.Ci;     // a tile's 32 rows share one tap (Ci is a multiple of 64)
            wtcopy[o.w_off + ((size_t)ci * o.taps + (o.taps - 1 - tap)) * o.Co + c0 + tx] = t[tx][ty + 8 * i];
        }
        return;
    }
    // the other ranges: float4 number q of their concatenation
    const size_t q = (size_t)(b - tb.total_tiles) * 256 + ty * 32 + tx;
    size_t first = 0;
    for (int j = 0; j < tb.nranges; ++j) {
        const size_t n4 = tb.ranges[j].count / 4;
        if (q < first + n4) {
            const size_t e = tb.ranges[j].start + (q - first) * 4;
            float4 w = *(const float4*)(master + e);
            if (has_grad) {
                const float4 g = *(const float4*)(grad + e);
                w.x = fmaf(-lr, g.x, w.x); w.y = fmaf(-lr, g.y, w.y); w.z = fmaf(-lr, g.z, w.z); w.w = fmaf(-lr, g.w, w.w);
                *(float4*)(master + e) = w;
            }
            if (e < tb.n_big) {
                __nv_bfloat162 lo = __floats2bfloat162_rn(w.x, w.y), hi = __floats2bfloat162_rn(w.z, w.w);
                uint2 pk; pk.x = *(unsigned*)&lo; pk.y = *(unsigned*)&hi;
                *(uint2*)(wcopy + e) = pk;
            } else {
                *(float4*)(small_copy + (e - tb.n_big)) = w;
            }
            return;
        }
        first += n4;
    }
}

cudaError_t run_update_module(const UpdTable& tb, float* master, const float* grad, void* wcopy, void* wtcopy, float* small_copy, float lr,
                              bool has_grad, cudaStream_t s) {
    size_t plain4 = 0;
    for (int j = 0; j < tb.nranges; ++j) plain4 += tb.ranges[j].count / 4;
    const unsigned blocks = (unsigned)(tb.total_tiles + (plain4 + 255) / 256);
    if (!blocks) return cudaSuccess;
    update_module_kernel<<<blocks, dim3(32, 8), 0, s>>>(tb, master, grad, (bf16*)wcopy, (bf16*)wtcopy, small_copy, lr, has_grad ? 1 : 0);
    return cudaGetLastError();
}

// Wt[ci][R*R-1-tap][co] = W[co][tap][ci]: the weights of the transposed convolution, K-major for km_kernel.
__global__ void flip_transpose_kernel(const bf16* __restrict__ w, bf16* __restrict__ wt, int Co, int taps, int Ci) {
    __shared__ bf16 t[32][34];
    const int tap = blockIdx.z;
    const int ci0 = blockIdx.x * 32, co0 = blockIdx.y * 32;
    const int tx = threadIdx.x, ty = threadIdx.y;
    for (int i = ty; i < 32; i += 8) t[i][tx] = w[((size_t)(co0 + i) * taps + tap) * Ci + ci0 + tx];
    __syncthreads();
    for (int i = ty; i < 32; i += 8) wt[((size_t)(ci0 + i) * taps + (taps - 1 - tap)) * Co + co0 + tx] = t[tx][i];
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

bool init() {
    if (g_encode) return true;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn) return false;
    g_encode = (EncodeTiledFn)fn;
    return true;
}

bool make_map_4d(TensorMap* out, const void* base, int C, int W, int H, int N, int boxC, int boxW, int boxH, int boxN, int stride) {
    static_assert(sizeof(TensorMap) == sizeof(CUtensorMap), "tensor map size");
    if (!init()) return false;
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
    cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    cuuint32_t box[4] = {(cuuint32_t)boxC, (cuuint32_t)(boxW * stride), (cuuint32_t)(boxH * stride), (cuuint32_t)boxN};
    cuuint32_t estr[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
    CUresult r = g_encode((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_map_out(TensorMap* out, const void* base, int C, int W, int H, int N, int Wt, int Ht) {
    // the 32 pixels an epilogue warp owns inside a 128-pixel tile of Wt x Ht x Nt pixels
    const int bw = Wt < 32 ? Wt : 32, bh = Ht < 32 / bw ? Ht : 32 / bw, bn = 32 / (bw * bh);
    return make_map_4d(out, base, C, W, H, N, EPI_SLICE, bw, bh, bn, 1);
}

bool make_map_2d(TensorMap* out, const void* base, long inner, long outer, int box_inner, int box_outer) {
    if (!init()) return false;
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)inner * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool pixel_tile(int H, int W, int pixels, int* Wt, int* Ht, int* Nt) {
    auto pow2 = [](int v) { return v > 0 && (v & (v - 1)) == 0; };
    if (!pow2(W) || !pow2(H)) return false;
    int wt = W < pixels ? W : pixels;
    int ht = H < pixels / wt ? H : pixels / wt;
    *Wt = wt; *Ht = ht; *Nt = pixels / (wt * ht);
    return true;
}

static int device_sms() {
    static int n = 0;
    if (!n) { int dev = 0; cudaGetDevice(&dev); cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev); if (n <= 0) n = 148; }
    return n;
}
// SMs a launcher sizes its grid (or its contraction splits) for: `sms` of the caller, clamped to the device; 0 = all.
// Fewer than the device has: kernels of different module streams then run side by side, a tensor-core kernel next to
// a memory-bound one.
static int sm_count(int sms) { return sms > 0 && sms < device_sms() ? sms : device_sms(); }

template <int N_TILE, int STAGES, int EPI_WARPS, int KSUB, bool ROWS, int RES_KB>
static cudaError_t launch_km(const TensorMap& a, const TensorMap& b, const TensorMap& o, const KmParams& p, cudaStream_t s) {
    constexpr int stage = ROWS ? ROWS_A_BYTES + (RES_KB ? 0 : 3 * N_TILE * BLOCK_K * 2) : KSUB * (BLOCK_M * BLOCK_K * 2 + N_TILE * BLOCK_K * 2);
    constexpr int smem = STAGES * stage + RES_KB * 1024 + EPI_WARPS * 2 * EPI_BUF_BYTES + 1024 + 256;
    static_assert(smem <= 232448, "shared memory");
    // CTAs of this variant that fit on an SM: shared memory (227 KB, 1 KB reserved per CTA) and 512 tensor-memory columns
    constexpr int by_smem = (227 * 1024) / (smem + 1024), by_tmem = 512 / (2 * N_TILE);
    constexpr int per_sm = by_smem < by_tmem ? by_smem : by_tmem;
    static_assert(per_sm >= 1 && per_sm <= 2, "CTAs per SM");
    auto kernel = km_kernel<N_TILE, STAGES, EPI_WARPS, false, KSUB, per_sm, ROWS, RES_KB>;
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    const int total = p.tiles_w * p.tiles_h * p.tiles_n * (p.Cn / N_TILE) * p.ncls;
    const int slots = sm_count(p.sms) * per_sm;
    const int grid = total < slots ? total : slots;
    kernel<<<grid, 64 + 32 * EPI_WARPS, smem, s>>>(*(const CUtensorMap*)&a, *(const CUtensorMap*)&b, *(const CUtensorMap*)&o, p);
    return cudaGetLastError();
}

// CTA pairs: `b` is a tensor map whose box holds N_TILE / 2 weight rows.
template <int N_TILE, int STAGES, int EPI_WARPS, int KSUB, bool ROWS>
static cudaError_t launch_km_pair(const TensorMap& a, const TensorMap& b, const TensorMap& o, const KmParams& p, cudaStream_t s) {
    constexpr int stage = ROWS ? ROWS_A_BYTES + 3 * (N_TILE / 2) * BLOCK_K * 2 : KSUB * (BLOCK_M * BLOCK_K * 2 + (N_TILE / 2) * BLOCK_K * 2);
    constexpr int smem = STAGES * stage + EPI_WARPS * 2 * EPI_BUF_BYTES + 1024 + 256;
    static_assert(smem <= 232448, "shared memory");
    auto kernel = km_kernel<N_TILE, STAGES, EPI_WARPS, true, KSUB, 1, ROWS, 0>;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(64 + 32 * EPI_WARPS); cfg.dynamicSmemBytes = smem; cfg.stream = s; cfg.attrs = at; cfg.numAttrs = 1;
    static int resident_pairs = 0;              // pairs that can be resident at once on the whole device
    if (!resident_pairs) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        cfg.gridDim = dim3(device_sms());
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n <= 0) { cudaGetLastError(); n = device_sms() / 2; }
        resident_pairs = n;
    }
    const int max_pairs = resident_pairs < sm_count(p.sms) / 2 ? resident_pairs : sm_count(p.sms) / 2;
    const int total = (p.tiles_w * p.tiles_h * p.tiles_n / 2) * (p.Cn / N_TILE) * p.ncls;
    cfg.gridDim = dim3(2 * (total < max_pairs ? total : max_pairs));
    return cudaLaunchKernelEx(&cfg, kernel, *(const CUtensorMap*)&a, *(const CUtensorMap*)&b, *(const CUtensorMap*)&o, p);
}

cudaError_t run_km(const KmMaps& m, const KmParams& p_in, int n_tile, cudaStream_t s) {
    KmParams p = p_in;
    // the store through the output map covers whole 32-pixel boxes and clips only at the tensor's edge: it needs a dense
    // output (stride 1) and a sample range that ends where the tiles end or where the tensor ends
    p.tma_out = m.out && p.os == 1 && p.ncls == 1 && (p.n_base + p.tiles_n * p.Nt <= p.N || p.N == p.Nfull) ? 1 : 0;
    const TensorMap& o = p.tma_out ? *m.out : *m.a;       // unused by the kernel without tma_out
    const bool even = (p.tiles_w * p.tiles_h * p.tiles_n) % 2 == 0;
    // rows mode: 3x3, stride 1, tiles that are whole rows of one image
    bool rows = m.a_rows && p.ncls == 1 && p.ntaps == 9 && p.xs == 1 && p.os == 1 && p.tiles_w == 1 && p.Nt == 1;
    if (rows) {
        for (int i = 0; i < 9; ++i) p.rows_tap[i] = -1;
        for (int t = 0; t < 9; ++t) {
            const int dwi = p.dw[t] + 1, dhi = p.dh[t] + 1;
            if (dwi < 0 || dwi > 2 || dhi < 0 || dhi > 2) { rows = false; break; }
            p.rows_tap[dwi * 3 + dhi] = t;
        }
        for (int i = 0; i < 9; ++i) rows = rows && p.rows_tap[i] >= 0;
    }
    // three stages: four or five (they fit) change the forward pass by 3 % and the step not at all
    if (rows && n_tile == 64 && p.Cn == 64 && p.kchunks == 1) return launch_km<64, 3, 4, 1, true, 72>(*m.a_rows, *m.b, o, p, s);
    if (rows && n_tile == 128 && p.kchunks >= 2 && m.b_half && even) return launch_km_pair<128, 4, 4, 1, true>(*m.a_rows, *m.b_half, o, p, s);
    // measured on a B200: the narrow tiles run best with two CTAs per SM and short pipelines (3 x 24 KB, 2 x 32 KB stages);
    // the 256-column tile as a CTA pair with six 32 KB stages; more sub-blocks per stage changed nothing
    if (m.b_half && n_tile == 256 && even) return launch_km_pair<256, 6, 4, 1, false>(*m.a, *m.b_half, o, p, s);
    if (n_tile == 64) return launch_km<64, 3, 4, 1, false, 0>(*m.a, *m.b, o, p, s);
    if (n_tile == 128) return launch_km<128, 2, 4, 1, false, 0>(*m.a, *m.b, o, p, s);
    if (n_tile == 256) return launch_km<256, 4, 4, 1, false, 0>(*m.a, *m.b, o, p, s);
    return cudaErrorInvalidValue;
}

template <int N_TILE, int STAGES>
static cudaError_t launch_wg(const TensorMap& x, const TensorMap& dy, const WgParams& p, dim3 grid, cudaStream_t s) {
    constexpr int smem = STAGES * (2 + N_TILE / 64) * 8192 + 1024 + 256;
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(wg_kernel<N_TILE, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    wg_kernel<N_TILE, STAGES><<<grid, NUM_THREADS, smem, s>>>(*(const CUtensorMap*)&x, *(const CUtensorMap*)&dy, p);
    return cudaGetLastError();
}

cudaError_t run_wg(const TensorMap& x, const TensorMap& dy, const WgParams& p, int n_tile, int splits, float* dw, bool accum, cudaStream_t s) {
    dim3 grid((p.row_blocks + 1) / 2, p.Co / n_tile, splits);
    cudaError_t e;
    if (n_tile == 64) e = launch_wg<64, 4>(x, dy, p, grid, s);      // 96 KB of stages: two CTAs per SM
    else if (n_tile == 128) e = launch_wg<128, 5>(x, dy, p, grid, s);
    else if (n_tile == 256) e = launch_wg<256, 4>(x, dy, p, grid, s);
    else return cudaErrorInvalidValue;
    if (e != cudaSuccess) return e;
    dim3 rgrid(p.row_blocks * 8, p.Co / 32), rblk(32, 8);
    wg_reduce_kernel<<<rgrid, rblk, 0, s>>>(p.partial, dw, splits, p.row_blocks, p.Co, accum);
    return cudaGetLastError();
}

template <int N_TILE, int NX, int XSUB_KB, int STAGES>
static cudaError_t launch_wg2(const TensorMap& x, const TensorMap& dy, const Wg2Params& p, dim3 grid, cudaStream_t s) {
    constexpr int smem = STAGES * (NX * XSUB_KB * 1024 + (N_TILE / 64) * 128 * 128) + 1024 + 256;
    static_assert(smem <= 232448, "shared memory");
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(wg2_kernel<N_TILE, NX, XSUB_KB, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    wg2_kernel<N_TILE, NX, XSUB_KB, STAGES><<<grid, NUM_THREADS, smem, s>>>(*(const CUtensorMap*)&x, *(const CUtensorMap*)&dy, p);
    return cudaGetLastError();
}

int wg_rows_variant(int H, int W, int C, int Co) {
    if (C == 64 && Co % 64 == 0 && W == 32 && H % 4 == 0) return 1;                               // nine taps of a 64-channel input, 64 columns
    if (C % 128 == 0 && Co % 128 == 0 && ((W == 16 && H % 8 == 0) || (W == 8 && H == 8))) return 2;  // one shift, two chunks, 128 columns
    return 0;
}

int wg_rows_splits(int variant, int C, int Co, long steps, int sms) {
    const int tiles = variant == 1 ? Co / 64 : 3 * (C / 128) * (Co / 128);
    long s = sm_count(sms) / tiles;
    if (s < 1) s = 1;
    if (s > steps) s = steps;
    const long per = (steps + s - 1) / s;
    return (int)((steps + per - 1) / per);
}

cudaError_t run_wg_rows(const TensorMap& x_rows, const TensorMap& dy128, const WgRowsParams& q, int variant, int splits, float* dw, bool accum,
                        cudaStream_t s) {
    Wg2Params p{};
    p.W = q.W; p.Ht = q.Ht; p.Nt = q.Nt; p.tiles_h = q.tiles_h; p.tiles_n = q.tiles_n; p.n_base = q.n_base;
    p.ptiles = q.tiles_h * q.tiles_n; p.ptiles_per_split = (p.ptiles + splits - 1) / splits;
    p.kchunks = q.C / 64; p.row_blocks = 9 * p.kchunks; p.Co = q.Co; p.partial = q.partial; p.err = q.err;
    const int z = (p.ptiles + p.ptiles_per_split - 1) / p.ptiles_per_split;
    cudaError_t e;
    if (variant == 1) e = launch_wg2<64, 3, 24, 2>(x_rows, dy128, p, dim3(1, q.Co / 64, z), s);
    else if (variant == 2) e = launch_wg2<128, 2, 20, 3>(x_rows, dy128, p, dim3(3 * (q.C / 128), q.Co / 128, z), s);
    else return cudaErrorInvalidValue;
    if (e != cudaSuccess) return e;
    dim3 rgrid(p.row_blocks * 8, p.Co / 32), rblk(32, 8);
    wg_reduce_kernel<<<rgrid, rblk, 0, s>>>(p.partial, dw, z, p.row_blocks, p.Co, accum);
    return cudaGetLastError();
}

bool make_map_raw_rows(TensorMap* out, const void* base, int C, int W, int H, int N, int box_rows) {
    if (!init()) return false;
    cuuint64_t dims[3] = {(cuuint64_t)W * C, (cuuint64_t)H, (cuuint64_t)N};
    cuuint64_t strides[2] = {(cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    cuuint32_t box[3] = {(cuuint32_t)(W * C), (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool stem_wg_supported(int H, int W, int C, int Co) {
    return C == 3 && Co % 64 == 0 && (W == 32 || W == 16) && H % (128 / W) == 0 && (W * C * 2) % 16 == 0 && (128 / W + 2) * W * 6 <= STEM_RAW_BYTES;
}
int stem_wg_ctas(long steps, int sms) { const long n = sm_count(sms); return (int)(steps < n ? steps : n); }
size_t stem_wg_workspace_elems(int Co, long steps, int sms) { return (size_t)(Co / 64) * stem_wg_ctas(steps, sms) * 64 * 64; }

cudaError_t run_stem_wg(const TensorMap& x_raw, const TensorMap& dy128, int H, int W, int N, int Co, float* partial, float* dw, bool accum, int* err,
                        int sms, cudaStream_t s) {
    constexpr int STAGES = 4;
    constexpr int smem = STAGES * (2 * 128 * 128 + STEM_RAW_BYTES) + 1024 + 256;
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(stem_wg_kernel<STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    StemWgParams p{};
    p.W = W; p.Ht = 128 / W; p.tiles_h = H / p.Ht; p.steps = N * p.tiles_h;
    const int ctas = stem_wg_ctas(p.steps, sms);
    p.steps_per_cta = (p.steps + ctas - 1) / ctas;
    p.partial = partial; p.err = err;
    stem_wg_kernel<STAGES><<<dim3(ctas, Co / 64), NUM_THREADS, smem, s>>>(*(const CUtensorMap*)&x_raw, *(const CUtensorMap*)&dy128, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    stem_wg_reduce_kernel<<<(Co * 27 + 127) / 128, 128, 0, s>>>(partial, dw, ctas, Co, accum);
    return cudaGetLastError();
}

cudaError_t run_stem_fw(const TensorMap& x_raw, const TensorMap& out_map, int H, int W, int N, int Co, const void* w, const float* bias, bool relu,
                        float* stat_part, int* err, int sms, cudaStream_t s) {
    constexpr int STAGES = 3;
    constexpr int smem = STAGES * (128 * 128 + STEM_RAW_BYTES) + 64 * 128 + 4 * 2 * EPI_BUF_BYTES + 1024 + 256;
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(stem_fw_kernel<STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    StemFwParams p{};
    p.W = W; p.Ht = 128 / W; p.tiles_h = H / p.Ht; p.tiles = N * p.tiles_h; p.Co = Co; p.epi = relu ? EPI_RELU : 0;
    p.w = (const bf16*)w; p.bias = bias; p.stat_part = stat_part; p.err = err;
    const int slots = 2 * sm_count(sms);
    stem_fw_kernel<STAGES><<<dim3(p.tiles < slots ? p.tiles : slots, Co / 64), 320, smem, s>>>(*(const CUtensorMap*)&x_raw, *(const CUtensorMap*)&out_map, p);
    return cudaGetLastError();
}

cudaError_t run_flip_transpose(const void* w, void* wt, int Co, int taps, int Ci, cudaStream_t s) {
    dim3 grid(Ci / 32, Co / 32, taps), blk(32, 8);
    flip_transpose_kernel<<<grid, blk, 0, s>>>((const bf16*)w, (bf16*)wt, Co, taps, Ci);
    return cudaGetLastError();
}

}  // namespace tc
}  // namespace fdg
