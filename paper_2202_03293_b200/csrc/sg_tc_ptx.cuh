// PTX wrappers shared by the tensor-core kernels of this library (sm_100a): mbarriers with
// bounded waits, TMA loads and stores, tcgen05 MMA / TMEM access, shared-memory matrix and
// instruction descriptors, cluster helpers.  Included by one .cu file per kernel family; every
// translation unit gets its own device status word.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sg.h"

namespace sg {
namespace {

constexpr long long WAIT_BUDGET_CYCLES = 2000000000LL;   // ~1 s: far beyond any legitimate wait

// Bit 0 is set by a kernel of this translation unit whose bounded wait expired.
__device__ unsigned int g_status_word = 0;


// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Same test with cluster-scope acquire: the barrier was signalled by threads of the peer CTA
// whose shared-memory writes must be visible afterwards.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the budget (in SM clock cycles) expired or another role already aborted.
template <bool CLUSTER_SCOPE = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          long long budget_cycles = WAIT_BUDGET_CYCLES) {
    auto test = [&]() { return CLUSTER_SCOPE ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity); };
    if (test()) return true;
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        if (test()) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > budget_cycles) {
                *abort_flag = 1;
                atomicOr(&g_status_word, 1u);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, int z, int w) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
// im2col mode: coordinates name the first base pixel (c, w, [h,] n); the 16-bit offsets are
// added to every pixel's spatial coordinates (the filter tap's kw*dw, kh*dh).
__device__ __forceinline__ void tma_load_im2col_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                                   int c, int w, int n, unsigned short off_w) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2], {%6};"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(n), "h"(off_w) : "memory");
}
__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                                   int c, int w, int h, int n, unsigned short off_w, unsigned short off_h) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap *map, uint32_t src, int x, int y) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], 128 x N x 16, bf16 inputs, f32 accumulate.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Same shape with tf32 inputs (f32 words in shared memory, k extent 8).
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the mbarrier once every tcgen05.mma issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// This warp's 32 lanes x 32 consecutive f32 columns of TMEM -> 32 registers per thread.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
// This warp's 32 lanes x 16 consecutive 32-bit columns of TMEM <- 16 registers per thread.
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
// ... and 8 consecutive columns <- 8 registers per thread.
__device__ __forceinline__ void tmem_st_32x8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem]: the A operand (128 lanes = rows, 8 columns = k) read from tensor memory.
__device__ __forceinline__ void umma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_tf32_ts_cg2(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// ... and 4 consecutive columns <- 4 registers per thread.
__device__ __forceinline__ void tmem_st_32x4(uint32_t taddr, const uint32_t (&r)[4]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem], bf16 inputs: the A operand's 128 rows x 16 k sit in 8 tensor-memory columns, two
// consecutive k per 32-bit column (the even k in the low half).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_bf16_ts_cg2(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format): start address, leading and stride byte
// offsets (all >> 4), descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;   // version
    d |= (uint64_t)2 << 61;   // SWIZZLE_128B
    return d;
}

// Instruction descriptor: f32 accumulator, A and B both bf16 (kind::f16) or both tf32
// (kind::tf32); each operand K-major, or MN-major (its rows/columns contiguous in shared memory
// instead of k; kind::tf32 takes K-major operands only: an MN-major descriptor makes the MMA a
// no-op there).
__host__ __device__ constexpr uint32_t make_idesc(int n, int m, bool tf32, bool a_mn_major, bool b_mn_major) {
    return (1u << 4)                       // D format: f32
         | ((tf32 ? 2u : 1u) << 7)         // A format: bf16 = 1 in kind::f16, tf32 = 2 in kind::tf32
         | ((tf32 ? 2u : 1u) << 10)        // B format: the same type as A
         | ((a_mn_major ? 1u : 0u) << 15)  // A major
         | ((b_mn_major ? 1u : 0u) << 16)  // B major
         | ((uint32_t)(n >> 3) << 17)      // N / 8
         | ((uint32_t)(m >> 4) << 24);     // M / 16 (128 for one CTA, 256 for a pair)
}

// ---- cluster helpers (CG = 2) ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Arrive on a barrier of another CTA of the cluster.  Default semantics (release at CTA scope):
// what the arriving thread wrote before goes to its own CTA's shared memory, which the
// tensor core reads after a proxy fence; a cluster-scope release costs a full memory barrier
// per arrive (measured: 1.6x on the whole f32 kernel) and orders nothing more that is needed.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA loads whose completion may be signalled on the peer CTA's mbarrier (cta_group::2).
__device__ __forceinline__ void tma_load_2d_cg2(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_load_4d_cg2(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, int z, int w) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void tma_load_im2col_3d_cg2(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                                       int c, int w, int n, unsigned short off_w) {
    asm volatile(
        "cp.async.bulk.tensor.3d.im2col.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2], {%6};"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(n), "h"(off_w) : "memory");
}
__device__ __forceinline__ void tma_load_im2col_4d_cg2(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                                       int c, int w, int h, int n, unsigned short off_w, unsigned short off_h) {
    asm volatile(
        "cp.async.bulk.tensor.4d.im2col.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h) : "memory");
}
// Rank-5 tiled load.  CG2: the mbarrier may belong to the peer CTA of a pair.  One TMA
// instruction costs the issuing thread several hundred cycles whatever the size of its box
// (measured: ~550 cycles, boxes of 8 to 64 KB), so operand tiles are fetched with as few and as
// large boxes as the layout allows, and the two operands are issued by different warps.
template <bool CG2>
__device__ __forceinline__ void tma_tile_5d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, int z, int w, int v) {
    if constexpr (CG2)
        asm volatile("cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
                     ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w), "r"(v) : "memory");
    else
        asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
                     ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w), "r"(v) : "memory");
}
template <bool CG2>
__device__ __forceinline__ void tma_tile_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, int z) {
    if constexpr (CG2)
        asm volatile("cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                     ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
    else
        asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                     ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}
// The four epilogue warps (128 threads, named barrier 1) agree on one answer: all of them reach this barrier whatever
// they found, so a bounded wait that one warp gave up on and another passed cannot leave them at different barriers.
__device__ __forceinline__ bool epilogue_all(bool mine) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out) : "r"((uint32_t)mine) : "memory");
    return out != 0;
}

// True in exactly one lane of the (converged) warp, the same lane on every call.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
// Starts the fetch of a tensor map (a kernel parameter) ahead of its first use.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
// D[tmem of both CTAs] (+)= A * B, 256 x N x 16 across the CTA pair.
__device__ __forceinline__ void umma_bf16_cg2(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_tf32_cg2(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives (once the pair's MMAs issued so far have finished) on a barrier that may live in
// either CTA of the pair; `cluster_bar` is a shared::cluster address.
__device__ __forceinline__ void umma_commit_cg2(uint32_t cluster_bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_bar) : "memory");
}


// ---------------------------------------------------------------- f32 inputs on the tensor cores: the hi/lo split
// 3xTF32 split of four f32 words.  hi = x rounded to the nearest tf32 value (10 mantissa bits;
// done on the bit pattern: add half an ulp, clear the low 13 bits); x - hi is exact in f32 and
// lo is that difference rounded to tf32 the same way, so x - hi - lo is below 2^-22 |x|.  The
// low bits of hi and lo are zero, so whatever rounding the tensor core applies to its inputs
// leaves them unchanged.  Words of magnitude >= 2^127 (where rounding up
// could reach infinity), infinities and NaNs take a slow path: hi truncated, lo = 0 unless
// finite.
__device__ __forceinline__ void split4(const uint4 v, uint4 &h, uint4 &l) {
    const float fx = __uint_as_float(v.x), fy = __uint_as_float(v.y), fz = __uint_as_float(v.z), fw = __uint_as_float(v.w);
    const float big = fmaxf(fmaxf(fabsf(fx), fabsf(fy)), fmaxf(fabsf(fz), fabsf(fw)));
    if (big < 1.7014118e38f) {
        h.x = (v.x + 0x1000u) & 0xFFFFE000u; l.x = (__float_as_uint(fx - __uint_as_float(h.x)) + 0x1000u) & 0xFFFFE000u;
        h.y = (v.y + 0x1000u) & 0xFFFFE000u; l.y = (__float_as_uint(fy - __uint_as_float(h.y)) + 0x1000u) & 0xFFFFE000u;
        h.z = (v.z + 0x1000u) & 0xFFFFE000u; l.z = (__float_as_uint(fz - __uint_as_float(h.z)) + 0x1000u) & 0xFFFFE000u;
        h.w = (v.w + 0x1000u) & 0xFFFFE000u; l.w = (__float_as_uint(fw - __uint_as_float(h.w)) + 0x1000u) & 0xFFFFE000u;
    } else {
        auto one = [](uint32_t x, uint32_t &hi, uint32_t &lo) {
            hi = x & 0xFFFFE000u;
            const float d = __uint_as_float(x) - __uint_as_float(hi);
            lo = (x & 0x7F800000u) == 0x7F800000u ? 0u : __float_as_uint(d);
        };
        one(v.x, h.x, l.x); one(v.y, h.y, l.y); one(v.z, h.z, l.z); one(v.w, h.w, l.w);
    }
}

// Packs two f32 values, rounded to the nearest bf16, into one word: `even` in the low half, `odd` in the high half.
__device__ __forceinline__ uint32_t pack_bf16(float even, float odd) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(odd), "f"(even));
    return d;
}
// The split used when the two correction products run as bf16 MMAs: x = hi + lo with hi = x rounded to tf32 (as above); the
// main product hi*hi runs in tf32, the corrections lo*hi + hi*lo with all four factors rounded to bf16.  A correction term
// is below 2^-11 of its product and bf16 keeps 8 bits of each factor, so the rounding moves a product by less than 2^-19 of
// itself (what the dropped lo*lo term and the tensor core's f32 accumulation cost already), and the two bf16 products of a k-block are one
// contraction over 64 values, [lo | hi] . [hi | lo], at twice the tf32 rate: two tensor-core units per term instead of three.
// Words of magnitude >= 2^127, infinities and NaNs: hi and its bf16 copy are truncated, never rounded up to infinity.
__device__ __forceinline__ void split4_mix(const uint4 v, uint4 &h, uint2 &h16, uint2 &l16) {
    const float fx = __uint_as_float(v.x), fy = __uint_as_float(v.y), fz = __uint_as_float(v.z), fw = __uint_as_float(v.w);
    const float big = fmaxf(fmaxf(fabsf(fx), fabsf(fy)), fmaxf(fabsf(fz), fabsf(fw)));
    if (big < 1.7014118e38f) {
        h.x = (v.x + 0x1000u) & 0xFFFFE000u; h.y = (v.y + 0x1000u) & 0xFFFFE000u;
        h.z = (v.z + 0x1000u) & 0xFFFFE000u; h.w = (v.w + 0x1000u) & 0xFFFFE000u;
        h16.x = pack_bf16(__uint_as_float(h.x), __uint_as_float(h.y));
        h16.y = pack_bf16(__uint_as_float(h.z), __uint_as_float(h.w));
        l16.x = pack_bf16(fx - __uint_as_float(h.x), fy - __uint_as_float(h.y));
        l16.y = pack_bf16(fz - __uint_as_float(h.z), fw - __uint_as_float(h.w));
    } else {
        auto one = [](uint32_t x, uint32_t &hi, uint32_t &hi16, uint32_t &lo16) {
            hi = x & 0xFFFFE000u;
            hi16 = x >> 16;
            const float d = __uint_as_float(x) - __uint_as_float(hi);
            lo16 = (x & 0x7F800000u) == 0x7F800000u ? 0u : (pack_bf16(d, 0.f) & 0xFFFFu);     // (small: rounding cannot overflow)
        };
        uint32_t a[4], b[4];
        one(v.x, h.x, a[0], b[0]); one(v.y, h.y, a[1], b[1]); one(v.z, h.z, a[2], b[2]); one(v.w, h.w, a[3], b[3]);
        h16.x = a[0] | (a[1] << 16); h16.y = a[2] | (a[3] << 16);
        l16.x = b[0] | (b[1] << 16); l16.y = b[2] | (b[3] << 16);
    }
}


// The same for eight values (two chunks of four): hi of each chunk, and the eight bf16 values of hi and of lo packed in k order.
__device__ __forceinline__ void split8_mix(const uint4 v0, const uint4 v1, uint4 &h0, uint4 &h1, uint4 &h16, uint4 &l16) {
    uint2 a, b, c, d;
    split4_mix(v0, h0, a, b);
    split4_mix(v1, h1, c, d);
    h16 = make_uint4(a.x, a.y, c.x, c.y);
    l16 = make_uint4(b.x, b.y, d.x, d.y);
}

// Reads and clears this translation unit's status word; the caller has synchronised the stream.
inline sg_status read_status_word(cudaStream_t stream) {
    unsigned int word = 0, zero = 0;
    if (cudaMemcpyFromSymbolAsync(&word, g_status_word, sizeof(word), 0, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return SG_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return SG_ERR_CUDA;
    if (word != 0) {
        if (cudaMemcpyToSymbolAsync(g_status_word, &zero, sizeof(zero), 0, cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return SG_ERR_CUDA;
        cudaStreamSynchronize(stream);
        return SG_ERR_DEVICE_TIMEOUT;
    }
    return SG_OK;
}

}  // namespace
}  // namespace sg
