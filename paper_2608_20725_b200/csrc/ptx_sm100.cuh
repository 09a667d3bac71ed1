// Inline-PTX wrappers for the sm_100a features the fp16 kernels use: mbarriers
// with bounded waits, TMA tile loads, tensor-memory allocation, tcgen05 MMA
// issue/commit and accumulator loads, and the shared-memory / instruction
// descriptors of the MMA.
#pragma once

#include <cuda.h>
#include <stdint.h>

#include "phase_timers.cuh"

namespace im2win {
namespace ptx {

constexpr uint32_t SPIN_LIMIT = 1u << 24;      // polls before a wait gives up (see mbar_wait)
constexpr uint32_t SPIN_CHUNK = 1024;          // polls between looks at the abort flag and the clock
constexpr uint64_t SPIN_TIME_NS = 4000000000ull;   // wall-time bound of one wait: 4 s
// Word 2 of the status block: this marker makes the one-k-block kernel's copy warp leave out one
// barrier arrival (the test of the bounded waits; nothing in the library writes it).
constexpr uint32_t kDebugDropArrive = 0x0d0a11feu;
// Word 2 again: with this marker the NHWC shifted-view kernel's first K part of a tile does not raise
// the tile's flag, so that the parts waiting for it run into their limit (same purpose).
constexpr uint32_t kDebugDropFlag = 0x0d0a11ffu;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Adds `bytes` to the barrier's pending transaction count without arriving.
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Untiled bulk copy global -> shared (both 16-byte aligned, size a multiple of 16), completion
// counted on an mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded waits.  A wait first polls SPIN_CHUNK times in line; only a wait that is still pending
// then (milliseconds: each poll may suspend the thread for a while) enters the slow path below,
// which gives up after SPIN_LIMIT polls or SPIN_TIME_NS of wall time, whichever comes first, or as
// soon as another thread of the CTA has given up.  Word 1 of the status block, when non-zero,
// replaces SPIN_LIMIT (a testing aid: the filter pack clears the block, a test may then lower the
// limit before the convolution runs).  On giving up the wait raises the CTA's abort flag and word
// 0 of the status block and returns false; the caller unwinds (drains its copies, frees its tensor
// memory) and the kernel returns normally.
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// The slow path is a function of its own by default (measured: the narrow-tile NHWC kernels lose 10-15 %
// when it is expanded at every wait); the one-k-block kernel defines IM2WIN_INLINE_SLOW_WAIT before
// including this header, because there the call costs more (a 3-channel 3x3 layer 1179 against 943 us).
#ifdef IM2WIN_INLINE_SLOW_WAIT
#define IM2WIN_SLOW_WAIT_ATTR __forceinline__
#else
#define IM2WIN_SLOW_WAIT_ATTR __noinline__
#endif
template <bool CLUSTER>
__device__ IM2WIN_SLOW_WAIT_ATTR bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                            uint32_t* status) {
  uint32_t limit = *reinterpret_cast<volatile uint32_t*>(status + 1);
  if (limit == 0u) limit = SPIN_LIMIT;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t i = SPIN_CHUNK; i < limit; i += SPIN_CHUNK) {
    for (uint32_t j = 0; j < SPIN_CHUNK; ++j) {
      uint32_t ok;
      if constexpr (CLUSTER) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
      } else {
        ok = mbar_try_wait(bar, parity);
      }
      if (ok) return true;
    }
    if (*abort_flag) return false;
    if (global_timer_ns() - t0 > SPIN_TIME_NS) break;
  }
  *abort_flag = 1u;
  atomicExch(status, 1u);
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status) {
  for (uint32_t i = 0; i < SPIN_CHUNK; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow<false>(bar, parity, abort_flag, status);
}
// True in exactly one lane of the (converged) warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// The same load without the wait, so that several can be in flight; tmem_ld_wait() before the
// registers are read.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// The wait for loads into r[]: naming the registers as in/out operands keeps every use of them after it.
__device__ __forceinline__ void tmem_ld_wait_for(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                 "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}

// Epilogue stores of one accumulator row: v[j] goes to base + j*stride floats for j < count (count
// may exceed 32).  Four independent address chains: with one running pointer every store waits for
// the 64-bit add before it (about 9 cycles per store, measured: 8 % of a whole output-bound layer).
__device__ __forceinline__ void store_strided32(float* base, int64_t stride, const uint32_t (&v)[32], int count) {
  float* p0 = base;
  float* p1 = p0 + stride;
  float* p2 = p1 + stride;
  float* p3 = p2 + stride;
  const int64_t step = 4 * stride;
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    if (j < count) *p0 = __uint_as_float(v[j]);
    if (j + 1 < count) *p1 = __uint_as_float(v[j + 1]);
    if (j + 2 < count) *p2 = __uint_as_float(v[j + 2]);
    if (j + 3 < count) *p3 = __uint_as_float(v[j + 3]);
    p0 += step; p1 += step; p2 += step; p3 += step;
  }
}

// Shared-memory matrix descriptor of a k-major tile whose rows are 128 bytes
// (64 halves) with the 128-byte swizzle: 8-row groups are 1024 bytes apart.
// The swizzle is a function of the shared-memory address, so a view may start
// at any row of a tile (and 32 bytes further per 16-element k step) as long as
// the tile itself is 1024-byte aligned; the base-offset field stays 0
// (measured: row-shifted views are exact with it clear, wrong with it set).
__device__ __forceinline__ uint64_t smem_desc_k_major_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3ffffu) >> 4);   // start address / 16
  d |= (uint64_t)1 << 16;                     // leading byte offset (unused with swizzle) = 16 B
  d |= (uint64_t)(1024 >> 4) << 32;           // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                     // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                     // 128-byte swizzle
  return d;
}
// The same descriptor split into its two 32-bit halves: the high half is the same for every
// k-major 128-byte-swizzled tile, and moving a view by 16 bytes adds 1 to the low half, so an
// MMA issue loop only does 32-bit adds.
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t saddr) {
  return ((saddr & 0x3ffffu) >> 4) | (1u << 16);
}
constexpr uint32_t kSmemDescHiSw128 = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ void umma_f16_lohi(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                              uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %5};\n\t"
      "mov.b64 db, {%2, %5};\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kSmemDescHiSw128)
      : "memory");
}

// K-major tile WITHOUT swizzle: 16-byte units (8 halves of one row) are the atoms; the 8 rows of
// a group lie 16 bytes apart, groups of 8 rows `sbo` bytes apart and the two 8-element halves of
// a 16-element k step `lbo` bytes apart.  With sbo = 128 the address is linear in the row, so a
// view may start at any row (16 bytes per row).  Low half: start address and lbo; high half: sbo.
__device__ __forceinline__ uint32_t smem_desc_lo_noswz(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr & 0x3ffffu) >> 4) | ((lbo_bytes >> 4) << 16);
}
constexpr uint32_t kSmemDescHiNoSwz128 = (uint32_t)(128 >> 4) | (1u << 14);
// MMA with separately described operands (A without swizzle, B with the 128-byte swizzle).
__device__ __forceinline__ void umma_f16_ab(uint32_t tmem_d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                            uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
      ::"r"(tmem_d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Four 8x8 matrices of 16-bit elements, shared memory -> registers, transposed on the way: lane l
// gives the address of row l%8 (16 bytes) of matrix l/8; afterwards lane i holds in r[t] the
// elements (row 2*(i%4), column i/4) and (row 2*(i%4)+1, column i/4) of matrix t.
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
// Four 8x8 matrices registers -> shared memory: lane i holds in r[t] the elements (row i/4,
// columns 2*(i%4), 2*(i%4)+1) of matrix t; lane l gives the address of row l%8 of matrix l/8.
__device__ __forceinline__ void stmatrix_x4(uint32_t addr, const uint32_t (&r)[4]) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(r[0]), "r"(r[1]),
               "r"(r[2]), "r"(r[3])
               : "memory");
}

// ---- CTA pairs (clusters of two CTAs that share one MMA) ------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster (shared::cluster window).
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// Arrive on an mbarrier given by a shared::cluster address (possibly in the other CTA).  Default
// semantics (release at CTA scope): what the arriving thread wrote is its own CTA's shared memory,
// read later by that CTA's tensor core; a cluster-scope release was measured to cost about a
// thousand cycles per arrival.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Wait on a local mbarrier whose arrivals may come from the other CTA (cluster-scope acquire).
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                  uint32_t* status) {
  for (uint32_t i = 0; i < SPIN_CHUNK; ++i)
    if (mbar_try_wait_cluster(bar, parity)) return true;
  return mbar_wait_slow<true>(bar, parity, abort_flag, status);
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Tensor memory of a CTA pair: one warp of EACH CTA issues these.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// MMA over both CTAs of a pair (issued by the leader CTA): M = 256 rows, 128 from each CTA's A
// tile; each CTA's B tile holds half of the N columns' rows.  Descriptors are shared-memory
// offsets valid in both CTAs.
__device__ __forceinline__ void umma_f16_ab_pair(uint32_t tmem_d, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                                 uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, p;\n\t}"
      ::"r"(tmem_d), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Commit of the pair's MMAs: arrives on the mbarrier at this offset in both CTAs.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
      "h"((uint16_t)3)
      : "memory");
}
// TMA tile load inside a CTA pair: the destination is this CTA's shared memory, the mbarrier may
// be the peer's (a shared::cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                                 uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar_cluster)
      : "memory");
}

// Instruction descriptor: fp16 A and B, both k-major, fp32 accumulator, M x N tile.
__host__ __device__ constexpr uint32_t instr_desc_f16(int M, int N) {
  return (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}


}  // namespace ptx
}  // namespace im2win
