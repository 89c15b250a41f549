// Device-side building blocks for the sm_100a tensor-core kernels: mbarrier
// waits with a time limit, TMA loads (tiled and im2col), tcgen05 MMA issue,
// commit, TMEM allocation and TMEM loads, shared-memory matrix descriptors.
// Everything is inline PTX; no library code.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace vgg {
namespace tc {

// A wait gives up after this long (far above any tile's duration, profiler
// replays included), records a DeviceError code and lets the CTA drain.
constexpr long long kWaitLimitCycles = 4000ll * 1000ll * 1000ll;  // about two seconds of SM clock

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// ---- mbarrier ---------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Wait for the phase with the given parity.  Returns false if another role has
// already given up (abort flag in shared memory) or if this wait ran out, in
// which case `code` is recorded in the device error word.  The limit is counted
// on the SM's own cycle counter, which is cheap to read; the global nanosecond
// timer costs on the order of a microsecond per read and would sit on the
// critical path of every hand-off.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* dev_error, int code, long long limit_cycles = kWaitLimitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 32; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit_cycles) {
      *abort_flag = 1;
      atomicCAS(dev_error, 0, code);
      return false;
    }
  }
}

// ---- TMA --------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// Tiled load of a [1][box_h][box_w][channels] box of an NHWC tensor; coordinates
// outside the tensor (a halo of the padding) read as zero.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c, int w, int h,
                                            int n) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n)
      : "memory");
}
// Tiled store of a [1][box_h][box_w][channels] box from shared memory (bulk async group).
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c, int w, int h, int n) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(map), "r"(src), "r"(c), "r"(w), "r"(h), "r"(n)
               : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Wait until all but `N` of this thread's store groups have finished READING shared memory.
template <int N>
__device__ __forceinline__ void tma_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// Barrier `id` over `threads` threads that also ORs a predicate: every participant gets the same
// answer, so a group of warps can leave a loop together.
__device__ __forceinline__ bool named_bar_or(int id, int threads, bool pred) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %3, 0;\n\t"
      "bar.red.or.pred q, %1, %2, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(out)
      : "r"(id), "r"(threads), "r"((uint32_t)pred)
      : "memory");
  return out != 0;
}
// im2col load of a [pixels][channels] box of an NHWC tensor: starts at pixel
// (n, h, w) of the bounding box, shifted by the filter offsets (off_w, off_h).
__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c, int w,
                                                   int h, int n, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], "
      "[%2], {%7, %8};"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---- tcgen05 ----------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t cols) {  // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {  // whole warp
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {  // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], bf16 x bf16 -> fp32, issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Same, always accumulating (no predicate to set up from a run-time value).
__device__ __forceinline__ void umma_bf16_acc(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.eq.b32 p, 0, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc)
      : "memory");
}
// A descriptor whose start address is `bytes` further on (bytes a multiple of 16, no carry out of
// the 14-bit address field): one 64-bit add instead of rebuilding the descriptor.
__device__ __forceinline__ uint64_t desc_advance(uint64_t desc, uint32_t bytes) { return desc + (uint64_t)(bytes >> 4); }
// The mbarrier gets one arrival once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets lane
// (lane base + i), register j = column (column base + j).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t addr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(addr)
      : "memory");
}
// 32 lanes x 16 consecutive fp32 columns.
__device__ __forceinline__ void tmem_ld_32x16(uint32_t addr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(addr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- 2x2 max-pool in an epilogue ----------------------------------------------
// The four values of a window sit in four lanes: this one (top left), lane + dx (its right neighbour),
// lane + dy (below), lane + dx + dy.  v[] holds WORDS bf16 pairs (2 * WORDS channels) of this lane's pixel
// and comes back as the window's maxima (meaningful in the top-left lane).
template <int WORDS>
__device__ __forceinline__ void pool2x2(uint32_t (&v)[WORDS], int dx, int dy) {
#pragma unroll
  for (int i = 0; i < WORDS; ++i) {
    __nv_bfloat162 m = *reinterpret_cast<__nv_bfloat162*>(&v[i]);
    uint32_t o = __shfl_down_sync(0xffffffffu, v[i], dx);
    m = __hmax2(m, *reinterpret_cast<__nv_bfloat162*>(&o));
    uint32_t mb = *reinterpret_cast<uint32_t*>(&m);
    o = __shfl_down_sync(0xffffffffu, mb, dy);
    m = __hmax2(m, *reinterpret_cast<__nv_bfloat162*>(&o));
    v[i] = *reinterpret_cast<uint32_t*>(&m);
  }
}
// The same, also giving each channel's arg-max code, one byte per channel in codes[] (four channels per
// word): 0..3 for the window positions (0,0), (0,1), (1,0), (1,1), the first maximum in that order on
// ties, or 4 when the maximum is not positive.  All comparisons are two channels at a time; the lower
// row's left-or-right decisions come up as one word of flag bits (WORDS <= 16).
template <int WORDS>
__device__ __forceinline__ void pool2x2_codes(uint32_t (&v)[WORDS], int dx, int dy, uint32_t (&codes)[WORDS / 2]) {
  static_assert(WORDS <= 16 && WORDS % 2 == 0, "flag bits i and 16 + i per word");
  uint32_t left[WORDS];  // per half 0xFFFF where the left value of this lane's row is >= the right one
  uint32_t flags = 0;
#pragma unroll
  for (int i = 0; i < WORDS; ++i) {
    const uint32_t right = __shfl_down_sync(0xffffffffu, v[i], dx);
    const __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&v[i]), b = *reinterpret_cast<const __nv_bfloat162*>(&right);
    left[i] = __hge2_mask(a, b);
    const __nv_bfloat162 m = __hmax2(a, b);
    v[i] = *reinterpret_cast<const uint32_t*>(&m);
    flags |= (left[i] & 0x00010001u) << i;
  }
  const uint32_t flags_below = __shfl_down_sync(0xffffffffu, flags, dy);
  const uint32_t zero2 = 0u;
  uint32_t k16[WORDS];  // the code of each channel in its 16-bit half
#pragma unroll
  for (int i = 0; i < WORDS; ++i) {
    const uint32_t below = __shfl_down_sync(0xffffffffu, v[i], dy);
    const __nv_bfloat162 t = *reinterpret_cast<__nv_bfloat162*>(&v[i]), b = *reinterpret_cast<const __nv_bfloat162*>(&below);
    const uint32_t top = __hge2_mask(t, b);  // the upper row holds the (first) maximum
    const __nv_bfloat162 m = __hmax2(t, b);
    v[i] = *reinterpret_cast<const uint32_t*>(&m);
    const uint32_t left_below = ((flags_below >> i) & 0x00010001u) * 0xFFFFu;
    const uint32_t is_left = (top & left[i]) | (~top & left_below);
    uint32_t k = (~top & 0x00020002u) | (~is_left & 0x00010001u);
    const uint32_t positive = __hgt2_mask(m, *reinterpret_cast<const __nv_bfloat162*>(&zero2));
    k16[i] = (k & positive) | (~positive & 0x00040004u);
  }
#pragma unroll
  for (int j = 0; j < WORDS / 2; ++j) codes[j] = __byte_perm(k16[2 * j], k16[2 * j + 1], 0x6420);
}

// ---- CTA pairs (cluster of two, tcgen05 cta_group::2) --------------------------
// One MMA spans both CTAs of the pair: each supplies its own 128 rows of A and half of the B tile
// from its own shared memory and holds its 128 accumulator rows in its own tensor memory.  The even
// CTA (cluster rank 0) issues; barriers the issuer waits on live in its shared memory.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in the CTA of rank `rank`
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync_all() { cluster_arrive(); cluster_wait(); }
// Arrival on a barrier given by its shared::cluster address (this CTA's or the peer's).  Relaxed: it
// publishes no memory, only the fact that this CTA's tcgen05.ld of an accumulator buffer have
// completed (tcgen05.wait::ld, then tcgen05.fence::before_thread_sync, come first).  A release at
// cluster scope would wait for every global store the thread still has in flight.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// Loads whose completion bytes are counted on a barrier given by its shared::cluster address,
// which may be the peer's; the data lands in this CTA's shared memory.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int c0, int c1,
                                                 int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int c, int w,
                                                 int h, int n) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c), "r"(w), "r"(h), "r"(n)
      : "memory");
}
__device__ __forceinline__ void tma_load_im2col_4d_pair(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int c,
                                                        int w, int h, int n, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], "
      "[%2], {%7, %8};"
      ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_result, uint32_t cols) {  // one whole warp in each CTA
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair_acc(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.eq.b32 p, 0, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc)
      : "memory");
}
// One arrival, once the pair's MMAs issued so far have finished, on the barrier at this
// shared-memory offset in each CTA of `cta_mask` (bit per cluster rank).
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint16_t cta_mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(cta_mask)
               : "memory");
}

// Shared-memory matrix descriptor for a 128-byte-swizzled operand tile whose
// rows are 128 bytes (64 bf16) and whose 8-row groups are 1024 bytes apart.
//   K-major operand  : a row is one M/N index, the 64 elements run along K.
//   MN-major operand : a row is one K index, the 64 elements run along M/N;
//                      `lbo_bytes` is the distance between 64-element M/N groups.
// Fields (PTX "matrix descriptor"): start address >> 4 in bits 0-13, leading
// byte offset >> 4 in bits 16-29, stride byte offset >> 4 in bits 32-45,
// descriptor version 1 in bits 46-47, swizzle mode 2 (128 B) in bits 61-63.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((1024u >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// The general form: leading byte offset and stride byte offset both given (128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc_sw128_full(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Same for a K-major operand whose 8-row groups are `sbo_bytes` apart (rows of a
// group still 128 bytes apart).  The start address may be any multiple of 128
// bytes inside a 1024-byte-aligned buffer: the 128-byte swizzle is a function
// of the absolute shared-memory address, for the copy engine and the MMA alike.
__device__ __forceinline__ uint64_t smem_desc_sw128_sbo(uint32_t addr, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Descriptor of an operand stored without swizzle as 8 x 16-byte "core
// matrices" (8 rows of 8 bf16, 128 contiguous bytes).
//   K-major : lbo = distance between the two 8-element K chunks of one MMA,
//             sbo = distance between 8-row groups along M/N.
//   MN-major: lbo = distance between 8-row groups along K,
//             sbo = distance between 8-element groups along M/N.
__device__ __forceinline__ uint64_t smem_desc_plain(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}

// Instruction descriptor of tcgen05.mma kind::f16: bf16 A and B, fp32 D.
// D format fp32 (bits 4-5 = 1), A/B format bf16 (bits 7-9, 10-12 = 1),
// A / B major (bit 15 / 16: 0 = K-major, 1 = MN-major), N >> 3 in bits 17-22,
// M >> 4 in bits 24-28.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// the same with fp16 A and B (format 0 in both fields)
__host__ __device__ constexpr uint32_t umma_idesc_f16(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

}  // namespace tc

// ---- host side: tensor maps --------------------------------------------------
// The driver entry points are looked up at run time so that the library does
// not link against libcuda.
struct TensorMapApi {
  CUresult (*encode_tiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                           const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                           CUtensorMapL2promotion, CUtensorMapFloatOOBfill) = nullptr;
  CUresult (*encode_im2col)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                            const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*, CUtensorMapInterleave,
                            CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill) = nullptr;
  bool ok = false;
};
const TensorMapApi& tensor_map_api();

// [rows][cols] bf16 row-major matrix, box = box_rows x 64 columns, 128 B swizzle.
bool make_tiled_map_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// [rows][cols] fp32 row-major matrix, box = box_rows x 32 columns (128 bytes), 128 B swizzle.
bool make_tiled_map_2d_f32(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// Same with a box of box_rows x 8 columns (16 bytes) and no swizzle.
bool make_tiled_map_2d_c8(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// Tap-major filter [9][Cout][Cin] bf16: box = 3 taps x box_cout rows x 64 channels, 128 B swizzle.
bool make_filter_row_map(CUtensorMap* map, const void* base, int Cout, int Cin, uint32_t box_cout);
// NHWC bf16 tensor, tiled box of box_h x box_w pixels x 64 channels, 128 B swizzle.
bool make_patch_map(CUtensorMap* map, const void* base, int N, int H, int W, int C, uint32_t box_w, uint32_t box_h);
// One of the four 2x2 window positions (a, b) of an NHWC bf16 tensor [N][H][W][C] as a tensor of its
// own: [N][H/2][W/2][C] whose pixel (h, w) is pixel (2h + a, 2w + b) of the tensor; box as above.
bool make_window_map(CUtensorMap* map, const void* base, int N, int H, int W, int C, int a, int b, uint32_t box_w,
                     uint32_t box_h);
// NHWC bf16 tensor read through a 3x3 / pad 1 window: box = `pixels` x 64 channels, 128 B swizzle.
bool make_im2col_map(CUtensorMap* map, const void* base, int N, int H, int W, int C, uint32_t pixels);
// NHWC bf16 tensor with 8 channels, tiled box of box_h x box_w pixels x 8 channels, no swizzle.
bool make_patch_map_c8(CUtensorMap* map, const void* base, int N, int H, int W, uint32_t box_w, uint32_t box_h);
// Same for a tensor with 8 channels: box = `pixels` x 8 channels (16 bytes), no swizzle.
bool make_im2col_map_c8(CUtensorMap* map, const void* base, int N, int H, int W, uint32_t pixels);

}  // namespace vgg
