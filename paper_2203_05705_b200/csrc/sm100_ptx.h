// PTX wrappers for the sm_100a tensor-core kernels: mbarriers with bounded waits, TMA loads, tensor
// memory, tcgen05.mma and the shared-memory / instruction descriptors.  Included by the kernels of
// this library only; everything is static to the including translation unit.
#pragma once

#include "ard_internal.h"

namespace {

constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;  // every wait gives up after 2 s
constexpr int UMMA_BM = 128;                                  // accumulator rows of one CTA

// ---- PTX wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, P;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// One poll of the barrier.  With a suspend-time hint the hardware parks the thread until the phase
// completes or about `hint_ns` have passed, so a waiting thread neither spins on the barrier nor
// competes for issue slots.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], %2, %3;\n\t"
      "selp.b32 %0, 1, 0, P;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(hint_ns)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false if the limit expired or another role already gave up.
// Reading %globaltimer costs a few hundred nanoseconds, so the clock is consulted only after a first
// long poll has failed; a wait that is merely a pipeline hand-off never touches it.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  constexpr uint32_t HINT_NS = 1000000u;  // 1 ms per poll; the abort flag is looked at between polls
  if (mbar_try_wait(bar, parity)) return true;
  if (mbar_try_wait_hint(bar, parity, HINT_NS)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
    if (mbar_try_wait_hint(bar, parity, HINT_NS)) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > WAIT_LIMIT_NS) {
      *abort_flag = 1;
      atomicMax(status, (int)ARD_ERR_TIMEOUT);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
// Four rows of a 2-D tensor in one instruction (tile::gather4): rows y0..y3, columns x .. x + box width - 1 of a
// descriptor whose box is one row high; the four pieces land one after the other at `dst` (4 x box bytes, counted
// on `bar`).  A row index outside the tensor delivers zeros.
__device__ __forceinline__ void tma_gather4_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y0, int y1,
                                               int y2, int y3) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y0), "r"(y1), "r"(y2), "r"(y3)
      : "memory");
}
__device__ __forceinline__ void tensormap_acquire(const CUtensorMap* map) {
  asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(map) : "memory");
}

__device__ __forceinline__ uint32_t sm_id() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%smid;" : "=r"(r));
  return r;
}

// Turns the whole-matrix descriptor `m` (a kernel parameter) into the descriptor of the pattern (dp, b, n_keep)
// and returns the address the TMA instructions of this CTA should use: the parameter itself when nothing
// changes (a plain descriptor, a dense pattern), else `slot` (global memory written by this CTA only), which
// receives a copy whose address, extent and row pitch were replaced:
//   MAP_STRIDED_ROWS  rows b-1, b-1+dp, ...: address + (b-1) rows, n_keep rows, pitch dp rows (Eq. 1);
//   MAP_COMPACT_COLS  columns 0 .. n_keep-1 (beyond them TMA fills zeros); a dense pattern reads dense_base.
// Called by all 32 lanes of ONE warp with the same arguments.  `stmp`: 128 bytes of shared memory, 128-byte
// aligned, not in use by anyone else (callers pass the start of an operand stage before the first load).  Every
// thread that later issues a copy through the returned address calls tensormap_acquire on it first.
__device__ __forceinline__ const CUtensorMap* tensormap_specialise(const TcMap* m, int dp, int b, int n_keep,
                                                                   uint8_t* stmp, CUtensorMap* slot, int lane) {
  const int variant = m->variant;
  const bool dense_elsewhere = variant == MAP_COMPACT_COLS && dp == 1 && m->dense_base != nullptr;
  if (variant == MAP_PLAIN || (dp == 1 && !dense_elsewhere)) return &m->tm;
  reinterpret_cast<uint32_t*>(stmp)[lane] = reinterpret_cast<const uint32_t*>(&m->tm)[lane];
  __syncwarp();
  const uint64_t sdesc = (uint64_t)smem_u32(stmp);
  if (lane == 0) {
    if (variant == MAP_STRIDED_ROWS) {
      const uint64_t addr = reinterpret_cast<uint64_t>(m->base) + (uint64_t)(b - 1) * (uint64_t)m->ld * 2ull;
      asm volatile("tensormap.replace.tile.global_address.shared::cta.b1024.b64 [%0], %1;" ::"l"(sdesc), "l"(addr) : "memory");
      asm volatile("tensormap.replace.tile.global_dim.shared::cta.b1024.b32 [%0], 1, %1;" ::"l"(sdesc), "r"(n_keep) : "memory");
      asm volatile("tensormap.replace.tile.global_stride.shared::cta.b1024.b64 [%0], 0, %1;"
                   ::"l"(sdesc), "l"((uint64_t)dp * (uint64_t)m->ld * 2ull) : "memory");
    } else {
      if (dense_elsewhere) {
        asm volatile("tensormap.replace.tile.global_address.shared::cta.b1024.b64 [%0], %1;"
                     ::"l"(sdesc), "l"(reinterpret_cast<uint64_t>(m->dense_base)) : "memory");
        asm volatile("tensormap.replace.tile.global_stride.shared::cta.b1024.b64 [%0], 0, %1;"
                     ::"l"(sdesc), "l"((uint64_t)m->dense_ld * 2ull) : "memory");
      }
      asm volatile("tensormap.replace.tile.global_dim.shared::cta.b1024.b32 [%0], 0, %1;" ::"l"(sdesc), "r"(n_keep) : "memory");
    }
  }
  __syncwarp();
  // copy to global memory and release it to the tensor-map proxy at GPU scope (one fused, warp-wide instruction)
  asm volatile("tensormap.cp_fenceproxy.global.shared::cta.tensormap::generic.release.gpu.sync.aligned [%0], [%1], 128;"
               ::"l"(slot), "r"((uint32_t)sdesc) : "memory");
  return slot;
}

// Where tensormap_specialise leaves (or finds) the descriptor, without doing anything: for a second thread that
// issues copies through the same descriptors.
__device__ __forceinline__ const CUtensorMap* tensormap_specialised_address(const TcMap* m, int dp, const CUtensorMap* slot) {
  const int variant = m->variant;
  const bool dense_elsewhere = variant == MAP_COMPACT_COLS && dp == 1 && m->dense_base != nullptr;
  if (variant == MAP_PLAIN || (dp == 1 && !dense_elsewhere)) return &m->tm;
  return slot;
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- CTA-pair (cluster of 2, cta_group::2) forms ---------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in the CTA of rank `rank`
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load issued inside a CTA pair: the data lands in this CTA, the byte count is reported to the
// mbarrier at `bar_cluster`, which may live in the peer CTA.  The data goes to this CTA only.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int x,
                                                 int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Arrives on the mbarrier at the same shared-memory offset in every CTA of `mask` once the MMAs issued
// so far by this thread have completed.
__device__ __forceinline__ void tc_commit2(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask)
               : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, Blackwell version field = 1.
//   K-major operand : rows of 128 bytes, 8-row groups 1024 bytes apart (SBO); LBO unused (1).
//   MN-major operand: 64-element chunks along M/N `lbo` bytes apart; 8-row K groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

__host__ __device__ constexpr uint32_t make_idesc(int n, bool a_mn, bool b_mn, int m = UMMA_BM) {
  return (1u << 4)                      // D format fp32
         | (1u << 7)                    // A format bf16
         | (1u << 10)                   // B format bf16
         | ((a_mn ? 1u : 0u) << 15)     // A major
         | ((b_mn ? 1u : 0u) << 16)     // B major
         | ((uint32_t)(n >> 3) << 17)   // N
         | ((uint32_t)(m >> 4) << 24);  // M (256 for a CTA pair)
}

}  // namespace

// ---- non-bulk asynchronous copies (row gathers: a TMA box cannot follow an index list) -------------------
// 16 bytes global -> shared; src_bytes = 0 writes zeros and reads nothing.
__device__ __forceinline__ void cp_async_16(uint32_t dst_smem, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}
// Arrives on the barrier once all earlier cp.async of this thread have landed; the barrier's expected count
// must already include this arrival.
__device__ __forceinline__ void cp_async_mbar_arrive_noinc(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
// Orders what the generic proxy wrote to shared memory (and this thread has observed) before later reads of
// the async proxy (tcgen05.mma operands).
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
