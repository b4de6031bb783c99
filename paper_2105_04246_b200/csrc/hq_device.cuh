// Device-side primitives shared by the kernels: shared-memory addresses, mbarriers with bounded waits, TMA tile loads.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hq_internal.h"

namespace hq {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One try_wait; the hardware may suspend the thread for up to `hint_ns` while the phase is pending, which keeps
// waiting threads from flooding the memory-instruction queue that the MMA and TMA issue also go through.
__device__ __forceinline__ uint32_t mbar_try(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3; selp.u32 %0, 1, 0, p; }"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(hint_ns)
      : "memory");
  return ok;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait on an mbarrier phase.  Gives up when another role has already given up or after kWaitLimitCycles of this
// SM's own cycle counter (monotonic and private to the SM; the global nanosecond timer is shared with the host side and
// may be stepped while a kernel runs); the first to give up records `code` in the status word.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status, int code,
                                          uint32_t hint_ns = 200u) {
  if (mbar_try(bar, parity, hint_ns)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  for (;;) {
    if (mbar_try(bar, parity, hint_ns)) return true;
    // A pause between polls: the try above returns after some tens of nanoseconds even with a long hint, and a warp
    // that polls back to back takes issue slots from the epilogue warps of its scheduler.  A quarter of the hint keeps
    // the wake-up latency of waits on the critical path (short hints) small.
    __nanosleep(hint_ns >> 2);
    if ((++spins & 15u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitLimitCycles) {
        *abort_flag = 1;
        atomicCAS(status, 0, code);
        return false;
      }
    }
  }
}

// one 32-byte store (dst 32-byte aligned): a whole sector per thread
__device__ __forceinline__ void st_global_v8(uint32_t* dst, const uint32_t* w) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]),
               "r"(w[6]), "r"(w[7])
               : "memory");
}

// After a CTA has given up (abort flag set), the thread that issued bulk copies waits, again bounded (about 10 ms), until
// the copy armed on `bar` for the phase of parity `parity` has delivered its bytes: the CTA does not return with copies
// into its shared memory in flight.  A stage that was never armed answers at once (parity of the phase before the first).
constexpr long long kDrainLimitCycles = 20000000ll;
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try(bar, parity, 1000u)) {
    if (clock64() - t0 > kDrainLimitCycles) break;
    __nanosleep(200);
  }
}
// the same for a ring of `stages` barriers of which `stage` (in the lap of parity `phase`) would have been armed next
template <typename BarFn>
__device__ __forceinline__ void ring_drain(BarFn bar, int stages, int stage, uint32_t phase) {
  for (int k = 1; k <= stages; ++k) {   // the stages armed last, newest first
    int s = stage - k;
    uint32_t ph = phase;
    if (s < 0) {
      s += stages;
      ph ^= 1u;
    }
    mbar_drain(bar(s), ph);
  }
}

// n / d for 0 <= n < 2^31 with the multiplier and shift prepared on the host (see make_fastdiv)
__device__ __forceinline__ int fdiv(int n, FastDiv d) { return (int)((__umulhi(d.m, (uint32_t)n) + (uint32_t)n) >> d.l); }

// all 32 lanes wait (warp-uniform result)
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status, int code,
                                          uint32_t hint_ns) {
  const bool ok = mbar_wait(bar, parity, abort_flag, status, code, hint_ns);
  return __all_sync(0xffffffffu, ok);
}
// true in exactly one lane of a converged warp
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{ .reg .pred p; elect.sync _|p, 0xffffffff; selp.u32 %0, 1, 0, p; }" : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(bar)
               : "memory");
}

// ---- CTA pairs (thread-block clusters of two; the pair shares one tcgen05.mma with cta_group::2) ----------------
__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
// all threads of both CTAs; orders shared-memory writes (barrier initialisation) before the peer's remote arrivals
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrivals on a barrier that may live in the other CTA of the pair (`cbar` is a shared::cluster address)
__device__ __forceinline__ void mbar_expect_tx_remote(uint32_t cbar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cbar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cbar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cbar) : "memory");
}
// TMA tile loads of a CTA pair: the data lands in this CTA, the byte count is reported to a barrier of either CTA
// (no multicast: each CTA fetches its own operand rows)
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t cbar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(cbar)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t cbar) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(cbar)
               : "memory");
}

}  // namespace hq
