// Thin inline-PTX helpers for sm_100a: mbarriers with bounded waits, bulk
// tensor (TMA) copies, and the status word that a wait which ran out writes to.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace maxdnn {

// Codes a kernel may leave in the per-device status word (0 = nothing happened).
enum DeviceCode : uint32_t {
  kDevOk = 0,
  kDevTimeoutFull = 0x100,    // consumer waited for a staged tile that never arrived
  kDevTimeoutEmpty = 0x200,   // producer waited for a ring slot that was never released
  kDevTimeoutAccum = 0x300,   // epilogue waited for an accumulator that never completed
  kDevTimeoutAccFree = 0x400, // MMA issuer waited for an accumulator that was never drained
  kDevTimeoutDrain = 0x500,   // exit path: a copy in flight did not land in time
  kDevTimeoutPeer = 0x600,    // split tail: another CTA's partial sums never arrived
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
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

// Where a wait that ran out reports, and how the other waits of the SAME launch learn of
// it.  `status` points to the device's status block: word 0 keeps the first code any
// launch recorded until the host reads it (sticky); word 1 holds the `epoch` — a number the
// host gives every launch — of the latest launch in which a wait gave up.  A wait leaves
// early only when word 1 equals its own launch's epoch, so a code left behind by an
// earlier launch never cuts a healthy launch's waits short.
struct WaitCtx {
  uint32_t* status;
  uint32_t epoch;
};

// Wait budget of every spin in these kernels: 2 s of wall clock, checked every
// 256 failed polls.  A wait that runs out records `code` and returns false; the
// caller then leaves its loops and the kernel ends normally.
constexpr uint64_t kWaitBudgetNs = 2000000000ull;

__device__ __forceinline__ bool launch_gave_up(const WaitCtx& wc) {
  return wc.status && reinterpret_cast<volatile uint32_t*>(wc.status)[1] == wc.epoch;
}

__device__ __forceinline__ void record_give_up(const WaitCtx& wc, uint32_t code) {
  if (!wc.status) return;
  atomicCAS(wc.status, 0u, code);
  atomicExch(wc.status + 1, wc.epoch);
}

__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const WaitCtx& wc,
                                            uint32_t code) {
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (globaltimer_ns() - t0 > kWaitBudgetNs) break;
    if (launch_gave_up(wc)) break;   // another wait of this launch ran out
  }
  record_give_up(wc, code);
  return false;
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& wc,
                                          uint32_t code) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, wc, code);
}

// Exit-path wait after another wait ran out: copies already issued land within
// microseconds; give their barrier one millisecond, then move on without a code.
__device__ __noinline__ void mbar_wait_grace(uint32_t bar, uint32_t parity) {
  const uint64_t t0 = globaltimer_ns();
  while (!mbar_try_wait(bar, parity))
    if (globaltimer_ns() - t0 > 1000000ull) break;
}

#ifndef MAXDNN_PRODUCER_SLEEP_NS
#define MAXDNN_PRODUCER_SLEEP_NS 250
#endif

// Producer-side wait: sleeps between polls, so that a warp waiting for a ring slot
// does not take issue slots from the arithmetic warps of its scheduler.  Same 2 s
// budget as mbar_wait.
__device__ __noinline__ bool mbar_wait_sleep_slow(uint32_t bar, uint32_t parity, const WaitCtx& wc,
                                                  uint32_t code) {
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
#if MAXDNN_PRODUCER_SLEEP_NS > 0
      __nanosleep(MAXDNN_PRODUCER_SLEEP_NS);
#endif
      if (mbar_try_wait(bar, parity)) return true;
    }
    if (globaltimer_ns() - t0 > kWaitBudgetNs) break;
    if (launch_gave_up(wc)) break;
  }
  record_give_up(wc, code);
  return false;
}

__device__ __forceinline__ bool mbar_wait_backoff(uint32_t bar, uint32_t parity, const WaitCtx& wc,
                                                  uint32_t code) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_sleep_slow(bar, parity, wc, code);
}

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}

// Tiled bulk tensor loads global -> shared, completion counted on an mbarrier.
// c0 is the innermost coordinate (its byte offset must be a multiple of 16).
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* m, uint32_t bar,
                                            int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* m, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* m, uint32_t bar,
                                            int c0, int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

// One 8-byte shared-memory load.  Written as an instruction of its own so that two
// neighbouring ones are not fused into a 16-byte load: next to a stream of packed
// multiply-adds a 16-byte load costs about 1.3 issue cycles, an 8-byte load about 0.1
// (measured: the microbenchmark in ubench_fp32.cu).
__device__ __forceinline__ float2 lds64(const void* p) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(smem_u32(p)));
  return v;
}

__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

}  // namespace maxdnn
