// Shared-memory pipeline helpers of the persistent kernels: mbarrier and bulk-copy PTX wrappers, release/acquire
// words in global memory, and the bounded waits (every wait gives up after a clock limit, raises a global abort
// flag and the status word MLORA_ERR_TIMEOUT, after which every wait of the launch returns at once).
#pragma once
#include "../../include/mlora.h"
#include "common.cuh"

namespace mlora {

constexpr long long PIPE_WAIT_CYCLES = 4000000000ll;   // ~2 s at 2 GHz

// ----------------------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void cp_async16_ca(void* smem, const void* gmem) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// a ring is addressed by the running stage count since the start of the launch
__device__ __forceinline__ int pos_stage(int pos, int nstages) { return pos % nstages; }
__device__ __forceinline__ uint32_t pos_parity(int pos, int nstages) { return (uint32_t)((pos / nstages) & 1); }

// ----------------------------------------------------------------------------- bounded waits
struct WaitCtx {
  long long limit;                  // clock cycles a wait may take
  volatile int* s_abort;            // shared: this CTA has given up waiting
  unsigned long long* sync;         // global: [0] barrier, [1] shrink, [2] abort, [3] where the first wait gave up
  int* status;
};
// where codes: 1 producer/free stage, 2 shrink/A piece, 3 GEMM/weight chunk, 4 T counter, 5 grid barrier
static __device__ __noinline__ void raise_abort(const WaitCtx& w, int where, int phase) {
  *w.s_abort = 1;
  atomicCAS(w.status, 0, MLORA_ERR_TIMEOUT);
  atomicCAS(w.sync + 3, 0ull, ((unsigned long long)where << 48) | ((unsigned long long)(phase & 0xffff) << 32) |
                                  ((unsigned long long)(blockIdx.x & 0xffff) << 16) | (unsigned long long)(threadIdx.x & 0xffff));
  atomicExch(w.sync + 2, 1ull);
}
// mbarrier wait; false when the CTA is (or goes) in abort mode.  The slow path is a function of its own: the waits
// sit in many places of the persistent kernels, whose code must stay small enough for the instruction cache.
static __device__ __noinline__ bool wait_mbar_slow(uint32_t bar, uint32_t parity, const WaitCtx& w, int where, int phase) {
  if (*w.s_abort) return false;
  const long long t0 = clock64();
  for (int it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255) == 255) {
      if (*w.s_abort) return false;
      if (ld_acquire_u64(w.sync + 2) != 0ull) { *w.s_abort = 1; return false; }
      if (clock64() - t0 > w.limit) { raise_abort(w, where, phase); return false; }
    }
  }
}
__device__ __forceinline__ bool wait_mbar(uint32_t bar, uint32_t parity, const WaitCtx& w, int where, int phase) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_mbar_slow(bar, parity, w, where, phase);
}
// one thread spins until *ctr >= target
__device__ __forceinline__ void wait_counter(const unsigned long long* ctr, unsigned long long target, const WaitCtx& w,
                                             int where, int phase) {
  if (*w.s_abort) return;
  const long long t0 = clock64();
  for (int it = 0;; ++it) {
    if (ld_acquire_u64(ctr) >= target) return;
    if ((it & 63) == 63) {
      if (ld_acquire_u64(w.sync + 2) != 0ull) { *w.s_abort = 1; return; }
      if (clock64() - t0 > w.limit) { raise_abort(w, where, phase); return; }
    }
  }
}

}  // namespace mlora
