// Device-side plumbing shared by the decode kernels: mbarrier and bulk-copy wrappers (every wait bounded),
// dependent-launch controls, and the running softmax state of a lane.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ssd {

constexpr float kNegBig = -1.0e30f;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // one second per wait, then give up

// ------------------------------------------------------------------ asynchronous-copy plumbing
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
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
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
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
// Wait for a phase of the barrier, for at most kWaitLimitNs.  Uniform over the warp.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  bool ok = mbar_try_wait(bar, parity);
  if (!ok) {
    const unsigned long long t0 = global_ns();
    do {
#pragma unroll 1
      for (int i = 0; i < 64 && !ok; ++i) ok = mbar_try_wait(bar, parity);
    } while (!ok && global_ns() - t0 < kWaitLimitNs);
  }
  return __all_sync(0xffffffffu, ok);
}
// Global -> shared bulk copy; bytes is a multiple of 16 and both addresses are 16-byte aligned.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute
// may start while its predecessor in the stream is still running, once the predecessor has allowed
// it; it must then wait for the predecessor to complete before touching memory the predecessor may
// write, or that anything earlier may have written and not yet flushed.  Both kernels of the decode
// step wait just before their first such access and allow their successor right after that wait.
// So launch latency, CTA start-up and the index planning overlap with the predecessor's tail; every
// kernel of the chain waits for its predecessor's completion, which preserves stream order
// transitively; and when a kernel starts, everything before its predecessor has completed (the
// predecessor passed its own wait before allowing it), which is what makes the slab prefetch of the
// decode kernel's prologue safe.
__device__ __forceinline__ void pdl_allow_successor() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------ arithmetic
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// the two bf16 values of a 32-bit word, widened exactly
__device__ __forceinline__ float2 widen2(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

// A lane's share of a row: 16 of the 128 dimensions, as 8 pairs.  Lane l8 of a group holds
// dimensions [8*l8, 8*l8 + 8) in pairs 0..3 and [64 + 8*l8, 64 + 8*l8 + 8) in pairs 4..7.
struct State {
  float m, l;
  float2 acc[8];
};

__device__ __forceinline__ void state_init(State& s) {
  s.m = kNegBig;
  s.l = 0.f;
#pragma unroll
  for (int d = 0; d < 8; ++d) s.acc[d] = make_float2(0.f, 0.f);
}

// s <- s (+) the state held by lane (lane ^ mask)
__device__ __forceinline__ void state_merge_lane(State& s, int mask) {
  const float m2 = __shfl_xor_sync(0xffffffffu, s.m, mask);
  const float l2 = __shfl_xor_sync(0xffffffffu, s.l, mask);
  const float mn = fmaxf(s.m, m2);
  const float c1 = ex2(s.m - mn), c2 = ex2(m2 - mn);
  s.l = s.l * c1 + l2 * c2;
#pragma unroll
  for (int d = 0; d < 8; ++d) {
    const float ax = __shfl_xor_sync(0xffffffffu, s.acc[d].x, mask);
    const float ay = __shfl_xor_sync(0xffffffffu, s.acc[d].y, mask);
    s.acc[d].x = s.acc[d].x * c1 + ax * c2;
    s.acc[d].y = s.acc[d].y * c1 + ay * c2;
  }
  s.m = mn;
}

}  // namespace ssd
