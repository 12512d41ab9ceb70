// Device-side building blocks of libsgdb (sm_100a): mbarrier and bulk-copy PTX
// wrappers, bounded waits, 16-byte vector access and the optimizer rules.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sgdb.h"

namespace sgdb {

// Epilogue selector of the row-streaming kernel: write the mean, or apply a rule.
enum : int { EP_MEAN = 0, EP_SGD = 1, EP_MOMENTUM = 2, EP_RMSPROP = 3, EP_ADAM = 4, EP_ADAGRAD = 5 };

// Hyper-parameters as the kernels use them; derived once on the host.
struct Hyper {
  float lr, mu, rho, one_minus_rho, b1, one_minus_b1, b2, one_minus_b2, eps;
  float bc1, bc2;  // Adam: 1 - beta1^step, 1 - beta2^step
};

// ---------------------------------------------------------------- shared memory / mbarrier

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// Makes freshly initialised barriers visible to the async (bulk copy) proxy.
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n"
      "  .reg .pred p;\n"
      "  mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "  selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}

// Non-blocking probe of a barrier phase (try_wait above may itself hold the thread for a while).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n"
      "  .reg .pred p;\n"
      "  mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "  selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}

// Every wait on a barrier is bounded by wall time.  In a correct run a phase completes
// within microseconds; the limit only exists so that a broken pipeline ends the kernel
// with an error status instead of hanging the device.  `abort_flag` (shared memory)
// lets one thread's time-out end every other thread's wait quickly.
constexpr unsigned long long kWaitLimitNs = 2000ull * 1000 * 1000;  // 2 s: the default patience

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// A limit of zero means no patience at all: the phase must be complete already, one probe decides.
__device__ __forceinline__ bool mbar_wait_for(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                              unsigned long long limit_ns) {
  if (limit_ns == 0ull) {
    if (mbar_test_wait(bar, parity)) return true;
    *abort_flag = 1;
    return false;
  }
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long deadline = global_timer_ns() + limit_ns;
  for (uint32_t spin = 0;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 15u) == 15u) {
      if (*abort_flag != 0) return false;
      if (global_timer_ns() > deadline) break;
    }
  }
  *abort_flag = 1;
  return false;
}


// ---------------------------------------------------------------- bulk copy global -> shared

__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
  return policy;
}

// 1-D bulk async copy of this GPU's own global memory into this block's shared
// memory (no multicast).  dst, src 16-byte aligned, bytes a multiple of 16.
// Completion is signalled as `bytes` transaction bytes on the mbarrier.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes,
                                              uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1], %2, [%3], %4;" ::"r"(dst),
      "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "r"(addr));
  return v;
}

// ---------------------------------------------------------------- element types

// Gradient storage types.  A bf16 value is the upper half of an fp32 value.
struct BF16 {
  uint16_t bits;
};

template <typename GT>
struct GradTraits;
template <>
struct GradTraits<float> {
  static constexpr int kVec = 4;  // elements per 16 bytes
  static __device__ __forceinline__ float widen(float x) { return x; }
  static __device__ __forceinline__ void unpack(const uint4& v, float (&out)[4]) {
    out[0] = __uint_as_float(v.x);
    out[1] = __uint_as_float(v.y);
    out[2] = __uint_as_float(v.z);
    out[3] = __uint_as_float(v.w);
  }
};
template <>
struct GradTraits<BF16> {
  static constexpr int kVec = 8;
  static __device__ __forceinline__ float widen(BF16 x) {
    return __uint_as_float(static_cast<uint32_t>(x.bits) << 16);
  }
  static __device__ __forceinline__ void unpack(const uint4& v, float (&out)[8]) {
    out[0] = __uint_as_float(v.x << 16);
    out[1] = __uint_as_float(v.x & 0xffff0000u);
    out[2] = __uint_as_float(v.y << 16);
    out[3] = __uint_as_float(v.y & 0xffff0000u);
    out[4] = __uint_as_float(v.z << 16);
    out[5] = __uint_as_float(v.z & 0xffff0000u);
    out[6] = __uint_as_float(v.w << 16);
    out[7] = __uint_as_float(v.w & 0xffff0000u);
  }
};

// ---------------------------------------------------------------- fp32 vectors in global memory

// Streaming (touch-once) loads and stores of V consecutive floats, V in {4, 8}.
// `vec` says the 16-byte path is legal (aligned, fully in range); otherwise elements
// with index < n are accessed one by one.
template <int V>
__device__ __forceinline__ void load_floats(const float* p, bool vec, int n, float (&out)[V]) {
  if (vec) {
#pragma unroll
    for (int q = 0; q < V / 4; ++q) {
      float4 v = __ldcs(reinterpret_cast<const float4*>(p) + q);
      out[4 * q + 0] = v.x;
      out[4 * q + 1] = v.y;
      out[4 * q + 2] = v.z;
      out[4 * q + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int e = 0; e < V; ++e) out[e] = (e < n) ? __ldcs(p + e) : 0.0f;
  }
}

template <int V>
__device__ __forceinline__ void store_floats(float* p, bool vec, int n, const float (&in)[V]) {
  if (vec) {
#pragma unroll
    for (int q = 0; q < V / 4; ++q)
      __stcs(reinterpret_cast<float4*>(p) + q,
             make_float4(in[4 * q + 0], in[4 * q + 1], in[4 * q + 2], in[4 * q + 3]));
  } else {
#pragma unroll
    for (int e = 0; e < V; ++e)
      if (e < n) __stcs(p + e, in[e]);
  }
}

// The same with an L2 eviction policy chosen by the caller (createpolicy): for data that
// is read again one launch later and should stay in L2 (evict-last), next to data of the
// same array that should not (evict-first).
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(policy));
  return policy;
}

__device__ __forceinline__ float4 ld_global_hint(const float4* p, uint64_t policy) {
  float4 v;
  asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "l"(p), "l"(policy)
               : "memory");
  return v;
}
__device__ __forceinline__ float ld_global_hint(const float* p, uint64_t policy) {
  float v;
  asm volatile("ld.global.L1::no_allocate.L2::cache_hint.f32 %0, [%1], %2;" : "=f"(v) : "l"(p), "l"(policy) : "memory");
  return v;
}
__device__ __forceinline__ void st_global_hint(float4* p, const float4& v, uint64_t policy) {
  asm volatile("st.global.L1::no_allocate.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(p), "f"(v.x),
               "f"(v.y), "f"(v.z), "f"(v.w), "l"(policy)
               : "memory");
}
__device__ __forceinline__ void st_global_hint(float* p, float v, uint64_t policy) {
  asm volatile("st.global.L1::no_allocate.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(p), "f"(v), "l"(policy) : "memory");
}

template <int V>
__device__ __forceinline__ void load_floats_hint(const float* p, bool vec, int n, float (&out)[V], uint64_t policy) {
  if (vec) {
#pragma unroll
    for (int q = 0; q < V / 4; ++q) {
      const float4 v = ld_global_hint(reinterpret_cast<const float4*>(p) + q, policy);
      out[4 * q + 0] = v.x;
      out[4 * q + 1] = v.y;
      out[4 * q + 2] = v.z;
      out[4 * q + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int e = 0; e < V; ++e) out[e] = (e < n) ? ld_global_hint(p + e, policy) : 0.0f;
  }
}

template <int V>
__device__ __forceinline__ void store_floats_hint(float* p, bool vec, int n, const float (&in)[V], uint64_t policy) {
  if (vec) {
#pragma unroll
    for (int q = 0; q < V / 4; ++q)
      st_global_hint(reinterpret_cast<float4*>(p) + q,
                     make_float4(in[4 * q + 0], in[4 * q + 1], in[4 * q + 2], in[4 * q + 3]), policy);
  } else {
#pragma unroll
    for (int e = 0; e < V; ++e)
      if (e < n) st_global_hint(p + e, in[e], policy);
  }
}

// ---------------------------------------------------------------- optimizer rules

// One element of the update.  Written with explicit round-to-nearest intrinsics so
// that no kernel contracts it differently from another: the fused, the separate and
// the arrival-by-arrival paths produce identical bits.
template <int EP>
__device__ __forceinline__ void apply_rule(const Hyper& h, float g, float& theta, float& s0,
                                           float& s1) {
  if (EP == EP_SGD) {
    theta = __fmaf_rn(-h.lr, g, theta);
  } else if (EP == EP_MOMENTUM) {
    s0 = __fmaf_rn(h.mu, s0, g);
    theta = __fmaf_rn(-h.lr, s0, theta);
  } else if (EP == EP_RMSPROP) {
    s0 = __fmaf_rn(h.rho, s0, __fmul_rn(h.one_minus_rho, __fmul_rn(g, g)));
    float root = __fsqrt_rn(__fadd_rn(s0, h.eps));
    s1 = __fmaf_rn(h.mu, s1, __fdiv_rn(__fmul_rn(h.lr, g), root));
    theta = __fsub_rn(theta, s1);
  } else if (EP == EP_ADAM) {
    s0 = __fmaf_rn(h.b1, s0, __fmul_rn(h.one_minus_b1, g));
    s1 = __fmaf_rn(h.b2, s1, __fmul_rn(h.one_minus_b2, __fmul_rn(g, g)));
    float m_hat = __fdiv_rn(s0, h.bc1);
    float v_hat = __fdiv_rn(s1, h.bc2);
    theta = __fsub_rn(theta, __fdiv_rn(__fmul_rn(h.lr, m_hat), __fadd_rn(__fsqrt_rn(v_hat), h.eps)));
  } else if (EP == EP_ADAGRAD) {
    s0 = __fmaf_rn(g, g, s0);
    theta = __fsub_rn(theta, __fdiv_rn(__fmul_rn(h.lr, g), __fadd_rn(__fsqrt_rn(s0), h.eps)));
  }
}

// Exponential moving average of the parameters: avg <- alpha * avg + (1 - alpha) * theta.
__device__ __forceinline__ float ema_rule(float alpha, float one_minus_alpha, float avg, float theta) {
  return __fmaf_rn(alpha, avg, __fmul_rn(one_minus_alpha, theta));
}

template <int EP>
struct RuleTraits {
  static constexpr bool kTheta = EP != EP_MEAN;
  static constexpr bool kState0 = EP == EP_MOMENTUM || EP == EP_RMSPROP || EP == EP_ADAM || EP == EP_ADAGRAD;
  static constexpr bool kState1 = EP == EP_RMSPROP || EP == EP_ADAM;
};

}  // namespace sgdb
