// Shared device/host helpers of libetr (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/etr.h"

namespace etr {

// ---- launch accounting and error mapping ------------------------------------------------
void note_launch(int n = 1);
// Optional per-kernel timing (etr_timing_enable): an event pair around every launch.
void timing_begin(const char* kernel_name, cudaStream_t st);
void timing_end(cudaStream_t st);
#define ETR_TIME_BEGIN(name) ::etr::timing_begin(name, st)
#define ETR_LAUNCH_CHECK()                                  \
  do {                                                      \
    ::etr::timing_end(st);                                  \
    ::etr::note_launch();                                   \
    cudaError_t e__ = cudaGetLastError();                   \
    if (e__ != cudaSuccess) return ETR_ERR_CUDA;            \
  } while (0)
#define ETR_TRY(expr)                                       \
  do {                                                      \
    etr_status s__ = (expr);                                \
    if (s__ != ETR_OK) return s__;                          \
  } while (0)

inline int c_stride_of(const etr_config* c) { return (c->capacity + 127) / 128 * 128; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t elem_bytes(int dtype) { return dtype == ETR_BF16 ? 2 : 4; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t grad_elem_bytes(const etr_config* c) { return c->grad_fp32 ? 4 : elem_bytes(c->dtype); }

// Opt-in to more than 48 KiB of dynamic shared memory: an attribute of the kernel on ONE device, so
// it is set once per device (a bit per device ordinal in `done`, one flag word per kernel).
template <class K>
inline bool ensure_dyn_smem(K kernel, size_t bytes, std::atomic<unsigned long long>& done) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  const unsigned long long bit = 1ull << (dev & 63);
  if (done.load(std::memory_order_acquire) & bit) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess)
    return false;
  done.fetch_or(bit, std::memory_order_release);
  return true;
}
// Multiprocessor count of the current device (cached per device ordinal).
inline int current_sm_count() {
  static std::atomic<int> cache[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  int n = cache[dev & 63].load(std::memory_order_relaxed);
  if (n <= 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cache[dev & 63].store(n, std::memory_order_relaxed);
  }
  return n;
}

// ---- order-preserving map float -> uint32 (larger float <=> larger key; key 0 is below
//      every finite float and is used as "not a candidate") --------------------------------
__host__ __device__ inline uint32_t ordered_key(float f) {
  uint32_t u;
#ifdef __CUDA_ARCH__
  u = __float_as_uint(f);
#else
  union { float f; uint32_t u; } c; c.f = f; u = c.u;
#endif
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__host__ __device__ inline float key_to_float(uint32_t k) {
  uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
#ifdef __CUDA_ARCH__
  return __uint_as_float(u);
#else
  union { float f; uint32_t u; } c; c.u = u; return c.f;
#endif
}

// ---- 8-element vectors of the activation dtype -----------------------------------------------
template <class T> struct Vec8;
template <> struct Vec8<float> {
  float v[8];
  __device__ static Vec8 load(const float* p) {
    Vec8 r;
    float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    r.v[0] = a.x; r.v[1] = a.y; r.v[2] = a.z; r.v[3] = a.w;
    r.v[4] = b.x; r.v[5] = b.y; r.v[6] = b.z; r.v[7] = b.w;
    return r;
  }
  __device__ static void store(float* p, const float* f) {
    *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
    *reinterpret_cast<float4*>(p + 4) = make_float4(f[4], f[5], f[6], f[7]);
  }
};
template <> struct Vec8<__nv_bfloat16> {
  float v[8];
  __device__ static Vec8 load(const __nv_bfloat16* p) {
    Vec8 r;
    uint4 q = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      r.v[2 * i] = __uint_as_float(w[i] << 16);
      r.v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    return r;
  }
  __device__ static void store(__nv_bfloat16* p, const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 b = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&b);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

template <class T> __device__ inline float to_f32(T v);
template <> __device__ inline float to_f32<float>(float v) { return v; }
template <> __device__ inline float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <class T> __device__ inline T from_f32(float v);
template <> __device__ inline float from_f32<float>(float v) { return v; }
template <> __device__ inline __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---- shared-memory barriers (mbarrier) and the bounded wait every pipeline of the library uses ----
// A wait never spins forever: after limit_cycles SM clock cycles it sets the CTA's abort flag and
// returns false; the kernel then stops issuing work, records a code in etr_stats.error_word and
// returns (the host reads it as ETR_ERR_TIMEOUT).
constexpr long long ETR_WAIT_LIMIT_CYCLES = 4000000000ll;   // about two seconds

#ifdef __CUDACC__
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
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
// Bounded wait: false if this or another thread of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          long long limit_cycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit_cycles) { *abort_flag = 1; return false; }
    }
  }
}
#endif

// ---- stage entry points, one translation unit each ------------------------------------------
etr_status affinity_forward(const etr_config* c, const void* X, const float* R, float* delta,
                            float* Z, float* xnorm, float* rnorm, etr_stats* stats, cudaStream_t st);
size_t affinity_bwd_workspace_bytes(const etr_config* c);
// score_tcgen05.cu: the score product on the tensor cores (E <= 64, 32 | d/D, 16-byte aligned Z, R, delta)
bool affinity_score_tc_takes(const etr_config* c, const float* Z, const float* R, const float* delta);
etr_status affinity_score_tc(const etr_config* c, const float* Z, const float* xnorm, const float* R, float* delta,
                             float* rnorm, etr_stats* stats, cudaStream_t st);
etr_status affinity_backward(const etr_config* c, const void* X, const float* R, const float* delta,
                             const float* Z, const float* xnorm, const float* rnorm,
                             const etr_route* rt, const float* dgate, const float* ddelta,
                             const void* dXp_fused, void* dX, float* dR, void* ws, etr_stats* stats,
                             cudaStream_t st);
// softmax-gate variant and load statistics (gate.cu)
etr_status gate_softmax_forward(const etr_config* c, const float* delta, const etr_route* rt, float* lse,
                                cudaStream_t st);
etr_status gate_softmax_backward(const etr_config* c, const float* delta, const float* lse,
                                 const etr_route* rt, const float* dgate, float* ddelta, cudaStream_t st);
etr_status load_stats_launch(const etr_config* c, const etr_route* rt, float* load, float* gate_mean,
                             cudaStream_t st);
size_t select_workspace_bytes(const etr_config* c);
int resolve_mode(const etr_config* c);
etr_status select_forward(const etr_config* c, const float* delta, etr_stats* stats,
                          const etr_route* rt, void* ws, cudaStream_t st);
etr_status dispatch_forward(const etr_config* c, const void* X, const etr_route* rt, void* Xp, cudaStream_t st);
etr_status combine_forward(const etr_config* c, const etr_route* rt, const void* O, void* Y, cudaStream_t st);
etr_status combine_backward(const etr_config* c, const etr_route* rt, const void* dY, const void* O,
                            void* dO, float* dgate, cudaStream_t st);
etr_status dispatch_backward(const etr_config* c, const etr_route* rt, const void* dXp, void* dX, cudaStream_t st);

// SIMT grouped GEMMs (fp32 or bf16 storage, fp32 accumulate).
etr_status simt_ffn_forward(const etr_config* cfg, const etr_route* route, const void* Xp,
                            const void* W1g, const void* W1u, const void* W2, void* G, void* U,
                            void* H, void* O, cudaStream_t st);
etr_status simt_ffn_backward(const etr_config* cfg, const etr_route* route, const void* dO,
                             const void* Xp, const void* G, const void* U, const void* H,
                             const void* W1g, const void* W1u, const void* W2, void* dG, void* dU,
                             void* dXp, void* dW1g, void* dW1u, void* dW2, cudaStream_t st);
// tcgen05 grouped GEMMs (bf16 only).  X_tokens != nullptr: the token rows are gathered from X
// through route->slot_token and Xp is not read (may be nullptr).
etr_status tc_ffn_forward(const etr_config* cfg, const etr_route* route, const void* Xp, const void* X_tokens,
                          const void* W1g, const void* W1u, const void* W2, void* G, void* U,
                          void* H, void* O, etr_stats* stats, void* ws, void* Y_top1, cudaStream_t st);
// Y_top1 != nullptr (Top-1 token choice only): the down GEMM's epilogue also writes gate * O of every
// row in use to the row of its token in Y; rows of tokens without a row are not touched.
etr_status zero_unrouted_rows(const etr_config* c, const etr_route* rt, void* Y, cudaStream_t st);
// n fp32 values rounded to bf16 (nearest even); n a multiple of 8, both pointers 16-byte aligned
etr_status cast_f32_to_bf16(const void* src, void* dst, size_t n, cudaStream_t st);
etr_status tc_ffn_backward(const etr_config* cfg, const etr_route* route, const void* dO,
                           const void* Xp, const void* X_tokens, const void* G, const void* U, const void* H,
                           const void* W1g, const void* W1u, const void* W2, void* dG, void* dU,
                           void* dXp, void* dW1g, void* dW1u, void* dW2, etr_stats* stats,
                           void* ws, cudaStream_t st);
size_t tc_workspace_bytes(const etr_config* cfg);
etr_status tc_wait_selftest(etr_stats* stats, long long limit_cycles, cudaStream_t st);
bool tc_available();

}  // namespace etr
