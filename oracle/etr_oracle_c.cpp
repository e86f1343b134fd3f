// extern "C" surface of the CPU oracle (test infrastructure; see etr_oracle.hpp).
// Each entry exists for float (_f32) and double (_f64).  All pointers are host memory
// owned by the caller.
#include "etr_oracle.hpp"
#ifdef _OPENMP
#include <omp.h>
#endif

using namespace etr_oracle;

#define ETR_ORACLE_API(S, SUF)                                                                       \
  extern "C" void etr_oracle_affinity_##SUF(int T, int d, int D, int E, const S* X, const S* R,      \
                                            S* delta, S* xnorm, S* rnorm, S* delta_max) {            \
    affinity<S>(T, d, D, E, X, R, delta, xnorm, rnorm, delta_max);                                   \
  }                                                                                                  \
  extern "C" void etr_oracle_select_##SUF(int T, int E, int k, int mode, int C, int C_stride,        \
                                          const S* delta, int32_t* topk_idx, int32_t* counts,        \
                                          int32_t* slot_token, S* gate, int32_t* tok_ptr,            \
                                          int32_t* tok_row, int32_t* dropped, int32_t* unrouted) {   \
    select<S>(T, E, k, mode, C, C_stride, delta, topk_idx, counts, slot_token, gate, tok_ptr,        \
              tok_row, dropped, unrouted);                                                           \
  }                                                                                                  \
  extern "C" void etr_oracle_select_thresholded_##SUF(                                               \
      int T, int E, int k, int mode, int C, int C_stride, int threshold_mode, double tau_expert,     \
      double tau_token, const S* delta, int32_t* topk_idx, int32_t* counts, int32_t* slot_token,     \
      S* gate, int32_t* tok_ptr, int32_t* tok_row, int32_t* dropped, int32_t* unrouted) {            \
    select_thresholded<S>(T, E, k, mode, C, C_stride, threshold_mode, tau_expert, tau_token, delta,  \
                          topk_idx, counts, slot_token, gate, tok_ptr, tok_row, dropped, unrouted);  \
  }                                                                                                  \
  extern "C" void etr_oracle_dispatch_##SUF(int E, int C_stride, int d, const S* X,                  \
                                            const int32_t* slot_token, S* Xp) {                      \
    dispatch<S>(E, C_stride, d, X, slot_token, Xp);                                                  \
  }                                                                                                  \
  extern "C" void etr_oracle_ffn_row_##SUF(int d, int h, const S* x, const S* W1g, const S* W1u,     \
                                           const S* W2, S* g, S* u, S* hh, S* o) {                   \
    ffn_row<S>(d, h, x, W1g, W1u, W2, g, u, hh, o);                                                  \
  }                                                                                                  \
  extern "C" void etr_oracle_expert_ffn_##SUF(int E, int C_stride, int d, int h,                     \
                                              const int32_t* counts, const S* Xp, const S* W1g,      \
                                              const S* W1u, const S* W2, S* G, S* U, S* H, S* O) {   \
    expert_ffn<S>(E, C_stride, d, h, counts, Xp, W1g, W1u, W2, G, U, H, O);                          \
  }                                                                                                  \
  extern "C" void etr_oracle_expert_ffn_down_##SUF(int E, int C_stride, int d, int h,                \
                                                   const int32_t* counts, const S* H, const S* W2,   \
                                                   S* O) {                                           \
    expert_ffn_down<S>(E, C_stride, d, h, counts, H, W2, O);                                         \
  }                                                                                                  \
  extern "C" void etr_oracle_combine_##SUF(int T, int d, const int32_t* tok_ptr,                     \
                                           const int32_t* tok_row, const S* gate, const S* O,        \
                                           S* Y) {                                                   \
    combine<S>(T, d, tok_ptr, tok_row, gate, O, Y);                                                  \
  }                                                                                                  \
  extern "C" void etr_oracle_combine_bwd_##SUF(int E, int C_stride, int d,                           \
                                               const int32_t* slot_token, const S* gate,             \
                                               const S* dY, const S* O, S* dO, S* dgate) {           \
    combine_bwd<S>(E, C_stride, d, slot_token, gate, dY, O, dO, dgate);                              \
  }                                                                                                  \
  extern "C" void etr_oracle_ffn_row_bwd_##SUF(int d, int h, const S* go, const S* g, const S* u,    \
                                               const S* W1g, const S* W1u, const S* W2, S* dg,       \
                                               S* du, S* dxp) {                                      \
    ffn_row_bwd<S>(d, h, go, g, u, W1g, W1u, W2, dg, du, dxp);                                       \
  }                                                                                                  \
  extern "C" void etr_oracle_ffn_weight_grads_##SUF(int n, int d, int h, const S* dOe, const S* He,  \
                                                    const S* dGe, const S* dUe, const S* Xpe,        \
                                                    S* dW1g, S* dW1u, S* dW2) {                      \
    ffn_weight_grads<S>(n, d, h, dOe, He, dGe, dUe, Xpe, dW1g, dW1u, dW2);                           \
  }                                                                                                  \
  extern "C" void etr_oracle_expert_ffn_bwd_##SUF(                                                   \
      int E, int C_stride, int d, int h, const int32_t* counts, const S* dO, const S* Xp,            \
      const S* G, const S* U, const S* H, const S* W1g, const S* W1u, const S* W2, S* dG, S* dU,     \
      S* dXp, S* dW1g, S* dW1u, S* dW2) {                                                            \
    expert_ffn_bwd<S>(E, C_stride, d, h, counts, dO, Xp, G, U, H, W1g, W1u, W2, dG, dU, dXp, dW1g,   \
                      dW1u, dW2);                                                                    \
  }                                                                                                  \
  extern "C" void etr_oracle_dispatch_bwd_##SUF(int T, int d, const int32_t* tok_ptr,                \
                                                const int32_t* tok_row, const S* dXp, S* dX) {       \
    dispatch_bwd<S>(T, d, tok_ptr, tok_row, dXp, dX);                                                \
  }                                                                                                  \
  extern "C" void etr_oracle_select_bwd_##SUF(int T, int E, int C_stride,                            \
                                              const int32_t* slot_token, const S* dgate,             \
                                              S* ddelta) {                                           \
    select_bwd<S>(T, E, C_stride, slot_token, dgate, ddelta);                                        \
  }                                                                                                  \
  extern "C" void etr_oracle_softmax_gate_##SUF(int T, int E, int C_stride, const S* delta,          \
                                                const int32_t* slot_token, S* gate) {                \
    softmax_gate<S>(T, E, C_stride, delta, slot_token, gate);                                        \
  }                                                                                                  \
  extern "C" void etr_oracle_softmax_gate_bwd_##SUF(int T, int E, int C_stride, const S* delta,      \
                                                    const int32_t* slot_token, const S* dgate,       \
                                                    S* ddelta) {                                     \
    softmax_gate_bwd<S>(T, E, C_stride, delta, slot_token, dgate, ddelta);                           \
  }                                                                                                  \
  extern "C" void etr_oracle_load_stats_##SUF(int T, int E, int C_stride, const int32_t* counts,     \
                                              const int32_t* slot_token, const S* gate, S* load,     \
                                              S* gate_mean) {                                        \
    load_stats<S>(T, E, C_stride, counts, slot_token, gate, load, gate_mean);                        \
  }                                                                                                  \
  extern "C" void etr_oracle_affinity_bwd_##SUF(int T, int d, int D, int E, const S* X, const S* R,  \
                                                const S* delta, const S* xnorm, const S* rnorm,      \
                                                const S* ddelta, S* dX, S* dR) {                     \
    affinity_bwd<S>(T, d, D, E, X, R, delta, xnorm, rnorm, ddelta, dX, dR);                          \
  }

ETR_ORACLE_API(float, f32)
ETR_ORACLE_API(double, f64)

extern "C" double etr_oracle_capacity_lower_bound(int d, int E, double delta_star) {
  return capacity_lower_bound(d, E, delta_star);
}
extern "C" int etr_oracle_capacity_bound(int d, int E, int capacity, int c_floor, int adaptive,
                                         double delta_star) {
  return capacity_bound(d, E, capacity, c_floor, adaptive, delta_star);
}
extern "C" int etr_oracle_mode_for_step(long long step, long long switch_step) {
  return mode_for_step(step, switch_step);
}
// Thread count for the loops over independent outputs (1 = the plain single-threaded
// oracle).  Returns the count in effect.
extern "C" int etr_oracle_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
  return omp_get_max_threads();
#else
  (void)n;
  return 1;
#endif
}
