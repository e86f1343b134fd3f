// CPU oracle for the Expert-Token Resonance (ETR) MoE layer, arXiv 2406.00023.
//
// TEST INFRASTRUCTURE ONLY.  This is a plain, slow, obviously-correct restatement of
// what the paper defines, used to check the CUDA library and as a timed CPU baseline.
// It shares no code with the CUDA path and the product never calls it.
//
// Every function follows the paper's steps in the paper's order:
//   affinity   : GrAP pooling (the W_aff equations of "Cost-Efficient Sparse
//                Expert-Token Affinity") followed by the cosine affinity score
//   capacity   : the capacity lower bound C_min of the Remark in "Dynamic Lower Bound
//                Module for Expert Capacity in ETR"
//   select     : the two "Routing Strategy" equations: Top-l experts per token, then
//                each expert keeps C of the tokens assigned to it
//   dispatch / ffn / combine : the general MoE form, MoE(x) = sum_t sum_i G_i(x_t) E_i(x_t)
//   *_bwd      : plain calculus on the forward definitions (the paper gives no backward)
//
// Scalar type S is float (parity, timing) or double (finite-difference checks).  Every
// reduction is accumulated in double and rounded to S once.  OpenMP, when enabled, only
// distributes independent output elements over threads; no element's arithmetic order
// changes, so results do not depend on the thread count.
//
// Pins (tests/test_oracle_*.py): closed form of the paper's own W_aff (R = I), D = 1
// textbook cosine, orthogonality, Bessel bound, scale invariance, hand-evaluated C_min
// values, brute-force subset selection on tiny inputs, routing invariants, library
// SwiGLU for E = 1, central finite differences for every gradient, permutation
// equivariance.  Parity unpinned: the TCR->ECR switch rule (a caller-supplied step
// threshold), the source of delta_max (batch maximum), the clamp of C_min into
// [c_floor, capacity], and the raw-affinity gate; the paper under-specifies these.  The
// softmax-gate variant and the load statistics are pinned by library softmax / autograd, finite
// differences and closed forms.  The threshold on the sum of affinity scores (select_thresholded)
// is a reading of a rule the paper names without stating: parity unpinned as a reading, the
// function pinned by brute force over prefixes, its two limits and monotonicity.
#pragma once
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <limits>
#include <numeric>
#include <vector>

namespace etr_oracle {

enum Mode { MODE_TCR = 1, MODE_ECR = 2 };

// ---- GrAP + cosine affinity ---------------------------------------------------------
// z_t[j]  = (1/D) sum_{r<D} x_t[jD + r]                       (average pooling by groups)
// s_ti    = sum_j z_t[j] R_i[j]
// w_i     = the d-vector that holds R_i[j]/D on group j, so x_t . w_i = s_ti and
//           ||w_i|| = ||R_i|| / sqrt(D)
// delta_ti = cos(x_t, w_i) = sqrt(D) s_ti / (||x_t|| ||R_i||);  0 when a norm is 0.
template <class S>
void affinity(int T, int d, int D, int E, const S* X, const S* R,
              S* delta, S* xnorm, S* rnorm, S* delta_max) {
  const int m = d / D;
  for (int i = 0; i < E; ++i) {
    double acc = 0.0;
    for (int j = 0; j < m; ++j) acc += (double)R[(size_t)i * m + j] * (double)R[(size_t)i * m + j];
    rnorm[i] = (S)std::sqrt(acc);
  }
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    const S* x = X + (size_t)t * d;
    std::vector<S> z(m);
    double sq = 0.0;
    for (int j = 0; j < m; ++j) {
      double acc = 0.0;
      for (int r = 0; r < D; ++r) acc += (double)x[j * D + r];
      z[j] = (S)(acc / (double)D);
    }
    for (int c = 0; c < d; ++c) sq += (double)x[c] * (double)x[c];
    xnorm[t] = (S)std::sqrt(sq);
    for (int i = 0; i < E; ++i) {
      double s = 0.0;
      for (int j = 0; j < m; ++j) s += (double)z[j] * (double)R[(size_t)i * m + j];
      const double den = (double)xnorm[t] * (double)rnorm[i];
      delta[(size_t)t * E + i] = den == 0.0 ? (S)0 : (S)(std::sqrt((double)D) * s / den);
    }
  }
  if (delta_max) {
    S mx = -std::numeric_limits<S>::infinity();
    for (size_t q = 0; q < (size_t)T * E; ++q) mx = std::max(mx, delta[q]);
    *delta_max = mx;
  }
}

// ---- capacity: C_min = (1/n) exp{ d delta_max^2 / (2 - delta_max^2) } -----------------
inline double capacity_lower_bound(int d, int E, double delta_star) {
  delta_star = std::min(1.0, std::max(0.0, delta_star));
  const double y = (double)d * delta_star * delta_star / (2.0 - delta_star * delta_star);
  return std::exp(y) / (double)E;
}

// C = capacity when not adaptive, else ceil(C_min) clamped into [c_floor, capacity].
inline int capacity_bound(int d, int E, int capacity, int c_floor, int adaptive, double delta_star) {
  if (!adaptive) return capacity;
  const double cmin = std::ceil(capacity_lower_bound(d, E, delta_star));
  const double c = std::min((double)capacity, std::max((double)c_floor, cmin));
  return (int)c;
}

// mode from the training step: token choice before the switch, expert choice after.
inline int mode_for_step(int64_t step, int64_t switch_step) {
  return step < switch_step ? MODE_TCR : MODE_ECR;
}

// ---- bidirectional selection ----------------------------------------------------------
// Token side: each token's k highest-affinity experts (ties: lower expert index).  In
// expert-choice mode every token is a candidate of every expert (l = n).
// Expert side: expert i keeps the min(C, |L_i|) candidates with the highest delta_ti
// (ties: lower token index); the remaining slots are the equation's "None".
// Maps: kept tokens of expert i sit in ascending token order at rows i*C_stride + p;
// tok_ptr/tok_row is the token-major inverse (rows of a token in ascending expert order).
template <class S>
void select(int T, int E, int k, int mode, int C, int C_stride, const S* delta,
            int32_t* topk_idx, int32_t* counts, int32_t* slot_token, S* gate,
            int32_t* tok_ptr, int32_t* tok_row, int32_t* dropped, int32_t* unrouted) {
  std::vector<std::vector<int32_t>> L(E);
  long n_cand = 0;
  for (int t = 0; t < T; ++t) {
    if (mode == MODE_TCR) {
      std::vector<int32_t> order(E);
      std::iota(order.begin(), order.end(), 0);
      const S* row = delta + (size_t)t * E;
      std::stable_sort(order.begin(), order.end(),
                       [row](int32_t a, int32_t b) { return row[a] > row[b]; });
      for (int j = 0; j < k; ++j) {
        topk_idx[(size_t)t * k + j] = order[j];
        L[order[j]].push_back(t);
      }
      n_cand += k;
    } else {
      for (int j = 0; j < k; ++j) topk_idx[(size_t)t * k + j] = -1;
      for (int i = 0; i < E; ++i) L[i].push_back(t);
      n_cand += E;
    }
  }
  for (size_t r = 0; r < (size_t)E * C_stride; ++r) { slot_token[r] = -1; gate[r] = (S)0; }
  std::vector<std::vector<int32_t>> rows_of(T);
  long kept = 0;
  for (int i = 0; i < E; ++i) {
    std::vector<int32_t>& cand = L[i];              // ascending token id by construction
    std::stable_sort(cand.begin(), cand.end(), [delta, E, i](int32_t a, int32_t b) {
      return delta[(size_t)a * E + i] > delta[(size_t)b * E + i];
    });
    const int n = std::min<int>(C, (int)cand.size());
    std::vector<int32_t> keep(cand.begin(), cand.begin() + n);
    std::sort(keep.begin(), keep.end());
    counts[i] = n;
    kept += n;
    for (int p = 0; p < n; ++p) {
      const size_t r = (size_t)i * C_stride + p;
      slot_token[r] = keep[p];
      gate[r] = delta[(size_t)keep[p] * E + i];
      rows_of[keep[p]].push_back((int32_t)r);
    }
  }
  int32_t un = 0, pos = 0;
  for (int t = 0; t < T; ++t) {
    tok_ptr[t] = pos;
    for (int32_t r : rows_of[t]) tok_row[pos++] = r;
    if (rows_of[t].empty()) ++un;
  }
  tok_ptr[T] = pos;
  if (dropped) *dropped = (int32_t)(n_cand - kept);
  if (unrouted) *unrouted = un;
}

// ---- selection with a threshold on the sum of affinity scores ------------------------------
// In "Routing Strategy" (the sentence that introduces the expert-side equation) the number l of
// tokens an expert takes depends on how large the accumulated affinity of its tokens has become,
// and "Training Strategy" says this number adapts during training; neither passage gives the rule.
// The reading implemented here
// (parity unpinned as a reading; the function itself is pinned by brute force over prefixes, by
// its limits tau = +infinity and tau <= first score, and by monotonicity in tau):
//
//   walk a candidate list in descending affinity (ties: lower index first); the candidate of
//   rank j (1-based) is kept while j is within the cap (C for an expert's tokens, k for a
//   token's experts) and the sum of the j-1 affinities before it is still below tau.
//
// threshold_mode bit 0 (expert side): applied to every expert's candidate tokens, in both modes.
// threshold_mode bit 1 (token side): applied to every token's Top-k experts in token choice, so a
// token takes between 0 and k experts; topk_idx holds -1 in the unused places.
// The sums are taken on affinities quantised to multiples of 2^-32, q(delta) = round-to-nearest
// (delta * 2^32), as 64-bit integers, and tau is quantised the same way, so that the decision does
// not depend on the order of summation; both sides of a parity test take it in this arithmetic.
inline int64_t quantise_affinity(double v) {
  const double s = v * 4294967296.0;
  if (!(s < 9.2e18)) return std::numeric_limits<int64_t>::max();       // +infinity (or NaN): never reached
  if (s < -9.2e18) return std::numeric_limits<int64_t>::min();
  return (int64_t)std::llrint(s);
}

template <class S>
void select_thresholded(int T, int E, int k, int mode, int C, int C_stride, int threshold_mode,
                        double tau_expert, double tau_token, const S* delta, int32_t* topk_idx,
                        int32_t* counts, int32_t* slot_token, S* gate, int32_t* tok_ptr,
                        int32_t* tok_row, int32_t* dropped, int32_t* unrouted) {
  const bool cut_expert = (threshold_mode & 1) != 0, cut_token = (threshold_mode & 2) != 0;
  const int64_t tq_expert = quantise_affinity(tau_expert), tq_token = quantise_affinity(tau_token);
  std::vector<std::vector<int32_t>> L(E);
  long n_cand = 0;
  for (int t = 0; t < T; ++t) {
    if (mode == MODE_TCR) {
      std::vector<int32_t> order(E);
      std::iota(order.begin(), order.end(), 0);
      const S* row = delta + (size_t)t * E;
      std::stable_sort(order.begin(), order.end(),
                       [row](int32_t a, int32_t b) { return row[a] > row[b]; });
      int64_t sum_before = 0;
      bool open = true;                               // the walk stops at the first rank it does not keep
      for (int j = 0; j < k; ++j) {
        open = open && (!cut_token || sum_before < tq_token);
        topk_idx[(size_t)t * k + j] = open ? order[j] : -1;
        if (open) { L[order[j]].push_back(t); ++n_cand; }
        sum_before += quantise_affinity((double)row[order[j]]);
      }
    } else {
      for (int j = 0; j < k; ++j) topk_idx[(size_t)t * k + j] = -1;
      for (int i = 0; i < E; ++i) L[i].push_back(t);
      n_cand += E;
    }
  }
  for (size_t r = 0; r < (size_t)E * C_stride; ++r) { slot_token[r] = -1; gate[r] = (S)0; }
  std::vector<std::vector<int32_t>> rows_of(T);
  long kept = 0;
  for (int i = 0; i < E; ++i) {
    std::vector<int32_t>& cand = L[i];              // ascending token id by construction
    std::stable_sort(cand.begin(), cand.end(), [delta, E, i](int32_t a, int32_t b) {
      return delta[(size_t)a * E + i] > delta[(size_t)b * E + i];
    });
    int n = 0;
    int64_t sum_before = 0;
    while (n < (int)cand.size() && n < C && (!cut_expert || sum_before < tq_expert)) {
      sum_before += quantise_affinity((double)delta[(size_t)cand[n] * E + i]);
      ++n;
    }
    std::vector<int32_t> keep(cand.begin(), cand.begin() + n);
    std::sort(keep.begin(), keep.end());
    counts[i] = n;
    kept += n;
    for (int p = 0; p < n; ++p) {
      const size_t r = (size_t)i * C_stride + p;
      slot_token[r] = keep[p];
      gate[r] = delta[(size_t)keep[p] * E + i];
      rows_of[keep[p]].push_back((int32_t)r);
    }
  }
  int32_t un = 0, pos = 0;
  for (int t = 0; t < T; ++t) {
    tok_ptr[t] = pos;
    for (int32_t r : rows_of[t]) tok_row[pos++] = r;
    if (rows_of[t].empty()) ++un;
  }
  tok_ptr[T] = pos;
  if (dropped) *dropped = (int32_t)(n_cand - kept);
  if (unrouted) *unrouted = un;
}

// ---- dispatch: Xp[r,:] = X[slot_token[r],:]; unused rows are zero -----------------------
template <class S>
void dispatch(int E, int C_stride, int d, const S* X, const int32_t* slot_token, S* Xp) {
#pragma omp parallel for schedule(static)
  for (long r = 0; r < (long)E * C_stride; ++r) {
    const int32_t t = slot_token[r];
    for (int c = 0; c < d; ++c) Xp[(size_t)r * d + c] = t < 0 ? (S)0 : X[(size_t)t * d + c];
  }
}

template <class S> inline double sigmoid(S v) { return 1.0 / (1.0 + std::exp(-(double)v)); }

// ---- one row of one expert's SwiGLU FFN --------------------------------------------------
// g = W1g x, u = W1u x, hh = silu(g) * u with silu(v) = v / (1 + e^-v), o = W2 hh.
template <class S>
void ffn_row(int d, int h, const S* x, const S* W1g, const S* W1u, const S* W2,
             S* g, S* u, S* hh, S* o) {
  for (int b = 0; b < h; ++b) {
    double ag = 0.0, au = 0.0;
    const S* wg = W1g + (size_t)b * d;
    const S* wu = W1u + (size_t)b * d;
    for (int c = 0; c < d; ++c) { ag += (double)wg[c] * (double)x[c]; au += (double)wu[c] * (double)x[c]; }
    g[b] = (S)ag;
    u[b] = (S)au;
    hh[b] = (S)((double)g[b] * sigmoid(g[b]) * (double)u[b]);
  }
  for (int a = 0; a < d; ++a) {
    double acc = 0.0;
    const S* w = W2 + (size_t)a * h;
    for (int b = 0; b < h; ++b) acc += (double)w[b] * (double)hh[b];
    o[a] = (S)acc;
  }
}

// Second half of ffn_row on its own: o = W2 hh for a given hidden activation (used to model a
// pipeline that stores hh in a narrower type between the two halves).
template <class S>
void ffn_down_row(int d, int h, const S* hh, const S* W2, S* o) {
  for (int a = 0; a < d; ++a) {
    double acc = 0.0;
    const S* w = W2 + (size_t)a * h;
    for (int b = 0; b < h; ++b) acc += (double)w[b] * (double)hh[b];
    o[a] = (S)acc;
  }
}

template <class S>
void expert_ffn_down(int E, int C_stride, int d, int h, const int32_t* counts, const S* H, const S* W2, S* O) {
#pragma omp parallel for schedule(dynamic, 8)
  for (long r = 0; r < (long)E * C_stride; ++r) {
    const int i = (int)(r / C_stride), p = (int)(r % C_stride);
    S* o = O + (size_t)r * d;
    if (p < counts[i]) ffn_down_row(d, h, H + (size_t)r * h, W2 + (size_t)i * d * h, o);
    else std::fill(o, o + d, (S)0);
  }
}

// All experts: rows p < counts[i] of expert i; other rows of G,U,H,O are set to zero.
template <class S>
void expert_ffn(int E, int C_stride, int d, int h, const int32_t* counts, const S* Xp,
                const S* W1g, const S* W1u, const S* W2, S* G, S* U, S* H, S* O) {
#pragma omp parallel for schedule(dynamic, 8)
  for (long r = 0; r < (long)E * C_stride; ++r) {
    const int i = (int)(r / C_stride), p = (int)(r % C_stride);
    S* g = G + (size_t)r * h; S* u = U + (size_t)r * h; S* hh = H + (size_t)r * h; S* o = O + (size_t)r * d;
    if (p < counts[i]) {
      ffn_row(d, h, Xp + (size_t)r * d, W1g + (size_t)i * h * d, W1u + (size_t)i * h * d,
              W2 + (size_t)i * d * h, g, u, hh, o);
    } else {
      std::fill(g, g + h, (S)0); std::fill(u, u + h, (S)0); std::fill(hh, hh + h, (S)0);
      std::fill(o, o + d, (S)0);
    }
  }
}

// ---- combine: Y[t,:] = sum_{r in rows(t)} gate[r] O[r,:] ----------------------------------
template <class S>
void combine(int T, int d, const int32_t* tok_ptr, const int32_t* tok_row, const S* gate,
             const S* O, S* Y) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int c = 0; c < d; ++c) {
      double acc = 0.0;
      for (int q = tok_ptr[t]; q < tok_ptr[t + 1]; ++q)
        acc += (double)gate[tok_row[q]] * (double)O[(size_t)tok_row[q] * d + c];
      Y[(size_t)t * d + c] = (S)acc;
    }
  }
}

// ---- backward of combine: dO[r,:] = gate[r] dY[t(r),:], dgate[r] = <dY[t(r),:], O[r,:]> ----
template <class S>
void combine_bwd(int E, int C_stride, int d, const int32_t* slot_token, const S* gate,
                 const S* dY, const S* O, S* dO, S* dgate) {
#pragma omp parallel for schedule(static)
  for (long r = 0; r < (long)E * C_stride; ++r) {
    const int32_t t = slot_token[r];
    double acc = 0.0;
    for (int c = 0; c < d; ++c) {
      if (t < 0) { dO[(size_t)r * d + c] = (S)0; continue; }
      dO[(size_t)r * d + c] = (S)((double)gate[r] * (double)dY[(size_t)t * d + c]);
      acc += (double)dY[(size_t)t * d + c] * (double)O[(size_t)r * d + c];
    }
    dgate[r] = (S)acc;
  }
}

// ---- backward of one FFN row (per-row part) ----------------------------------------------
// dhh = W2^T do;  sg = sigmoid(g);  dg = dhh*u*sg*(1 + g*(1-sg));  du = dhh*g*sg;
// dxp = W1g^T dg + W1u^T du.
template <class S>
void ffn_row_bwd(int d, int h, const S* go, const S* g, const S* u,
                 const S* W1g, const S* W1u, const S* W2, S* dg, S* du, S* dxp) {
  for (int b = 0; b < h; ++b) {
    double acc = 0.0;
    for (int a = 0; a < d; ++a) acc += (double)W2[(size_t)a * h + b] * (double)go[a];
    const double dhh = (double)(S)acc;
    const double sg = sigmoid(g[b]);
    dg[b] = (S)(dhh * (double)u[b] * sg * (1.0 + (double)g[b] * (1.0 - sg)));
    du[b] = (S)(dhh * (double)g[b] * sg);
  }
  for (int c = 0; c < d; ++c) {
    double acc = 0.0;
    for (int b = 0; b < h; ++b)
      acc += (double)W1g[(size_t)b * d + c] * (double)dg[b] + (double)W1u[(size_t)b * d + c] * (double)du[b];
    dxp[c] = (S)acc;
  }
}

// Weight gradients of one expert from its per-row quantities (n rows, contiguous):
// dW2[a,b] = sum_r do_r[a] hh_r[b];  dW1g[b,c] = sum_r dg_r[b] xp_r[c];  dW1u likewise.
template <class S>
void ffn_weight_grads(int n, int d, int h, const S* dOe, const S* He, const S* dGe, const S* dUe,
                      const S* Xpe, S* dW1g, S* dW1u, S* dW2) {
#pragma omp parallel for schedule(static)
  for (int a = 0; a < d; ++a) {
    std::vector<double> acc(h, 0.0);
    for (int r = 0; r < n; ++r) {
      const double v = (double)dOe[(size_t)r * d + a];
      const S* hr = He + (size_t)r * h;
      for (int b = 0; b < h; ++b) acc[b] += v * (double)hr[b];
    }
    for (int b = 0; b < h; ++b) dW2[(size_t)a * h + b] = (S)acc[b];
  }
#pragma omp parallel for schedule(static)
  for (int b = 0; b < h; ++b) {
    std::vector<double> ag(d, 0.0), au(d, 0.0);
    for (int r = 0; r < n; ++r) {
      const double vg = (double)dGe[(size_t)r * h + b], vu = (double)dUe[(size_t)r * h + b];
      const S* xr = Xpe + (size_t)r * d;
      for (int c = 0; c < d; ++c) { ag[c] += vg * (double)xr[c]; au[c] += vu * (double)xr[c]; }
    }
    for (int c = 0; c < d; ++c) { dW1g[(size_t)b * d + c] = (S)ag[c]; dW1u[(size_t)b * d + c] = (S)au[c]; }
  }
}

// All experts.  dG, dU (scratch, [E*C_stride, h]) and dXp are outputs too.
template <class S>
void expert_ffn_bwd(int E, int C_stride, int d, int h, const int32_t* counts, const S* dO,
                    const S* Xp, const S* G, const S* U, const S* H,
                    const S* W1g, const S* W1u, const S* W2,
                    S* dG, S* dU, S* dXp, S* dW1g, S* dW1u, S* dW2) {
#pragma omp parallel for schedule(dynamic, 8)
  for (long r = 0; r < (long)E * C_stride; ++r) {
    const int i = (int)(r / C_stride), p = (int)(r % C_stride);
    S* dg = dG + (size_t)r * h; S* du = dU + (size_t)r * h; S* dx = dXp + (size_t)r * d;
    if (p < counts[i]) {
      ffn_row_bwd(d, h, dO + (size_t)r * d, G + (size_t)r * h, U + (size_t)r * h,
                  W1g + (size_t)i * h * d, W1u + (size_t)i * h * d, W2 + (size_t)i * d * h, dg, du, dx);
    } else {
      std::fill(dg, dg + h, (S)0); std::fill(du, du + h, (S)0); std::fill(dx, dx + d, (S)0);
    }
  }
  for (int i = 0; i < E; ++i) {
    const size_t r0 = (size_t)i * C_stride;
    ffn_weight_grads(counts[i], d, h, dO + r0 * d, H + r0 * h, dG + r0 * h, dU + r0 * h, Xp + r0 * d,
                     dW1g + (size_t)i * h * d, dW1u + (size_t)i * h * d, dW2 + (size_t)i * d * h);
  }
}

// ---- backward of dispatch: dX[t,:] = sum_{r in rows(t)} dXp[r,:] ----------------------------
template <class S>
void dispatch_bwd(int T, int d, const int32_t* tok_ptr, const int32_t* tok_row, const S* dXp, S* dX) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int c = 0; c < d; ++c) {
      double acc = 0.0;
      for (int q = tok_ptr[t]; q < tok_ptr[t + 1]; ++q) acc += (double)dXp[(size_t)tok_row[q] * d + c];
      dX[(size_t)t * d + c] = (S)acc;
    }
  }
}

// ---- backward of the selection: d delta_ti = dgate[r] on selected pairs, 0 elsewhere ---------
template <class S>
void select_bwd(int T, int E, int C_stride, const int32_t* slot_token, const S* dgate, S* ddelta) {
  std::fill(ddelta, ddelta + (size_t)T * E, (S)0);
  for (int i = 0; i < E; ++i)
    for (int p = 0; p < C_stride; ++p) {
      const size_t r = (size_t)i * C_stride + p;
      if (slot_token[r] >= 0) ddelta[(size_t)slot_token[r] * E + i] = dgate[r];
    }
}

// ---- softmax gate (variant) ---------------------------------------------------------------------
// The general MoE form names G(x) = Softmax(.) as its example of a gating weight.  In this variant
// the gate of a selected pair (t, i) is the softmax of token t's affinities over ALL n experts,
//   p_ti = exp(delta_ti) / sum_j exp(delta_tj),
// instead of the raw affinity delta_ti.  Rows without a token keep gate 0.
template <class S>
void softmax_gate(int T, int E, int C_stride, const S* delta, const int32_t* slot_token, S* gate) {
  (void)T;
  for (int i = 0; i < E; ++i)
    for (int p = 0; p < C_stride; ++p) {
      const size_t r = (size_t)i * C_stride + p;
      const int t = slot_token[r];
      if (t < 0) { gate[r] = (S)0; continue; }
      const S* dt = delta + (size_t)t * E;
      double mx = (double)dt[0];
      for (int j = 1; j < E; ++j) mx = std::max(mx, (double)dt[j]);
      double den = 0.0;
      for (int j = 0; j < E; ++j) den += std::exp((double)dt[j] - mx);
      gate[r] = (S)(std::exp((double)dt[i] - mx) / den);
    }
}

// Its backward.  With g_ti the incoming gradient of the gate of a selected pair (0 for pairs not
// selected) and s_t = sum_i g_ti p_ti over the selected experts of token t,
//   d delta_tj = p_tj (g_tj - s_t)        for every expert j (the softmax couples them all).
template <class S>
void softmax_gate_bwd(int T, int E, int C_stride, const S* delta, const int32_t* slot_token,
                      const S* dgate, S* ddelta) {
  std::vector<double> g((size_t)T * E, 0.0);
  for (int i = 0; i < E; ++i)
    for (int p = 0; p < C_stride; ++p) {
      const size_t r = (size_t)i * C_stride + p;
      if (slot_token[r] >= 0) g[(size_t)slot_token[r] * E + i] = (double)dgate[r];
    }
  for (int t = 0; t < T; ++t) {
    const S* dt = delta + (size_t)t * E;
    double mx = (double)dt[0];
    for (int j = 1; j < E; ++j) mx = std::max(mx, (double)dt[j]);
    double den = 0.0;
    for (int j = 0; j < E; ++j) den += std::exp((double)dt[j] - mx);
    double st = 0.0;
    for (int j = 0; j < E; ++j) st += g[(size_t)t * E + j] * (std::exp((double)dt[j] - mx) / den);
    for (int j = 0; j < E; ++j) {
      const double pj = std::exp((double)dt[j] - mx) / den;
      ddelta[(size_t)t * E + j] = (S)(pj * (g[(size_t)t * E + j] - st));
    }
  }
}

// ---- load statistics (inputs of the auxiliary and locality losses) -------------------------------
// load[i] = counts[i] / T, the share of the batch's tokens expert i processes;
// gate_mean[i] = (1/T) sum of the gates of expert i's rows (its mean gate over all T tokens, a
// token it does not process counting as 0).
template <class S>
void load_stats(int T, int E, int C_stride, const int32_t* counts, const int32_t* slot_token,
                const S* gate, S* load, S* gate_mean) {
  for (int i = 0; i < E; ++i) {
    double acc = 0.0;
    for (int p = 0; p < C_stride; ++p) {
      const size_t r = (size_t)i * C_stride + p;
      if (slot_token[r] >= 0) acc += (double)gate[r];
    }
    load[i] = (S)((double)counts[i] / (double)T);
    gate_mean[i] = (S)(acc / (double)T);
  }
}

// ---- backward of the affinity ----------------------------------------------------------------
// With a = ||x_t||, b = ||R_i||, c = sqrt(D)/(a b):
//   d delta_ti / d x_t[q] = c R_i[q div D]/D - delta_ti x_t[q]/a^2
//   d delta_ti / d R_i[j] = c z_t[j]         - delta_ti R_i[j]/b^2
// dX is ACCUMULATED into (it already holds the FFN path's gradient); dR is overwritten.
template <class S>
void affinity_bwd(int T, int d, int D, int E, const S* X, const S* R, const S* delta,
                  const S* xnorm, const S* rnorm, const S* ddelta, S* dX, S* dR) {
  const int m = d / D;
  const double sqD = std::sqrt((double)D);
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    const double a = (double)xnorm[t];
    if (a == 0.0) continue;
    for (int q = 0; q < d; ++q) {
      double acc = 0.0;
      for (int i = 0; i < E; ++i) {
        const double dd = (double)ddelta[(size_t)t * E + i];
        const double b = (double)rnorm[i];
        if (dd == 0.0 || b == 0.0) continue;
        acc += dd * (sqD / (a * b) * (double)R[(size_t)i * m + q / D] / (double)D
                     - (double)delta[(size_t)t * E + i] * (double)X[(size_t)t * d + q] / (a * a));
      }
      dX[(size_t)t * d + q] = (S)((double)dX[(size_t)t * d + q] + acc);
    }
  }
  std::vector<S> Z((size_t)T * m);
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t)
    for (int j = 0; j < m; ++j) {
      double acc = 0.0;
      for (int r = 0; r < D; ++r) acc += (double)X[(size_t)t * d + j * D + r];
      Z[(size_t)t * m + j] = (S)(acc / (double)D);
    }
#pragma omp parallel for schedule(static)
  for (int i = 0; i < E; ++i) {
    const double b = (double)rnorm[i];
    std::vector<double> acc(m, 0.0);
    for (int t = 0; t < T; ++t) {
      const double dd = (double)ddelta[(size_t)t * E + i];
      const double a = (double)xnorm[t];
      if (dd == 0.0 || a == 0.0 || b == 0.0) continue;
      const double c = sqD / (a * b), dl = (double)delta[(size_t)t * E + i];
      for (int j = 0; j < m; ++j)
        acc[j] += dd * (c * (double)Z[(size_t)t * m + j] - dl * (double)R[(size_t)i * m + j] / (b * b));
    }
    for (int j = 0; j < m; ++j) dR[(size_t)i * m + j] = (S)acc[j];
  }
}

}  // namespace etr_oracle
