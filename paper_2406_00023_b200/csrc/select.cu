// Bidirectional selection: token-side top-k, expert-side top-C, routing maps.
//
// All decisions are taken on order-preserving 32-bit integer images of the fp32
// affinities, so there is no floating-point arithmetic here and the result is exact:
//   1. token side (one warp per token): the k best experts by (key desc, index asc);
//      writes topk_idx and the transposed key matrix keyT[E][T] (0 = not a candidate;
//      in expert choice every pair is a candidate).  Block 0 also fixes mode and C.
//   2. expert side (one CTA per expert): 4-pass 8-bit radix select over the expert's row
//      of keyT finds the C-th largest key tau; tokens with key > tau are kept, and of the
//      tokens with key == tau the lowest token ids fill the remaining quota; a ballot
//      scan in token order assigns slots (ascending token id).  The row of keyT is
//      overwritten with the slot position (or -1).
//   3. token-major CSR from the position matrix: count, exclusive scan, fill.
#include <mutex>

#include "common.cuh"

namespace etr {

constexpr int SEL_TB = 32;         // tokens per CTA on the token side
constexpr int SEL_MAX_EPL = 8;     // experts per lane: E <= 256

struct SelectParams {
  int T, E, k, d, C_stride, capacity, c_floor, adaptive, mode;
  float delta_max_override;
  int cut_token;              // token choice: a token stops taking experts once the sum of the taken affinities reaches tq_token
  long long tq_token;         // threshold on 2^-32 integers
};

// Affinity as a multiple of 2^-32 (round to nearest even): the unit the threshold sums are taken in,
// so that they are exact and independent of the order of summation.
__device__ __forceinline__ long long quantise_affinity(float delta) {
  return __double2ll_rn((double)delta * 4294967296.0);
}
static long long quantise_threshold(float tau) {
  const double s = (double)tau * 4294967296.0;
  if (!(s < 9.2e18)) return 0x7fffffffffffffffll;        // +infinity: never reached
  if (s < -9.2e18) return (long long)0x8000000000000000ull;
  return llrint(s);
}

// C = capacity, or clamp(ceil((1/E) exp{d dm^2/(2-dm^2)}), c_floor, capacity).
__device__ inline int capacity_from_delta(const SelectParams& p, float delta_max) {
  if (!p.adaptive) return p.capacity;
  double ds = p.delta_max_override >= 0.f ? (double)p.delta_max_override : (double)delta_max;
  ds = fmin(1.0, fmax(0.0, ds));
  const double y = (double)p.d * ds * ds / (2.0 - ds * ds);
  const double cmin = ceil(exp(y) / (double)p.E);
  const double c = fmin((double)p.capacity, fmax((double)p.c_floor, cmin));
  return (int)c;
}

__global__ void __launch_bounds__(256)
select_token_side_kernel(const float* __restrict__ delta, int32_t* __restrict__ topk_idx,
                         uint32_t* __restrict__ keyT, etr_stats* stats, int32_t* __restrict__ skipped,
                         SelectParams p) {
  __shared__ uint32_t tile[256 * (SEL_TB + 1)];      // [E][33]
  __shared__ int s_skipped;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t0 = blockIdx.x * SEL_TB;
  if (tid == 0) s_skipped = 0;
  if (p.cut_token) __syncthreads();
  int n_skipped = 0;                                 // ranks this warp's tokens gave up (lane 0 counts)
  if (blockIdx.x == 0 && tid == 0) {
    const uint32_t mk = stats->delta_max_key;
    const float dm = mk ? key_to_float(mk) : 0.f;
    stats->delta_max = dm;
    stats->mode = p.mode;
    stats->C = capacity_from_delta(p, dm);
    // the CSR kernels that follow on the stream add to these: every selection starts them at zero
    stats->unrouted = 0;
    stats->dropped = 0;
    stats->rows_total = 0;
  }
  for (int tt = warp; tt < SEL_TB; tt += 8) {
    const int t = t0 + tt;
    uint32_t key[SEL_MAX_EPL];
    bool cand[SEL_MAX_EPL], taken[SEL_MAX_EPL];
#pragma unroll
    for (int u = 0; u < SEL_MAX_EPL; ++u) {
      const int i = lane + 32 * u;
      key[u] = (t < p.T && i < p.E) ? ordered_key(delta[(size_t)t * p.E + i]) : 0u;
      cand[u] = (p.mode == ETR_MODE_ECR);
      taken[u] = false;
    }
    if (p.mode == ETR_MODE_TCR && t < p.T) {
      long long sum_before = 0;                      // of the affinities of the ranks before j (threshold walk)
      bool open = true;
      for (int j = 0; j < p.k; ++j) {
        // arg-max over (key, lower index wins) among experts not yet taken
        unsigned long long best = 0ull;
#pragma unroll
        for (int u = 0; u < SEL_MAX_EPL; ++u) {
          const int i = lane + 32 * u;
          if (i < p.E && !taken[u]) {
            const unsigned long long v = ((unsigned long long)key[u] << 32) | (uint32_t)(0x7fffffff - i);
            best = v > best ? v : best;
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
          best = other > best ? other : best;
        }
        const int win = 0x7fffffff - (int)(uint32_t)(best & 0xffffffffull);
        if (p.cut_token) {                           // the walk stops at the first rank it does not keep
          open = open && sum_before < p.tq_token;
          sum_before += quantise_affinity(key_to_float((uint32_t)(best >> 32)));
          n_skipped += !open;
        }
        if (lane == (win & 31)) {
#pragma unroll
          for (int u = 0; u < SEL_MAX_EPL; ++u) if (u == (win >> 5)) { taken[u] = true; cand[u] = open; }
        }
        if (lane == 0) topk_idx[(size_t)t * p.k + j] = open ? win : -1;
      }
    } else if (t < p.T) {
      for (int j = lane; j < p.k; j += 32) topk_idx[(size_t)t * p.k + j] = -1;
    }
#pragma unroll
    for (int u = 0; u < SEL_MAX_EPL; ++u) {
      const int i = lane + 32 * u;
      if (i < p.E) tile[i * (SEL_TB + 1) + tt] = cand[u] ? key[u] : 0u;
    }
  }
  if (p.cut_token && lane == 0 && n_skipped) atomicAdd(&s_skipped, n_skipped);
  __syncthreads();
  if (tid == 0 && skipped) skipped[blockIdx.x] = s_skipped;        // candidates given up by this block's tokens
  for (int idx = tid; idx < p.E * SEL_TB; idx += 256) {
    const int i = idx / SEL_TB, tt = idx % SEL_TB;
    if (t0 + tt < p.T) keyT[(size_t)i * p.T + t0 + tt] = tile[i * (SEL_TB + 1) + tt];
  }
}

// Histogram add.  In the first pass (top byte) affinity keys share their top bits and plain
// atomics would serialise on a handful of bins, so lanes holding the same digit elect one
// leader that adds their number.
__device__ __forceinline__ void hist_add(uint32_t* hist, uint32_t digit, bool active, bool aggregate) {
  if (aggregate) {
    const uint32_t amask = __ballot_sync(0xffffffffu, active);
    if (active) {
      const uint32_t peers = __match_any_sync(amask, digit);
      if ((threadIdx.x & 31) == (uint32_t)(__ffs(peers) - 1)) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
    }
  } else if (active) {
    atomicAdd(&hist[digit], 1u);      // later passes: few keys match the prefix and their digits spread
  }
}

// Radix step by one warp: walking the 256 bins from the top, the first bin whose count reaches
// `rem` (bin 0 takes whatever is left); rem is reduced by the counts of the bins above it.
// Lane l owns bins 255-8l .. 248-8l.  The result is returned in every lane.
__device__ __forceinline__ void pick_bin(const uint32_t* hist, uint32_t rem, int lane, uint32_t& bin,
                                         uint32_t& rem_out) {
  uint32_t c[8], mine = 0;
#pragma unroll
  for (int u = 0; u < 8; ++u) { c[u] = hist[255 - 8 * lane - u]; mine += c[u]; }
  uint32_t inc = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  const uint32_t hit = __ballot_sync(0xffffffffu, inc >= rem || lane == 31);
  const int owner = __ffs(hit) - 1;
  uint32_t b = 0, r = rem - (inc - mine);
  if (lane == owner) {
    int u = 0;
    for (; u < 8; ++u) {
      const int idx = 255 - 8 * lane - u;
      if (idx == 0 || c[u] >= r) break;
      r -= c[u];
    }
    b = (uint32_t)(255 - 8 * lane - u);
  }
  bin = __shfl_sync(0xffffffffu, b, owner);
  rem_out = __shfl_sync(0xffffffffu, r, owner);
}

// Expert-side threshold: limit[i] = how many of expert i's candidates, taken in descending affinity,
// it takes before the running sum of their affinities (2^-32 integers) reaches tq; INT_MAX if it
// never does.  The candidate of rank j is kept while the sum of the j-1 before it is below tq, so the
// number kept is the first j whose sum reaches tq.  Sums only grow while affinities are positive, and
// a radix bin never mixes signs (the sign is the key's top bit), so the crossing is found like the
// C-th largest key: four 8-bit passes over the expert's keys, here with a histogram of counts and one
// of sums per pass, walking the bins from the top to the first one whose cumulated sum reaches what
// is left of tq.  In the last pass a bin is a single key value q > 0, of which ceil(left / q) are needed.
__global__ void __launch_bounds__(1024)
select_threshold_limit_kernel(const uint32_t* __restrict__ keyT, int32_t* __restrict__ limit, int T,
                              long long tq) {
  __shared__ uint32_t hist_cnt[256];
  __shared__ unsigned long long hist_sum[256];
  __shared__ uint32_t s_prefix, s_before;
  __shared__ long long s_left;
  __shared__ int s_state;                            // 0: walking, 1: never reached
  const int i = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  const uint32_t* row = keyT + (size_t)i * T;
  if (tq <= 0) { if (tid == 0) limit[i] = 0; return; }
  if (tid == 0) { s_prefix = 0; s_before = 0; s_left = tq; s_state = 0; }
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) { hist_cnt[tid] = 0; hist_sum[tid] = 0ull; }
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t pmask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    for (int c0 = 0; c0 < T; c0 += 1024) {
      const int t = c0 + tid;
      const uint32_t kx = t < T ? row[t] : 0u;
      const bool active = kx != 0u && (kx & pmask) == prefix;
      const uint32_t digit = (kx >> shift) & 0xffu;
      const long long q = active ? quantise_affinity(key_to_float(kx)) : 0ll;
      // lanes holding the same digit add once, through their first lane
      uint32_t todo = __ballot_sync(0xffffffffu, active);
      while (todo) {
        const int leader = __ffs(todo) - 1;
        const uint32_t d0 = __shfl_sync(0xffffffffu, digit, leader);
        const bool mine = active && digit == d0;
        const uint32_t group = __ballot_sync(0xffffffffu, mine);
        long long sum = mine ? q : 0ll;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == leader) {
          atomicAdd(&hist_cnt[d0], (uint32_t)__popc(group));
          atomicAdd(&hist_sum[d0], (unsigned long long)sum);
        }
        todo &= ~group;
      }
    }
    __syncthreads();
    if (tid == 0) {
      long long cum = 0, left = s_left;
      uint32_t cnt = 0;
      int found = -1;
      for (int b = 255; b >= 0; --b) {
        if (hist_cnt[b] == 0) continue;
        const long long sb = (long long)hist_sum[b];
        if (cum + sb >= left) { found = b; break; }
        cum += sb;
        cnt += hist_cnt[b];
      }
      if (found < 0) {
        s_state = 1;
      } else {
        s_prefix = prefix | ((uint32_t)found << shift);
        s_left = left - cum;
        s_before += cnt;
      }
    }
    __syncthreads();
    if (s_state) break;                              // uniform across the CTA
  }
  if (tid == 0) {
    if (s_state) {
      limit[i] = 0x7fffffff;
    } else {
      const long long q = quantise_affinity(key_to_float(s_prefix));      // > 0: its bin's sum crossed
      limit[i] = (int32_t)(s_before + (uint32_t)((s_left + q - 1) / q));
    }
  }
}

// One CTA (1024 threads) per expert; every thread owns 4 consecutive tokens per sweep.
constexpr int SEL_KPT = 4;
constexpr int SEL_SWEEP = 1024 * SEL_KPT;

__device__ __forceinline__ void load_keys(const uint32_t* __restrict__ row, int t0, int T, uint32_t* k) {
#pragma unroll
  for (int u = 0; u < SEL_KPT; ++u) k[u] = t0 + u < T ? row[t0 + u] : 0u;
}

__global__ void __launch_bounds__(1024)
select_expert_side_kernel(uint32_t* __restrict__ keyT, const etr_stats* __restrict__ stats,
                          const int32_t* __restrict__ limit, int32_t* __restrict__ counts,
                          int32_t* __restrict__ slot_token, float* __restrict__ gate, int T, int C_stride) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_remaining, s_ncand;
  __shared__ uint32_t warp_tot[32], warp_pre[32];
  __shared__ uint32_t base_sel, base_eq;
  const int i = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t* row = keyT + (size_t)i * T;
  int32_t* my_slot = slot_token + (size_t)i * C_stride;
  float* my_gate = gate + (size_t)i * C_stride;
  const int C = limit ? min(stats->C, limit[i]) : stats->C;      // limit: the threshold on the sum of affinities

  // radix select, 4 passes of 8 bits: the n_keep-th largest key; pass 0 also counts candidates
  uint32_t tau = 0, quota = 0, n_keep = 0;
  if (tid == 0) { s_prefix = 0; s_ncand = 0; }
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t pmask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    uint32_t nc = 0;
    uint32_t cur[SEL_KPT], nxt[SEL_KPT];
    load_keys(row, tid * SEL_KPT, T, cur);
    for (int c0 = 0; c0 < T; c0 += SEL_SWEEP) {
      if (c0 + SEL_SWEEP < T) load_keys(row, c0 + SEL_SWEEP + tid * SEL_KPT, T, nxt);   // prefetch
#pragma unroll
      for (int u = 0; u < SEL_KPT; ++u) {
        const uint32_t kx = cur[u];
        const bool in_range = c0 + tid * SEL_KPT + u < T;
        nc += (in_range && kx != 0u);
        hist_add(hist, (kx >> shift) & 0xffu, in_range && (kx & pmask) == prefix, pass == 0);
      }
#pragma unroll
      for (int u = 0; u < SEL_KPT; ++u) cur[u] = nxt[u];
    }
    if (pass == 0) {
      for (int o = 16; o > 0; o >>= 1) nc += __shfl_xor_sync(0xffffffffu, nc, o);
      if (lane == 0 && nc) atomicAdd(&s_ncand, nc);
    }
    __syncthreads();
    if (pass == 0) n_keep = min((uint32_t)C, s_ncand);
    if (n_keep == 0) break;                       // uniform across the CTA
    if (warp == 0) {
      uint32_t b, rem;
      pick_bin(hist, pass == 0 ? n_keep : s_remaining, lane, b, rem);
      if (lane == 0) {
        s_prefix = prefix | (b << shift);
        s_remaining = rem;      // after the last pass: how many keys == tau are admitted
      }
    }
    __syncthreads();
  }
  if (n_keep > 0) { tau = s_prefix; quota = s_remaining; }

  // slot assignment in ascending token order
  if (tid == 0) { base_sel = 0; base_eq = 0; }
  __syncthreads();
  uint32_t cur[SEL_KPT], nxt[SEL_KPT];
  load_keys(row, tid * SEL_KPT, T, cur);
  for (int c0 = 0; c0 < T; c0 += SEL_SWEEP) {
    if (c0 + SEL_SWEEP < T) load_keys(row, c0 + SEL_SWEEP + tid * SEL_KPT, T, nxt);
    const int tb = c0 + tid * SEL_KPT;
    uint32_t ngt = 0, neq = 0;
#pragma unroll
    for (int u = 0; u < SEL_KPT; ++u) {
      const bool live = n_keep > 0 && tb + u < T && cur[u] != 0u;
      ngt += live && cur[u] > tau;
      neq += live && cur[u] == tau;
    }
    // block-wide exclusive scan of (ngt, neq), packed 16 bits apart (each < 2^13 per sweep)
    const uint32_t mine = ngt | (neq << 16);
    uint32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += y;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      const uint32_t wt = warp_tot[lane];
      uint32_t winc = wt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += y;
      }
      warp_pre[lane] = winc - wt;
      if (lane == 31) warp_tot[0] = winc;          // sweep totals
    }
    __syncthreads();
    const uint32_t excl = warp_pre[warp] + inc - mine;
    const uint32_t tot = warp_tot[0];
    uint32_t gt_before = excl & 0xffffu, eq_rank = base_eq + (excl >> 16);
    const uint32_t eq_before_sweep = min(base_eq, quota);
    const uint32_t bs = base_sel;
#pragma unroll
    for (int u = 0; u < SEL_KPT; ++u) {
      const int t = tb + u;
      const uint32_t kx = cur[u];
      const bool live = n_keep > 0 && t < T && kx != 0u;
      const bool gt = live && kx > tau, eq = live && kx == tau;
      int pos = -1;
      if (gt || (eq && eq_rank < quota)) {
        pos = (int)(bs + gt_before + (min(eq_rank, quota) - eq_before_sweep));
        my_slot[pos] = t;
        my_gate[pos] = key_to_float(kx);
      }
      if (t < T) row[t] = (uint32_t)pos;
      gt_before += gt;
      eq_rank += eq;
    }
    __syncthreads();
    if (tid == 0) {
      const uint32_t tot_gt = tot & 0xffffu, tot_eq = tot >> 16;
      const uint32_t eq_after = min(base_eq + tot_eq, quota);
      base_sel += tot_gt + (eq_after - eq_before_sweep);
      base_eq += tot_eq;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < SEL_KPT; ++u) cur[u] = nxt[u];
  }
  for (int p = (int)n_keep + tid; p < C_stride; p += 1024) { my_slot[p] = -1; my_gate[p] = 0.f; }
  if (tid == 0) counts[i] = (int)n_keep;
}

// The same selection with an expert's row of keys split over a thread-block cluster of CL CTAs
// (large T: one CTA per expert leaves most SMs idle and walks 64 Ki keys five times).  Each CTA
// histograms its own quarter of the tokens; the CL histograms are added through distributed
// shared memory after a hardware cluster barrier, so every CTA takes the same radix decision;
// the slot positions of a CTA start after the kept tokens of the lower-ranked CTAs.
__device__ __forceinline__ uint32_t sel_cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void sel_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t sel_peer_load(const uint32_t* local, uint32_t rank) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(local), ra, v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(ra) : "memory");
  return v;
}

template <int CL>
__global__ void __launch_bounds__(1024, 2)
select_expert_side_cluster_kernel(uint32_t* __restrict__ keyT, const etr_stats* __restrict__ stats,
                                  const int32_t* __restrict__ limit, int32_t* __restrict__ counts,
                                  int32_t* __restrict__ slot_token, float* __restrict__ gate, int T,
                                  int C_stride) {
  __shared__ uint32_t hist[256], tot[256];
  __shared__ uint32_t s_prefix, s_remaining, s_ncand_local, s_ncand;
  __shared__ uint32_t s_cnt_gt, s_cnt_eq;
  __shared__ uint32_t warp_tot[32], warp_pre[32];
  __shared__ uint32_t base_sel, base_eq;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t rank = sel_cluster_rank();
  const int i = blockIdx.x / CL;
  const int span = ((T + CL - 1) / CL + SEL_KPT - 1) / SEL_KPT * SEL_KPT;
  const int t_beg = min(T, (int)rank * span), t_end = min(T, t_beg + span);
  uint32_t* row = keyT + (size_t)i * T;
  int32_t* my_slot = slot_token + (size_t)i * C_stride;
  float* my_gate = gate + (size_t)i * C_stride;
  const int C = limit ? min(stats->C, limit[i]) : stats->C;

  // this CTA's keys are read from global memory once and stay in shared memory for every pass
  extern __shared__ uint32_t sk[];
  for (int t = t_beg + tid; t < t_end; t += 1024) sk[t - t_beg] = row[t];
  const uint32_t* rowl = sk - t_beg;              // rowl[t] for t in [t_beg, t_end)

  uint32_t tau = 0, quota = 0, n_keep = 0;
  if (tid == 0) { s_prefix = 0; s_ncand_local = 0; s_cnt_gt = 0; s_cnt_eq = 0; }
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t pmask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    uint32_t nc = 0;
    uint32_t cur[SEL_KPT], nxt[SEL_KPT];
    load_keys(rowl, t_beg + tid * SEL_KPT, t_end, cur);
    for (int c0 = t_beg; c0 < t_end; c0 += SEL_SWEEP) {
      if (c0 + SEL_SWEEP < t_end) load_keys(rowl, c0 + SEL_SWEEP + tid * SEL_KPT, t_end, nxt);
#pragma unroll
      for (int u = 0; u < SEL_KPT; ++u) {
        const uint32_t kx = cur[u];
        const bool in_range = c0 + tid * SEL_KPT + u < t_end;
        nc += (in_range && kx != 0u);
        hist_add(hist, (kx >> shift) & 0xffu, in_range && (kx & pmask) == prefix, pass == 0);
      }
#pragma unroll
      for (int u = 0; u < SEL_KPT; ++u) cur[u] = nxt[u];
    }
    if (pass == 0) {
      for (int o = 16; o > 0; o >>= 1) nc += __shfl_xor_sync(0xffffffffu, nc, o);
      if (lane == 0 && nc) atomicAdd(&s_ncand_local, nc);
    }
    __syncthreads();
    sel_cluster_sync();                           // every CTA's histogram of this pass is complete
    if (tid < 256) {
      uint32_t sum = 0;
#pragma unroll
      for (int r = 0; r < CL; ++r) sum += sel_peer_load(&hist[tid], r);
      tot[tid] = sum;
    }
    if (pass == 0 && tid == 256) {
      uint32_t sum = 0;
      for (int r = 0; r < CL; ++r) sum += sel_peer_load(&s_ncand_local, r);
      s_ncand = sum;
    }
    __syncthreads();
    if (pass == 0) n_keep = min((uint32_t)C, s_ncand);
    if (n_keep > 0 && warp == 0) {
      uint32_t b, rem;
      pick_bin(tot, pass == 0 ? n_keep : s_remaining, lane, b, rem);
      if (lane == 0) {
        s_prefix = prefix | (b << shift);
        s_remaining = rem;
      }
    }
    __syncthreads();
    sel_cluster_sync();                           // peers have read this CTA's histogram
    if (n_keep == 0) break;                       // same decision in every CTA of the cluster
  }
  __syncthreads();
  if (n_keep > 0) { tau = s_prefix; quota = s_remaining; }

  // kept tokens of the lower-ranked CTAs: count own keys above / equal to tau, exchange
  {
    uint32_t ngt = 0, neq = 0;
    for (int t = t_beg + tid; t < t_end; t += 1024) {
      const uint32_t kx = rowl[t];
      ngt += (n_keep > 0 && kx != 0u && kx > tau);
      neq += (n_keep > 0 && kx != 0u && kx == tau);
    }
    for (int o = 16; o > 0; o >>= 1) {
      ngt += __shfl_xor_sync(0xffffffffu, ngt, o);
      neq += __shfl_xor_sync(0xffffffffu, neq, o);
    }
    if (lane == 0) { if (ngt) atomicAdd(&s_cnt_gt, ngt); if (neq) atomicAdd(&s_cnt_eq, neq); }
    __syncthreads();
    sel_cluster_sync();
    if (tid == 0) {
      uint32_t gt_before = 0, eq_before = 0;
      for (uint32_t r = 0; r < rank; ++r) { gt_before += sel_peer_load(&s_cnt_gt, r); eq_before += sel_peer_load(&s_cnt_eq, r); }
      base_eq = eq_before;
      base_sel = gt_before + min(eq_before, quota);
    }
    __syncthreads();
  }

  // slot assignment over this CTA's tokens, ascending token order
  uint32_t cur[SEL_KPT], nxt[SEL_KPT];
  load_keys(rowl, t_beg + tid * SEL_KPT, t_end, cur);
  for (int c0 = t_beg; c0 < t_end; c0 += SEL_SWEEP) {
    if (c0 + SEL_SWEEP < t_end) load_keys(rowl, c0 + SEL_SWEEP + tid * SEL_KPT, t_end, nxt);
    const int tb = c0 + tid * SEL_KPT;
    uint32_t ngt = 0, neq = 0;
#pragma unroll
    for (int u = 0; u < SEL_KPT; ++u) {
      const bool live = n_keep > 0 && tb + u < t_end && cur[u] != 0u;
      ngt += live && cur[u] > tau;
      neq += live && cur[u] == tau;
    }
    const uint32_t mine = ngt | (neq << 16);
    uint32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += y;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      const uint32_t wt = warp_tot[lane];
      uint32_t winc = wt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += y;
      }
      warp_pre[lane] = winc - wt;
      if (lane == 31) warp_tot[0] = winc;
    }
    __syncthreads();
    const uint32_t excl = warp_pre[warp] + inc - mine;
    const uint32_t totals = warp_tot[0];
    uint32_t gt_before = excl & 0xffffu, eq_rank = base_eq + (excl >> 16);
    const uint32_t eq_before_sweep = min(base_eq, quota);
    const uint32_t bs = base_sel;
#pragma unroll
    for (int u = 0; u < SEL_KPT; ++u) {
      const int t = tb + u;
      const uint32_t kx = cur[u];
      const bool live = n_keep > 0 && t < t_end && kx != 0u;
      const bool gt = live && kx > tau, eq = live && kx == tau;
      int pos = -1;
      if (gt || (eq && eq_rank < quota)) {
        pos = (int)(bs + gt_before + (min(eq_rank, quota) - eq_before_sweep));
        my_slot[pos] = t;
        my_gate[pos] = key_to_float(kx);
      }
      if (t < t_end) row[t] = (uint32_t)pos;
      gt_before += gt;
      eq_rank += eq;
    }
    __syncthreads();
    if (tid == 0) {
      const uint32_t tot_gt = totals & 0xffffu, tot_eq = totals >> 16;
      const uint32_t eq_after = min(base_eq + tot_eq, quota);
      base_sel += tot_gt + (eq_after - eq_before_sweep);
      base_eq += tot_eq;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < SEL_KPT; ++u) cur[u] = nxt[u];
  }
  for (int p = (int)n_keep + (int)rank * 1024 + tid; p < C_stride; p += CL * 1024) { my_slot[p] = -1; my_gate[p] = 0.f; }
  if (tid == 0 && rank == 0) counts[i] = (int)n_keep;
  sel_cluster_sync();                             // no CTA leaves while a peer may still read its counters
}

// Token-major CSR in three small kernels without a long serial scan:
//   count  per-token row counts, exclusive scan inside each 256-token block (left in
//          tok_ptr[t+1]), block totals to scratch
//   scan   exclusive scan of the block totals (one CTA; T/256 values)
//   fill   tok_row from the position matrix, final tok_ptr
__global__ void __launch_bounds__(256)
csr_count_kernel(const int32_t* __restrict__ posT, int32_t* __restrict__ tok_ptr,
                 int32_t* __restrict__ block_total, etr_stats* stats, int T, int E) {
  __shared__ int wsum[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t = blockIdx.x * 256 + tid;
  int n = 0;
  if (t < T)
    for (int i = 0; i < E; ++i) n += posT[(size_t)i * T + t] >= 0;
  const uint32_t un = __ballot_sync(0xffffffffu, t < T && n == 0);
  if (lane == 0 && un) atomicAdd(&stats->unrouted, __popc(un));
  int inc = n;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) wsum[warp] = inc;
  __syncthreads();
  int pre = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < 8; ++w) { if (w < warp) pre += wsum[w]; tot += wsum[w]; }
  if (t < T) tok_ptr[t + 1] = pre + inc - n;          // exclusive, within the block
  if (tid == 0) block_total[blockIdx.x] = tot;
}

__global__ void __launch_bounds__(1024)
csr_scan_kernel(int32_t* __restrict__ block_total, int32_t* __restrict__ tok_ptr, etr_stats* stats,
                int nblocks, int n_cand, const int32_t* __restrict__ skipped, int n_skipped_blocks) {
  __shared__ int wsum[32], wpre[32];
  __shared__ int carry, given_up;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { carry = 0; given_up = 0; tok_ptr[0] = 0; }
  __syncthreads();
  if (skipped) {              // candidates the tokens gave up themselves (token-side threshold): integer sum
    int s = 0;
    for (int b = tid; b < n_skipped_blocks; b += 1024) s += skipped[b];
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0 && s) atomicAdd(&given_up, s);
    __syncthreads();
  }
  for (int c0 = 0; c0 < nblocks; c0 += 1024) {
    const int b = c0 + tid;
    const int v = b < nblocks ? block_total[b] : 0;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += y;
    }
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      const int wt = wsum[lane];
      int winc = wt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += y;
      }
      wpre[lane] = winc - wt;
      if (lane == 31) wsum[0] = winc;
    }
    __syncthreads();
    if (b < nblocks) block_total[b] = carry + wpre[warp] + inc - v;     // exclusive block offset
    const int total = wsum[0];
    __syncthreads();
    if (tid == 0) carry += total;
    __syncthreads();
  }
  if (tid == 0) {
    stats->rows_total = carry;
    stats->dropped = n_cand - given_up - carry;
  }
}

__global__ void __launch_bounds__(256)
csr_fill_kernel(const int32_t* __restrict__ posT, const int32_t* __restrict__ block_offset,
                int32_t* __restrict__ tok_ptr, int32_t* __restrict__ tok_row, int T, int E,
                int C_stride) {
  const int t = blockIdx.x * 256 + threadIdx.x;
  if (t >= T) return;
  int q = block_offset[blockIdx.x] + tok_ptr[t + 1];
  for (int i = 0; i < E; ++i) {
    const int pos = posT[(size_t)i * T + t];
    if (pos >= 0) tok_row[q++] = i * C_stride + pos;
  }
  tok_ptr[t + 1] = q;
}

// key / position matrix [E][T], then one int per 256-token block
static size_t select_keys_bytes(const etr_config* c) { return align_up((size_t)c->T * c->E * sizeof(uint32_t), 256); }
// ... then the per-expert threshold limits and the per-block counts of given-up candidates
static size_t select_scan_bytes(const etr_config* c) { return align_up((size_t)ceil_div(c->T, 256) * sizeof(int32_t), 256); }
static size_t select_limit_bytes(const etr_config* c) { return align_up((size_t)c->E * sizeof(int32_t), 256); }
size_t select_workspace_bytes(const etr_config* c) {
  return select_keys_bytes(c) + select_scan_bytes(c) + select_limit_bytes(c) +
         align_up((size_t)ceil_div(c->T, SEL_TB) * sizeof(int32_t), 256);
}

int resolve_mode(const etr_config* c) {
  if (c->mode == ETR_MODE_TCR || c->mode == ETR_MODE_ECR) return c->mode;
  return c->step < c->switch_step ? ETR_MODE_TCR : ETR_MODE_ECR;
}

etr_status select_forward(const etr_config* c, const float* delta, etr_stats* stats,
                          const etr_route* rt, void* ws, cudaStream_t st) {
  SelectParams p;
  p.T = c->T; p.E = c->E; p.k = c->k; p.d = c->d; p.C_stride = c_stride_of(c);
  p.capacity = c->capacity; p.c_floor = c->c_floor < 1 ? 1 : c->c_floor; p.adaptive = c->adaptive;
  p.mode = resolve_mode(c); p.delta_max_override = c->delta_max_override;
  p.cut_token = (c->threshold_mode & ETR_THRESHOLD_TOKEN) != 0 && p.mode == ETR_MODE_TCR;
  p.tq_token = quantise_threshold(c->threshold_tau_token);
  uint32_t* keyT = (uint32_t*)ws;
  char* ws_tail = reinterpret_cast<char*>(ws) + select_keys_bytes(c) + select_scan_bytes(c);
  int32_t* limit = (c->threshold_mode & ETR_THRESHOLD_EXPERT) ? reinterpret_cast<int32_t*>(ws_tail) : nullptr;
  int32_t* skipped = p.cut_token ? reinterpret_cast<int32_t*>(ws_tail + select_limit_bytes(c)) : nullptr;
  ETR_TIME_BEGIN("select_token_side_kernel");
  select_token_side_kernel<<<ceil_div(c->T, SEL_TB), 256, 0, st>>>(delta, rt->topk_idx, keyT, stats, skipped, p);
  ETR_LAUNCH_CHECK();
  if (limit) {
    ETR_TIME_BEGIN("select_threshold_limit_kernel");
    select_threshold_limit_kernel<<<c->E, 1024, 0, st>>>(keyT, limit, c->T, quantise_threshold(c->threshold_tau));
    ETR_LAUNCH_CHECK();
  }
  ETR_TIME_BEGIN("select_expert_side_kernel");
  if (c->T >= 8192 && c->T <= 4 * 49152) {     // split each expert's row over a cluster of 4 CTAs
    constexpr int CL = 4;
    const size_t key_bytes = (size_t)((ceil_div(c->T, CL) + SEL_KPT - 1) / SEL_KPT * SEL_KPT) * sizeof(uint32_t);
    static std::atomic<unsigned long long> attr_done{0};      // one bit per device
    if (!ensure_dyn_smem(select_expert_side_cluster_kernel<CL>, 196608, attr_done)) return ETR_ERR_CUDA;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(c->E * CL);
    lc.blockDim = dim3(1024);
    lc.dynamicSmemBytes = key_bytes;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (cudaLaunchKernelEx(&lc, select_expert_side_cluster_kernel<CL>, keyT, (const etr_stats*)stats,
                           (const int32_t*)limit, rt->counts, rt->slot_token, rt->gate, c->T,
                           p.C_stride) != cudaSuccess) {
      timing_end(st);
      return ETR_ERR_CUDA;
    }
  } else {
    select_expert_side_kernel<<<c->E, 1024, 0, st>>>(keyT, stats, limit, rt->counts, rt->slot_token, rt->gate,
                                                     c->T, p.C_stride);
  }
  ETR_LAUNCH_CHECK();
  ETR_TIME_BEGIN("csr_count_kernel");
  int32_t* block_total = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(ws) + select_keys_bytes(c));
  const int nblocks = ceil_div(c->T, 256);
  csr_count_kernel<<<nblocks, 256, 0, st>>>((const int32_t*)keyT, rt->tok_ptr, block_total, stats, c->T, c->E);
  ETR_LAUNCH_CHECK();
  const int n_cand = p.mode == ETR_MODE_TCR ? c->T * c->k : c->T * c->E;
  ETR_TIME_BEGIN("csr_scan_kernel");
  csr_scan_kernel<<<1, 1024, 0, st>>>(block_total, rt->tok_ptr, stats, nblocks, n_cand, skipped,
                                      ceil_div(c->T, SEL_TB));
  ETR_LAUNCH_CHECK();
  ETR_TIME_BEGIN("csr_fill_kernel");
  csr_fill_kernel<<<nblocks, 256, 0, st>>>((const int32_t*)keyT, block_total, rt->tok_ptr, rt->tok_row,
                                           c->T, c->E, p.C_stride);
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

}  // namespace etr

// ---- selection without caller scratch ----------------------------------------------------------
// Same kernels as select_forward, but the key matrix lives in a fixed device array that is
// part of the library image, for callers that have no way to allocate device memory (see
// etr_select_static in etr.h).  Every GPU that loads the library holds these bytes until the
// process exits.
namespace etr {

// the keys, plus the small arrays select_forward keeps behind them: one int per 256 tokens (scan), one
// per expert (threshold limits), one per 32 tokens (candidates given up); T <= 4 Mi, E <= 256
constexpr size_t SELECT_STATIC_MAX_BYTES = ETR_SELECT_STATIC_MAX_ENTRIES * sizeof(uint32_t) + (640u << 10);
static __device__ __align__(256) unsigned char g_select_scratch[SELECT_STATIC_MAX_BYTES];

// In host code `g_select_scratch` is only a handle for the runtime's symbol table, not a
// device address; the address is looked up once per device and cached.
static std::mutex g_scratch_mu;
static void* g_scratch_addr[64] = {};

static etr_status select_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return ETR_ERR_CUDA; }
  std::lock_guard<std::mutex> lk(g_scratch_mu);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();      // the failure is reported by the status; it must not stick to the next launch check
      return ETR_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return ETR_OK;
}

}  // namespace etr

extern "C" etr_status etr_select_static(const etr_config* cfg, const float* delta, etr_stats* stats,
                                        const etr_route* route, void* stream) {
  using namespace etr;
  ETR_TRY(etr_validate(cfg));
  // the same argument rules as etr_select
  if (delta == nullptr || stats == nullptr || route == nullptr) return ETR_ERR_ARG;
  const void* ptrs[6] = {route->topk_idx, route->counts, route->slot_token, route->gate, route->tok_ptr,
                         route->tok_row};
  for (const void* q : ptrs)
    if (q == nullptr) return ETR_ERR_ARG;
  if (!aligned16(delta) || !aligned16(stats)) return ETR_ERR_ALIGN;
  for (const void* q : ptrs)
    if (!aligned16(q)) return ETR_ERR_ALIGN;
  if ((unsigned long long)cfg->T * (unsigned long long)cfg->E > ETR_SELECT_STATIC_MAX_ENTRIES ||
      select_workspace_bytes(cfg) > SELECT_STATIC_MAX_BYTES)
    return ETR_ERR_WORKSPACE;
  void* scratch = nullptr;
  ETR_TRY(select_scratch_address(&scratch));
  return select_forward(cfg, delta, stats, route, scratch, (cudaStream_t)stream);
}
