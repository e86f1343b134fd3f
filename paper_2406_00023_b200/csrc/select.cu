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
};

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
                         uint32_t* __restrict__ keyT, etr_stats* stats, SelectParams p) {
  __shared__ uint32_t tile[256 * (SEL_TB + 1)];      // [E][33]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t0 = blockIdx.x * SEL_TB;
  if (blockIdx.x == 0 && tid == 0) {
    const uint32_t mk = stats->delta_max_key;
    const float dm = mk ? key_to_float(mk) : 0.f;
    stats->delta_max = dm;
    stats->mode = p.mode;
    stats->C = capacity_from_delta(p, dm);
  }
  for (int tt = warp; tt < SEL_TB; tt += 8) {
    const int t = t0 + tt;
    uint32_t key[SEL_MAX_EPL];
    bool cand[SEL_MAX_EPL];
#pragma unroll
    for (int u = 0; u < SEL_MAX_EPL; ++u) {
      const int i = lane + 32 * u;
      key[u] = (t < p.T && i < p.E) ? ordered_key(delta[(size_t)t * p.E + i]) : 0u;
      cand[u] = (p.mode == ETR_MODE_ECR);
    }
    if (p.mode == ETR_MODE_TCR && t < p.T) {
      for (int j = 0; j < p.k; ++j) {
        // arg-max over (key, lower index wins) among experts not yet taken
        unsigned long long best = 0ull;
#pragma unroll
        for (int u = 0; u < SEL_MAX_EPL; ++u) {
          const int i = lane + 32 * u;
          if (i < p.E && !cand[u]) {
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
        if (lane == (win & 31)) {
#pragma unroll
          for (int u = 0; u < SEL_MAX_EPL; ++u) if (u == (win >> 5)) cand[u] = true;
        }
        if (lane == 0) topk_idx[(size_t)t * p.k + j] = win;
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
  __syncthreads();
  for (int idx = tid; idx < p.E * SEL_TB; idx += 256) {
    const int i = idx / SEL_TB, tt = idx % SEL_TB;
    if (t0 + tt < p.T) keyT[(size_t)i * p.T + t0 + tt] = tile[i * (SEL_TB + 1) + tt];
  }
}

// Histogram add with warp aggregation: lanes holding the same digit elect one leader that
// adds their number.  Affinity keys share their top bits, so the unaggregated form would
// serialise on a handful of bins.
__device__ __forceinline__ void hist_add(uint32_t* hist, uint32_t digit, bool active) {
  const uint32_t amask = __ballot_sync(0xffffffffu, active);
  if (active) {
    const uint32_t peers = __match_any_sync(amask, digit);
    if ((threadIdx.x & 31) == (uint32_t)(__ffs(peers) - 1)) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
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
                          int32_t* __restrict__ counts, int32_t* __restrict__ slot_token,
                          float* __restrict__ gate, int T, int C_stride) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_remaining, s_ncand;
  __shared__ uint32_t warp_tot[32], warp_pre[32];
  __shared__ uint32_t base_sel, base_eq;
  const int i = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t* row = keyT + (size_t)i * T;
  int32_t* my_slot = slot_token + (size_t)i * C_stride;
  float* my_gate = gate + (size_t)i * C_stride;
  const int C = stats->C;

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
        hist_add(hist, (kx >> shift) & 0xffu, in_range && (kx & pmask) == prefix);
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
    if (tid == 0) {
      uint32_t rem = pass == 0 ? n_keep : s_remaining;
      int b = 255;
      for (; b > 0; --b) {
        if (hist[b] >= rem) break;
        rem -= hist[b];
      }
      s_prefix = prefix | ((uint32_t)b << shift);
      s_remaining = rem;        // after the last pass: how many keys == tau are admitted
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
                int nblocks, int n_cand) {
  __shared__ int wsum[32], wpre[32];
  __shared__ int carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { carry = 0; tok_ptr[0] = 0; }
  __syncthreads();
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
    stats->dropped = n_cand - carry;
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
size_t select_workspace_bytes(const etr_config* c) {
  return select_keys_bytes(c) + align_up((size_t)ceil_div(c->T, 256) * sizeof(int32_t), 256);
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
  uint32_t* keyT = (uint32_t*)ws;
  ETR_TIME_BEGIN("select_token_side_kernel");
  select_token_side_kernel<<<ceil_div(c->T, SEL_TB), 256, 0, st>>>(delta, rt->topk_idx, keyT, stats, p);
  ETR_LAUNCH_CHECK();
  ETR_TIME_BEGIN("select_expert_side_kernel");
  select_expert_side_kernel<<<c->E, 1024, 0, st>>>(keyT, stats, rt->counts, rt->slot_token, rt->gate,
                                                   c->T, p.C_stride);
  ETR_LAUNCH_CHECK();
  ETR_TIME_BEGIN("csr_count_kernel");
  int32_t* block_total = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(ws) + select_keys_bytes(c));
  const int nblocks = ceil_div(c->T, 256);
  csr_count_kernel<<<nblocks, 256, 0, st>>>((const int32_t*)keyT, rt->tok_ptr, block_total, stats, c->T, c->E);
  ETR_LAUNCH_CHECK();
  const int n_cand = p.mode == ETR_MODE_TCR ? c->T * c->k : c->T * c->E;
  ETR_TIME_BEGIN("csr_scan_kernel");
  csr_scan_kernel<<<1, 1024, 0, st>>>(block_total, rt->tok_ptr, stats, nblocks, n_cand);
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

// the keys, plus the per-block scan scratch (one int per 256 tokens; T <= 4 Mi)
constexpr size_t SELECT_STATIC_MAX_BYTES = ETR_SELECT_STATIC_MAX_ENTRIES * sizeof(uint32_t) + (64u << 10) + 512u;
static __device__ __align__(256) unsigned char g_select_scratch[SELECT_STATIC_MAX_BYTES];

// In host code `g_select_scratch` is only a handle for the runtime's symbol table, not a
// device address; the address is looked up once per device and cached.
static std::mutex g_scratch_mu;
static void* g_scratch_addr[64] = {};

static etr_status select_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ETR_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_scratch_mu);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || p == nullptr) return ETR_ERR_CUDA;
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
  if (delta == nullptr || stats == nullptr || route == nullptr) return ETR_ERR_ARG;
  if (!route->topk_idx || !route->counts || !route->slot_token || !route->gate || !route->tok_ptr ||
      !route->tok_row)
    return ETR_ERR_ARG;
  if (!aligned16(delta) || !aligned16(stats)) return ETR_ERR_ALIGN;
  if ((unsigned long long)cfg->T * (unsigned long long)cfg->E > ETR_SELECT_STATIC_MAX_ENTRIES ||
      select_workspace_bytes(cfg) > SELECT_STATIC_MAX_BYTES)
    return ETR_ERR_WORKSPACE;
  void* scratch = nullptr;
  ETR_TRY(select_scratch_address(&scratch));
  return select_forward(cfg, delta, stats, route, scratch, (cudaStream_t)stream);
}
