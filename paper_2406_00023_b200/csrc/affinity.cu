// GrAP pooling + cosine affinity (forward) and the router gradient (backward).
//
// Forward, in the order the host code tries them:
//   split form (the caller keeps Z, which the backward pass needs anyway):
//     grap_pool_kernel             one streaming pass over X: pooled rows Z and ||x_t||
//     affinity_score_tile_kernel   s = Z R^T as a register-tiled fp32 GEMM, cosine, batch max
//                                  (E <= 64, 16 | m, a 256-token tile for every SM)
//     affinity_score_kernel        the same products with lane = expert, 8 tokens per warp
//   affinity_fwd_warp_kernel       one pass, pooling and score per warp (no Z kept)
//   affinity_fwd_kernel            one CTA per tile of AFF_TB tokens (shapes the others do not take):
//     phase 0  R -> shared memory (rows padded so 128-bit reads of 8 different rows hit
//              32 different banks), ||R_i|| by one warp per row
//     phase 1  each warp streams its tokens' rows of X once with 16-byte loads, pools the
//              D-groups in registers, accumulates ||x||^2, leaves z_t in shared memory
//     phase 2  s = Z R^T register-tiled (2 tokens x 4 experts per thread, float4 operands),
//              delta = sqrt(D) s / (||x|| ||R||), batch max through one atomicMax on the
//              order-preserving integer image (exact and order independent)
// Backward: affinity_bwd_dx_chunk_kernel (dX with the dispatch backward fused in, by chunks of
// tokens), affinity_bwd_dx_kernel (stage form, dense d delta, shapes the chunked form does not take),
// affinity_bwd_dr_*_kernel (dR in two fixed-order stages).
#include <algorithm>

#include "common.cuh"

namespace etr {

constexpr int AFF_TB = 32;        // tokens per CTA
constexpr int AFF_THREADS = 256;

// Raw 16-byte pieces of a row, converted only when consumed (keeps a batch of loads cheap
// in registers).
template <class T> struct Raw16;
template <> struct Raw16<__nv_bfloat16> {          // 8 elements
  static constexpr int ELEMS = 8;
  uint4 w;
  __device__ void load(const __nv_bfloat16* p) { w = __ldg(reinterpret_cast<const uint4*>(p)); }
  __device__ void reduce(float& s, float& sq) const {
    const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float a = __uint_as_float(u[i] << 16), b = __uint_as_float(u[i] & 0xffff0000u);
      s += a; s += b; sq = fmaf(a, a, sq); sq = fmaf(b, b, sq);
    }
  }
};
template <> struct Raw16<float> {                  // 4 elements
  static constexpr int ELEMS = 4;
  float4 w;
  __device__ void load(const float* p) { w = __ldg(reinterpret_cast<const float4*>(p)); }
  __device__ void reduce(float& s, float& sq) const {
    s += w.x; s += w.y; s += w.z; s += w.w;
    sq = fmaf(w.x, w.x, sq); sq = fmaf(w.y, w.y, sq); sq = fmaf(w.z, w.z, sq); sq = fmaf(w.w, w.w, sq);
  }
};

// Whole groups owned by a lane, PPG 16-byte pieces per group.  Loads are issued in batches of
// 8 independent pieces per lane before any is consumed, so one warp keeps 4 KiB in flight.
// Out-of-range groups re-read the lane's first group and are discarded (no predicated loads).
template <class T, int PPG>
__device__ inline float pool_groups(const T* __restrict__ x, float* __restrict__ zrow, int m, int lane,
                                    float invD) {
  constexpr int GB = PPG >= 8 ? 1 : 8 / PPG;      // groups per batch
  constexpr int D = Raw16<T>::ELEMS * PPG;
  float sq = 0.f;
  for (int j0 = lane; j0 < m; j0 += 32 * GB) {
    Raw16<T> q[GB][PPG];
#pragma unroll
    for (int g = 0; g < GB; ++g) {
      const int j = j0 + 32 * g;
      const T* src = x + (size_t)(j < m ? j : lane) * D;
#pragma unroll
      for (int v = 0; v < PPG; ++v) q[g][v].load(src + v * Raw16<T>::ELEMS);
    }
#pragma unroll
    for (int g = 0; g < GB; ++g) {
      const int j = j0 + 32 * g;
      float s = 0.f, q2 = 0.f;
#pragma unroll
      for (int v = 0; v < PPG; ++v) q[g][v].reduce(s, q2);
      if (j < m) { zrow[j] = s * invD; sq += q2; }
    }
  }
  return sq;
}

// Pools one token row into zrow[0..m) (lane-strided) and returns this lane's share of ||x||^2.
template <class T>
__device__ inline float pool_token_partial(const T* __restrict__ x, float* __restrict__ zrow, int d,
                                           int D, int m, int lane) {
  const float invD = 1.0f / (float)D;
  constexpr int PE = Raw16<T>::ELEMS;
  if (D == PE) return pool_groups<T, 1>(x, zrow, m, lane, invD);
  if (D == 2 * PE) return pool_groups<T, 2>(x, zrow, m, lane, invD);
  if (D == 4 * PE) return pool_groups<T, 4>(x, zrow, m, lane, invD);
  float sq = 0.f;
  if (D % 8 == 0) {                 // a lane owns whole groups: D/8 vectors each
    const int vpg = D / 8;
    for (int j = lane; j < m; j += 32) {
      float s = 0.f;
      for (int v = 0; v < vpg; ++v) {
        Vec8<T> q = Vec8<T>::load(x + (size_t)j * D + v * 8);
#pragma unroll
        for (int e = 0; e < 8; ++e) { s += q.v[e]; sq += q.v[e] * q.v[e]; }
      }
      zrow[j] = s * invD;
    }
  } else if (8 % D == 0) {          // a vector holds 8/D whole groups
    const int gpv = 8 / D;
#pragma unroll 4
    for (int v = lane; v < d / 8; v += 32) {
      Vec8<T> q = Vec8<T>::load(x + (size_t)v * 8);
#pragma unroll
      for (int e = 0; e < 8; ++e) sq += q.v[e] * q.v[e];
      for (int g = 0; g < gpv; ++g) {
        float s = 0.f;
        for (int r = 0; r < D; ++r) s += q.v[g * D + r];
        zrow[v * gpv + g] = s * invD;
      }
    }
  } else {                          // any other group size: scalar
    for (int j = lane; j < m; j += 32) {
      float s = 0.f;
      for (int r = 0; r < D; ++r) { float v = to_f32<T>(x[(size_t)j * D + r]); s += v; sq += v * v; }
      zrow[j] = s * invD;
    }
  }
  return sq;
}

template <class T>
__device__ inline void pool_token(const T* __restrict__ x, float* __restrict__ zrow, int d, int D,
                                  int m, int lane, float& sumsq) {
  sumsq = warp_sum(pool_token_partial<T>(x, zrow, d, D, m, lane));
}

// ---- forward, split form (the default when the caller keeps Z) -----------------------------------
// Kernel 1 streams X once and leaves the pooled rows Z and ||x_t||: one warp per token, the
// row dealt to the lanes as consecutive 16-byte pieces (each load instruction moves 512
// contiguous bytes), 8 independent loads per lane in flight; a group of D elements is PPG
// adjacent pieces whose partial sums meet through xor-shuffles.  Pure HBM streaming.
template <class T, int PPG>
__global__ void __launch_bounds__(256)
grap_pool_kernel(const T* __restrict__ X, float* __restrict__ Z, float* __restrict__ xnorm, int Ttok,
                 int d, int D, int m) {
  constexpr int PE = Raw16<T>::ELEMS;
  constexpr int BATCH = 8;
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= Ttok) return;
  const T* x = X + (size_t)t * d;
  float* zrow = Z + (size_t)t * m;
  float sq = 0.f;
  if (PPG > 0) {
    const float invD = 1.0f / (float)D;
    const int npieces = m * PPG;
    for (int p0 = 0; p0 < npieces; p0 += 32 * BATCH) {
      Raw16<T> q[BATCH];
#pragma unroll
      for (int g = 0; g < BATCH; ++g) {
        const int p = p0 + 32 * g + lane;
        q[g].load(x + (size_t)(p < npieces ? p : lane) * PE);
      }
#pragma unroll
      for (int g = 0; g < BATCH; ++g) {
        const int p = p0 + 32 * g + lane;
        float s = 0.f, q2 = 0.f;
        q[g].reduce(s, q2);
#pragma unroll
        for (int o = 1; o < (PPG > 0 ? PPG : 1); o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (p < npieces) {
          sq += q2;
          if ((lane & ((PPG > 0 ? PPG : 1) - 1)) == 0) zrow[p / (PPG > 0 ? PPG : 1)] = s * invD;
        }
      }
    }
  } else {
    sq = pool_token_partial<T>(x, zrow, d, D, m, lane);     // any group size
  }
  sq = warp_sum(sq);
  if (lane == 0) xnorm[t] = sqrtf(sq);
}

// Kernel 2: s = Z R^T and the cosine.  R stays in shared memory; each warp copies the pooled
// rows of TPG tokens into its slice (coalesced float4), then lane = expert, TPG x EPL
// accumulators, float4 operands (R rows conflict-free, z rows broadcast).  Bound by the fp32
// FMA rate (2 m E flop per token against 4 m bytes), not by HBM.
template <int EPL, int TPG>
__global__ void __launch_bounds__(512, 1)
affinity_score_kernel(const float* __restrict__ Z, const float* __restrict__ xnorm,
                      const float* __restrict__ R, float* __restrict__ delta,
                      float* __restrict__ rnorm, etr_stats* stats, int Ttok, int D, int E, int m,
                      int ldm) {
  extern __shared__ __align__(16) float smem[];
  constexpr int EROWS = 32 * EPL;
  const int nw = blockDim.x >> 5;
  float* Rs = smem;                               // [EROWS][ldm]
  float* rn = Rs + (size_t)EROWS * ldm;           // [EROWS]
  float* Zall = rn + EROWS;                       // [nw][TPG][ldm]
  __shared__ uint32_t red[16];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (int idx = tid; idx < EROWS * ldm; idx += blockDim.x) {
    const int i = idx / ldm, j = idx - i * ldm;
    Rs[idx] = (i < E && j < m) ? R[(size_t)i * m + j] : 0.f;
  }
  float* zs = Zall + (size_t)warp * TPG * ldm;
  for (int idx = lane; idx < TPG * ldm; idx += 32) zs[idx] = 0.f;
  __syncthreads();
  for (int i = warp; i < EROWS; i += nw) {
    float s = 0.f;
    for (int j = lane; j < m; j += 32) s += Rs[i * ldm + j] * Rs[i * ldm + j];
    s = warp_sum(s);
    if (lane == 0) {
      rn[i] = sqrtf(s);
      if (blockIdx.x == 0 && i < E) rnorm[i] = rn[i];
    }
  }
  __syncthreads();

  const float sqD = sqrtf((float)D);
  const int mr4 = (m + 3) / 4, rs4 = ldm / 4;
  const bool vec_ok = (m & 3) == 0;
  const int ngroups = (Ttok + TPG - 1) / TPG;
  float best = -INFINITY;
  for (int g = blockIdx.x * nw + warp; g < ngroups; g += gridDim.x * nw) {
    const int t0 = g * TPG;
    float xn[TPG];
#pragma unroll
    for (int u = 0; u < TPG; ++u) {
      const int t = t0 + u;
      xn[u] = t < Ttok ? xnorm[t] : 0.f;
      float* zr = zs + (size_t)u * ldm;
      if (t < Ttok) {
        const float* src = Z + (size_t)t * m;
        if (vec_ok) {
          for (int j = lane; j < m / 4; j += 32)
            reinterpret_cast<float4*>(zr)[j] = __ldg(reinterpret_cast<const float4*>(src) + j);
        } else {
          for (int j = lane; j < m; j += 32) zr[j] = src[j];
        }
      } else {
        for (int j = lane; j < m; j += 32) zr[j] = 0.f;
      }
    }
    __syncwarp();
    float acc[TPG][EPL];
#pragma unroll
    for (int u = 0; u < TPG; ++u)
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[u][e] = 0.f;
    const float4* r4 = reinterpret_cast<const float4*>(Rs) + (size_t)lane * rs4;
    const float4* z4 = reinterpret_cast<const float4*>(zs);
#pragma unroll 2
    for (int j = 0; j < mr4; ++j) {
      float4 r[EPL];
#pragma unroll
      for (int e = 0; e < EPL; ++e) r[e] = r4[(size_t)(32 * e) * rs4 + j];
#pragma unroll
      for (int u = 0; u < TPG; ++u) {
        const float4 z = z4[(size_t)u * rs4 + j];
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          acc[u][e] = fmaf(z.x, r[e].x, acc[u][e]); acc[u][e] = fmaf(z.y, r[e].y, acc[u][e]);
          acc[u][e] = fmaf(z.z, r[e].z, acc[u][e]); acc[u][e] = fmaf(z.w, r[e].w, acc[u][e]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < TPG; ++u) {
      const int t = t0 + u;
      if (t >= Ttok) continue;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int i = lane + 32 * e;
        if (i < E) {
          const float den = xn[u] * rn[i];
          const float v = den == 0.f ? 0.f : sqD * acc[u][e] / den;
          delta[(size_t)t * E + i] = v;
          best = fmaxf(best, v);
        }
      }
    }
    __syncwarp();        // the slice is rewritten by the next group's copy
  }
  uint32_t key = best == -INFINITY ? 0u : ordered_key(best);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
  if (lane == 0) red[warp] = key;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < nw; ++w) key = max(key, red[w]);
    if (key) atomicMax(&stats->delta_max_key, key);
  }
}

// Kernel 2, tiled form (E <= 64, m a multiple of 32): the same products as affinity_score_kernel, in
// the same order per (token, expert), laid out like a register-tiled fp32 GEMM.  A block of 8 warps
// takes tiles of 256 tokens; a lane is (token group tg = lane / 8, expert group eg = lane % 8) and
// owns 8 tokens (rows 4 u + tg of the warp's 32) x EPT experts (e 8 + eg): 8 EPT accumulators fed by
// 8 + EPT 16-byte shared-memory loads per 4 k, every one of them a single wavefront (4 consecutive
// token rows, 8 consecutive expert rows; both row strides are 4 banks modulo 32).  The pooled rows
// arrive 32 columns at a time by asynchronous 16-byte copies into two buffers: the copy of a stage
// runs under the products of the one before, one block barrier per stage.
constexpr int SC_TM = 256;            // tokens per tile
constexpr int SC_KC = 16;             // pooled columns per stage
constexpr int SC_ZLD = SC_KC + 4;     // row stride of a stage buffer, in floats

template <int EPT>
__global__ void __launch_bounds__(256, 2)
affinity_score_tile_kernel(const float* __restrict__ Z, const float* __restrict__ xnorm,
                           const float* __restrict__ R, float* __restrict__ delta,
                           float* __restrict__ rnorm, etr_stats* stats, int Ttok, int D, int E, int m,
                           int ldm) {
  extern __shared__ __align__(16) float smem[];
  constexpr int EROWS = 8 * EPT;
  float* Rs = smem;                               // [EROWS][ldm]
  float* rn = Rs + (size_t)EROWS * ldm;           // [EROWS]
  float* Zs = rn + EROWS;                         // [2][SC_TM][SC_ZLD]
  __shared__ uint32_t red[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int eg = lane & 7, tg = lane >> 3;

  for (int idx = tid; idx < EROWS * ldm; idx += 256) {
    const int i = idx / ldm, j = idx - i * ldm;
    Rs[idx] = (i < E && j < m) ? R[(size_t)i * m + j] : 0.f;
  }
  __syncthreads();
  for (int i = warp; i < EROWS; i += 8) {
    float q = 0.f;
    for (int j = lane; j < m; j += 32) q += Rs[i * ldm + j] * Rs[i * ldm + j];
    q = warp_sum(q);
    if (lane == 0) {
      rn[i] = sqrtf(q);
      if (blockIdx.x == 0 && i < E) rnorm[i] = rn[i];
    }
  }
  // (the first stage barrier below also orders rn before its first use)

  const int ntiles = (Ttok + SC_TM - 1) / SC_TM, nk = m / SC_KC;
  auto fetch = [&](int tile, int chunk, int buf) {
    float* dst0 = Zs + (size_t)buf * SC_TM * SC_ZLD;
#pragma unroll
    for (int q = 0; q < SC_TM * (SC_KC / 4) / 256; ++q) {
      const int idx = tid + 256 * q, row = idx / (SC_KC / 4), c4 = idx % (SC_KC / 4);
      const int t = tile * SC_TM + row;
      float* dst = dst0 + row * SC_ZLD + c4 * 4;
      if (t < Ttok) {
        const uint32_t sa = (uint32_t)__cvta_generic_to_shared(dst);
        const float* src = Z + (size_t)t * m + chunk * SC_KC + c4 * 4;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(src) : "memory");
      } else {
        *reinterpret_cast<float4*>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  const float sqD = sqrtf((float)D);
  const int rs4 = ldm / 4;
  const float4* r4 = reinterpret_cast<const float4*>(Rs) + (size_t)eg * rs4;
  float best = -INFINITY;
  int stage = 0;
  if ((int)blockIdx.x < ntiles) fetch(blockIdx.x, 0, 0);
  for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    float acc[8][EPT];
#pragma unroll
    for (int u = 0; u < 8; ++u)
#pragma unroll
      for (int e = 0; e < EPT; ++e) acc[u][e] = 0.f;
    for (int chunk = 0; chunk < nk; ++chunk, ++stage) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();             // this stage has landed; everyone is done with the other buffer
      if (chunk + 1 < nk) fetch(tile, chunk + 1, (stage + 1) & 1);
      else if (tile + (int)gridDim.x < ntiles) fetch(tile + gridDim.x, 0, (stage + 1) & 1);
      const float4* z4 = reinterpret_cast<const float4*>(Zs + (size_t)(stage & 1) * SC_TM * SC_ZLD) +
                         (size_t)(warp * 32 + tg) * (SC_ZLD / 4);
      const float4* rc = r4 + chunk * (SC_KC / 4);
#pragma unroll 1
      for (int j = 0; j < SC_KC / 4; ++j) {
        float4 r[EPT];
#pragma unroll
        for (int e = 0; e < EPT; ++e) r[e] = rc[(size_t)(8 * e) * rs4 + j];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float4 z = z4[(size_t)(4 * u) * (SC_ZLD / 4) + j];
#pragma unroll
          for (int e = 0; e < EPT; ++e) {
            acc[u][e] = fmaf(z.x, r[e].x, acc[u][e]); acc[u][e] = fmaf(z.y, r[e].y, acc[u][e]);
            acc[u][e] = fmaf(z.z, r[e].z, acc[u][e]); acc[u][e] = fmaf(z.w, r[e].w, acc[u][e]);
          }
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int t = tile * SC_TM + warp * 32 + 4 * u + tg;
      if (t >= Ttok) continue;
      const float a = xnorm[t];
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        const int i = 8 * e + eg;
        if (i < E) {
          const float den = a * rn[i];
          const float v = den == 0.f ? 0.f : sqD * acc[u][e] / den;
          delta[(size_t)t * E + i] = v;
          best = fmaxf(best, v);
        }
      }
    }
  }
  uint32_t key = best == -INFINITY ? 0u : ordered_key(best);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
  if (lane == 0) red[warp] = key;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < 8; ++w) key = max(key, red[w]);
    if (key) atomicMax(&stats->delta_max_key, key);
  }
}

// ---- forward, warp-autonomous persistent form (the default) ------------------------------------
// R stays in shared memory for the life of the CTA; every warp owns a private slice for the
// pooled rows of TPG tokens and loops on its own: pool TPG tokens (16-byte loads, one pass
// over X), then s = z R^T with lane = expert (EPL experts per lane, TPG x EPL accumulators,
// float4 operands: R rows conflict-free, z rows broadcast), then coalesced stores of delta.
// No block-wide barrier after set-up, so the loads of some warps overlap the FMAs of others.
template <class T, int EPL, int TPG>
__global__ void __launch_bounds__(512, 1)
affinity_fwd_warp_kernel(const T* __restrict__ X, const float* __restrict__ R,
                         float* __restrict__ delta, float* __restrict__ Z, float* __restrict__ xnorm,
                         float* __restrict__ rnorm, etr_stats* stats, int Ttok, int d, int D, int E,
                         int m, int ldm) {
  extern __shared__ __align__(16) float smem[];
  constexpr int EROWS = 32 * EPL;
  const int nw = blockDim.x >> 5;
  float* Rs = smem;                               // [EROWS][ldm]
  float* rn = Rs + (size_t)EROWS * ldm;           // [EROWS]
  float* Zall = rn + EROWS;                       // [nw][TPG][ldm]
  __shared__ uint32_t red[16];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (int idx = tid; idx < EROWS * ldm; idx += blockDim.x) {
    const int i = idx / ldm, j = idx - i * ldm;
    Rs[idx] = (i < E && j < m) ? R[(size_t)i * m + j] : 0.f;
  }
  float* zs = Zall + (size_t)warp * TPG * ldm;
  for (int idx = lane; idx < TPG * ldm; idx += 32) zs[idx] = 0.f;
  __syncthreads();
  for (int i = warp; i < EROWS; i += nw) {
    float s = 0.f;
    for (int j = lane; j < m; j += 32) s += Rs[i * ldm + j] * Rs[i * ldm + j];
    s = warp_sum(s);
    if (lane == 0) {
      rn[i] = sqrtf(s);
      if (blockIdx.x == 0 && i < E) rnorm[i] = rn[i];
    }
  }
  __syncthreads();

  const float sqD = sqrtf((float)D);
  const int mr4 = (m + 3) / 4, rs4 = ldm / 4;
  const int ngroups = (Ttok + TPG - 1) / TPG;
  float best = -INFINITY;
  for (int g = blockIdx.x * nw + warp; g < ngroups; g += gridDim.x * nw) {
    const int t0 = g * TPG;
    // pooling, one token at a time (its loads are batched inside); ||x_t|| is parked in the
    // last pad column of the token's slice row, which the product below never reads
#pragma unroll 1
    for (int u = 0; u < TPG; ++u) {
      const int t = t0 + u;
      float part = 0.f;
      if (t < Ttok) {
        part = pool_token_partial<T>(X + (size_t)t * d, zs + (size_t)u * ldm, d, D, m, lane);
      } else {
        for (int j = lane; j < m; j += 32) zs[(size_t)u * ldm + j] = 0.f;
      }
      part = warp_sum(part);
      if (lane == 0) zs[(size_t)u * ldm + ldm - 1] = sqrtf(part);
    }
    __syncwarp();
    if (Z != nullptr) {
#pragma unroll
      for (int u = 0; u < TPG; ++u)
        if (t0 + u < Ttok)
          for (int j = lane; j < m; j += 32) Z[(size_t)(t0 + u) * m + j] = zs[(size_t)u * ldm + j];
    }
    float acc[TPG][EPL];
#pragma unroll
    for (int u = 0; u < TPG; ++u)
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[u][e] = 0.f;
    const float4* r4 = reinterpret_cast<const float4*>(Rs) + (size_t)lane * rs4;
    const float4* z4 = reinterpret_cast<const float4*>(zs);
#pragma unroll 2
    for (int j = 0; j < mr4; ++j) {
      float4 r[EPL];
#pragma unroll
      for (int e = 0; e < EPL; ++e) r[e] = r4[(size_t)(32 * e) * rs4 + j];
#pragma unroll
      for (int u = 0; u < TPG; ++u) {
        const float4 z = z4[(size_t)u * rs4 + j];
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          acc[u][e] = fmaf(z.x, r[e].x, acc[u][e]); acc[u][e] = fmaf(z.y, r[e].y, acc[u][e]);
          acc[u][e] = fmaf(z.z, r[e].z, acc[u][e]); acc[u][e] = fmaf(z.w, r[e].w, acc[u][e]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < TPG; ++u) {
      const int t = t0 + u;
      if (t >= Ttok) continue;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int i = lane + 32 * e;
        if (i < E) {
          const float den = zs[(size_t)u * ldm + ldm - 1] * rn[i];
          const float v = den == 0.f ? 0.f : sqD * acc[u][e] / den;
          delta[(size_t)t * E + i] = v;
          best = fmaxf(best, v);
        }
      }
      if (lane == 0) xnorm[t] = zs[(size_t)u * ldm + ldm - 1];
    }
    __syncwarp();        // the slice is rewritten by the next group's pooling
  }
  uint32_t key = best == -INFINITY ? 0u : ordered_key(best);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
  if (lane == 0) red[warp] = key;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < nw; ++w) key = max(key, red[w]);
    if (key) atomicMax(&stats->delta_max_key, key);
  }
}

// ---- forward, tiled form (fallback for shapes whose R does not fit next to the warp slices) ----
template <class T>
__global__ void __launch_bounds__(AFF_THREADS)
affinity_fwd_kernel(const T* __restrict__ X, const float* __restrict__ R, float* __restrict__ delta,
                    float* __restrict__ Z, float* __restrict__ xnorm, float* __restrict__ rnorm,
                    etr_stats* stats, int Ttok, int d, int D, int E, int m, int ldm, int Epad) {
  extern __shared__ __align__(16) float smem[];
  float* Rs = smem;                          // [Epad][ldm]
  float* Zs = Rs + (size_t)Epad * ldm;       // [TB][ldm]
  float* xn = Zs + (size_t)AFF_TB * ldm;     // [TB]
  float* rn = xn + AFF_TB;                   // [Epad]
  __shared__ uint32_t red[AFF_THREADS / 32];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t0 = blockIdx.x * AFF_TB;

  // phase 0
  for (int idx = tid; idx < Epad * ldm; idx += AFF_THREADS) {
    const int i = idx / ldm, j = idx - i * ldm;
    Rs[idx] = (i < E && j < m) ? R[(size_t)i * m + j] : 0.f;
  }
  for (int idx = tid; idx < AFF_TB * ldm; idx += AFF_THREADS) Zs[idx] = 0.f;
  __syncthreads();
  for (int i = warp; i < Epad; i += AFF_THREADS / 32) {
    float s = 0.f;
    for (int j = lane; j < m; j += 32) s += Rs[i * ldm + j] * Rs[i * ldm + j];
    s = warp_sum(s);
    if (lane == 0) {
      rn[i] = sqrtf(s);
      if (blockIdx.x == 0 && i < E) rnorm[i] = rn[i];
    }
  }

  // phase 1
  for (int tt = warp; tt < AFF_TB; tt += AFF_THREADS / 32) {
    const int t = t0 + tt;
    if (t < Ttok) {
      float sq;
      pool_token<T>(X + (size_t)t * d, Zs + (size_t)tt * ldm, d, D, m, lane, sq);
      if (lane == 0) { xn[tt] = sqrtf(sq); xnorm[t] = xn[tt]; }
    } else if (lane == 0) {
      xn[tt] = 0.f;
    }
  }
  __syncthreads();
  if (Z != nullptr) {
    for (int idx = tid; idx < AFF_TB * m; idx += AFF_THREADS) {
      const int tt = idx / m, j = idx - tt * m;
      if (t0 + tt < Ttok) Z[(size_t)(t0 + tt) * m + j] = Zs[tt * ldm + j];
    }
  }

  // phase 2
  const int nq = Epad / 4;
  const float sqD = sqrtf((float)D);
  const int mr4 = (m + 3) / 4;
  float best = -INFINITY;
  for (int item = tid; item < nq * (AFF_TB / 2); item += AFF_THREADS) {
    const int q = item % nq, tp = item / nq;
    const float4* z0 = reinterpret_cast<const float4*>(Zs + (size_t)(2 * tp) * ldm);
    const float4* z1 = reinterpret_cast<const float4*>(Zs + (size_t)(2 * tp + 1) * ldm);
    const float4* r0 = reinterpret_cast<const float4*>(Rs + (size_t)(4 * q) * ldm);
    const int rs = ldm / 4;
    float acc[2][4] = {};
#pragma unroll 2
    for (int j = 0; j < mr4; ++j) {
      const float4 a = z0[j], b = z1[j];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float4 r = r0[e * rs + j];
        acc[0][e] = fmaf(a.x, r.x, acc[0][e]); acc[0][e] = fmaf(a.y, r.y, acc[0][e]);
        acc[0][e] = fmaf(a.z, r.z, acc[0][e]); acc[0][e] = fmaf(a.w, r.w, acc[0][e]);
        acc[1][e] = fmaf(b.x, r.x, acc[1][e]); acc[1][e] = fmaf(b.y, r.y, acc[1][e]);
        acc[1][e] = fmaf(b.z, r.z, acc[1][e]); acc[1][e] = fmaf(b.w, r.w, acc[1][e]);
      }
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int tt = 2 * tp + u, t = t0 + tt;
      if (t >= Ttok) continue;
      float out[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float den = xn[tt] * rn[4 * q + e];
        out[e] = den == 0.f ? 0.f : sqD * acc[u][e] / den;
        if (4 * q + e < E) best = fmaxf(best, out[e]);
      }
      float* dst = delta + (size_t)t * E + 4 * q;
      if ((E & 3) == 0) {
        *reinterpret_cast<float4*>(dst) = make_float4(out[0], out[1], out[2], out[3]);
      } else {
        for (int e = 0; e < 4; ++e) if (4 * q + e < E) dst[e] = out[e];
      }
    }
  }
  uint32_t key = best == -INFINITY ? 0u : ordered_key(best);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
  if (lane == 0) red[warp] = key;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < AFF_THREADS / 32; ++w) key = max(key, red[w]);
    if (key) atomicMax(&stats->delta_max_key, key);
  }
}

// ---- backward -----------------------------------------------------------------------------
// dX[t,:] += cz[q/D] - beta x[t,:]  with  cz = sum_r (dgate_r sqrt(D)/(a b_i D)) R_i,
// beta = sum_r dgate_r delta_ti / a^2 over the rows r of token t.  One warp per token.
// FUSED: dX is not read; the FFN path's gradient is gathered here from dXp (the backward of the
// token rearrangement, dX[t] = sum of the token's rows of dXp), so dX is written exactly once.
template <class T, bool FUSED, bool DENSE>
__global__ void __launch_bounds__(256)
affinity_bwd_dx_kernel(const T* __restrict__ X, const float* __restrict__ R,
                       const float* __restrict__ delta, const float* __restrict__ xnorm,
                       const float* __restrict__ rnorm, const int32_t* __restrict__ tok_ptr,
                       const int32_t* __restrict__ tok_row, const float* __restrict__ dgate,
                       const float* __restrict__ ddelta, const T* __restrict__ dXp, T* __restrict__ dX,
                       int Ttok, int d, int D, int E, int m, int C_stride) {
  extern __shared__ __align__(16) float smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* cz = smem + (size_t)warp * m;
  const int t = blockIdx.x * 8 + warp;
  if (t >= Ttok) return;
  const int beg = tok_ptr[t], end = tok_ptr[t + 1];
  const float a = xnorm[t];
  T* g = dX + (size_t)t * d;
  if (beg == end) {
    if (FUSED)
      for (int v = lane; v < d * (int)sizeof(T) / 16; v += 32) reinterpret_cast<uint4*>(g)[v] = make_uint4(0, 0, 0, 0);
    return;
  }
  if (!FUSED && a == 0.f) return;
  for (int j = lane; j < m; j += 32) cz[j] = 0.f;
  float beta = 0.f;
  const float sqD = sqrtf((float)D);
  if (DENSE && a != 0.f) {
    // dense d delta (softmax gate): every expert contributes, in ascending expert order
    for (int i = 0; i < E; ++i) {
      const float b = rnorm[i], dg = ddelta[(size_t)t * E + i];
      if (b == 0.f || dg == 0.f) continue;
      const float w = dg * sqD / (a * b) / (float)D;
      beta += dg * delta[(size_t)t * E + i];
      for (int j = lane; j < m; j += 32) cz[j] = fmaf(w, R[(size_t)i * m + j], cz[j]);
    }
    beta /= (a * a);
  } else if (!DENSE && a != 0.f) {
    for (int q = beg; q < end; ++q) {
      const int r = tok_row[q], i = r / C_stride;
      const float b = rnorm[i], dg = dgate[r];
      if (b == 0.f) continue;
      const float w = dg * sqD / (a * b) / (float)D;
      beta += dg * delta[(size_t)t * E + i];
      for (int j = lane; j < m; j += 32) cz[j] = fmaf(w, R[(size_t)i * m + j], cz[j]);
    }
    beta /= (a * a);
  }
  __syncwarp();
  const T* x = X + (size_t)t * d;
  for (int v = lane; v < d / 8; v += 32) {
    Vec8<T> xv = Vec8<T>::load(x + v * 8);
    float base[8];
    if (FUSED) {
#pragma unroll
      for (int e = 0; e < 8; ++e) base[e] = 0.f;
      for (int q = beg; q < end; ++q) {
        Vec8<T> rv = Vec8<T>::load(dXp + (size_t)tok_row[q] * d + v * 8);
#pragma unroll
        for (int e = 0; e < 8; ++e) base[e] += rv.v[e];
      }
    } else {
      Vec8<T> gv = Vec8<T>::load(g + v * 8);
#pragma unroll
      for (int e = 0; e < 8; ++e) base[e] = gv.v[e];
    }
    float out[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) out[e] = base[e] + (cz[(v * 8 + e) / D] - beta * xv.v[e]);
    Vec8<T>::store(g + v * 8, out);
  }
}

// The fused form for selected pairs (the default of the layer backward), by chunks of tokens.  A block
// takes `tpb` consecutive tokens: (1) all threads copy the chunk's row lists to shared memory together
// with the per-row scalars (expert, weight of R_i in cz, dgate, delta), so the dependent chain
// pointer -> row -> scalars is walked once per chunk and not once per token; (2) cz[tl][:] and
// beta[tl] of every routed token of the chunk go to shared memory, one thread per pooled column,
// rows in list order; (3) the streaming pass: every thread owns NV groups of 8 elements of a token,
// 1/NV of a row apart, loads x and the token's rows of dXp two rows at a time (no load waits for an
// index) and writes dX once.  Unrouted tokens get zeros without reading X.  Same arithmetic, in the
// same order, as affinity_bwd_dx_kernel<T, true, false>: the results are bit-identical.
constexpr int DXC_MAX_TOKENS = 16;
constexpr int DXC_ROWS = 512;          // row entries held in shared memory; later ones are read in place

// cz and beta of every routed token of a chunk (phase 2 of the chunked dX kernels), for the pooled
// columns j = tid, tid + 256, ...  The chunk's staged row entries are walked as ONE flat list, eight at
// a time: the eight R values a thread needs are requested together before any is used, so a chunk
// costs a few rounds of L2 latency instead of one per token and entry.  Within a token the entries
// are still added in list order (same sums, bit for bit, as a loop per token).  Entries beyond the
// staged ones (DXC_ROWS) are read in place.
__device__ __forceinline__ void dx_chunk_cz(float* __restrict__ cz, float* __restrict__ s_beta,
                                            const int* __restrict__ s_ptr, const int* __restrict__ s_exp,
                                            const float* __restrict__ s_w, const float* __restrict__ s_dg,
                                            const float* __restrict__ s_dl, const float* __restrict__ s_a,
                                            const float* __restrict__ R, const float* __restrict__ rnorm,
                                            const float* __restrict__ delta, const float* __restrict__ dgate,
                                            const int32_t* __restrict__ tok_row, int base, int staged_max,
                                            int nt, int m, int E, int C_stride, int t0, float sqD, int D,
                                            int tid) {
  for (int j = tid; j < m; j += 256) {
    int tl = 0;
    while (tl < nt && s_ptr[tl + 1] == s_ptr[tl]) ++tl;              // first routed token
    float acc = 0.f, beta = 0.f;
    const int total = s_ptr[nt] - base;
    const int staged = min(total, staged_max);
    for (int e0 = 0; e0 < staged; e0 += 8) {
      float rv[8];
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        const int e = e0 + b;
        const int i = e < staged ? s_exp[e] : -1;
        rv[b] = i >= 0 ? R[(size_t)i * m + j] : 0.f;
      }
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        const int e = e0 + b;
        if (e >= staged) break;
        while (s_ptr[tl + 1] - base <= e) {                          // the entry opens a later token: close this one
          const float a = s_a[tl];
          cz[(size_t)tl * m + j] = acc;
          if (j == 0) s_beta[tl] = a != 0.f ? beta / (a * a) : 0.f;
          acc = 0.f; beta = 0.f;
          ++tl;
          while (s_ptr[tl + 1] == s_ptr[tl]) ++tl;
        }
        if (s_exp[e] >= 0 && s_a[tl] != 0.f) {
          beta = fmaf(s_dg[e], s_dl[e], beta);
          acc = fmaf(s_w[e], rv[b], acc);
        }
      }
    }
    // entries that did not fit the staged lists, token by token
    while (tl < nt) {
      const int beg = max(s_ptr[tl] - base, staged), end = s_ptr[tl + 1] - base;
      const float a = s_a[tl];
      if (a != 0.f) {
        for (int q = beg; q < end; ++q) {
          const int r = tok_row[base + q];
          const int i = r / C_stride;
          const float b = rnorm[i];
          if (b == 0.f) continue;
          const float dg = dgate[r];
          beta = fmaf(dg, delta[(size_t)(t0 + tl) * E + i], beta);
          acc = fmaf(dg * sqD / (a * b) / (float)D, R[(size_t)i * m + j], acc);
        }
      }
      if (s_ptr[tl + 1] > s_ptr[tl]) {
        cz[(size_t)tl * m + j] = acc;
        if (j == 0) s_beta[tl] = a != 0.f ? beta / (a * a) : 0.f;
      }
      acc = 0.f; beta = 0.f;
      ++tl;
    }
  }
}



template <class T, int NV, bool GROUP8>
__global__ void __launch_bounds__(256, 4)
affinity_bwd_dx_chunk_kernel(const T* __restrict__ X, const float* __restrict__ R,
                             const float* __restrict__ delta, const float* __restrict__ xnorm,
                             const float* __restrict__ rnorm, const int32_t* __restrict__ tok_ptr,
                             const int32_t* __restrict__ tok_row, const float* __restrict__ dgate,
                             const T* __restrict__ dXp, T* __restrict__ dX,
                             int Ttok, int d, int D, int E, int m, int C_stride, int tpb, int d_shift) {
  extern __shared__ __align__(16) float cz[];      // [tpb][m]
  __shared__ int s_ptr[DXC_MAX_TOKENS + 1];
  __shared__ int s_row[DXC_ROWS];
  __shared__ int s_exp[DXC_ROWS];                  // expert of the entry, -1 if ||R_i|| = 0
  __shared__ float s_w[DXC_ROWS];
  __shared__ float s_dg[DXC_ROWS];
  __shared__ float s_dl[DXC_ROWS];
  __shared__ float s_a[DXC_MAX_TOKENS];
  __shared__ float s_beta[DXC_MAX_TOKENS];
  const int tid = threadIdx.x;
  const int t0 = blockIdx.x * tpb;
  const int nt = min(tpb, Ttok - t0);
  if (tid <= nt) s_ptr[tid] = tok_ptr[t0 + tid];
  if (tid < nt) s_a[tid] = xnorm[t0 + tid];
  __syncthreads();
  const int base = s_ptr[0];
  const int staged = min(s_ptr[nt] - base, DXC_ROWS);
  const float sqD = sqrtf((float)D);
  for (int e = tid; e < staged; e += 256) {
    const int r = tok_row[base + e];
    int tl = 0;
    while (s_ptr[tl + 1] - base <= e) ++tl;        // the entry's token (at most tpb steps)
    const int i = r / C_stride;
    const float a = s_a[tl], b = rnorm[i], dg = dgate[r];
    s_row[e] = r;
    s_exp[e] = b == 0.f ? -1 : i;
    s_dg[e] = dg;
    s_dl[e] = delta[(size_t)(t0 + tl) * E + i];
    s_w[e] = dg * sqD / (a * b) / (float)D;
  }
  __syncthreads();
  dx_chunk_cz(cz, s_beta, s_ptr, s_exp, s_w, s_dg, s_dl, s_a, R, rnorm, delta, dgate, tok_row, base,
              DXC_ROWS, nt, m, E, C_stride, t0, sqD, D, tid);
  __syncthreads();
  const int vpt = d / 8 / NV;                      // threads per token
  for (int wi = tid; wi < nt * vpt; wi += 256) {
    const int tl = wi / vpt, v = wi - tl * vpt;
    const int beg = s_ptr[tl] - base, end = s_ptr[tl + 1] - base;
    T* g = dX + (size_t)(t0 + tl) * d;
    float bs[NV][8];
#pragma unroll
    for (int u = 0; u < NV; ++u)
#pragma unroll
      for (int e = 0; e < 8; ++e) bs[u][e] = 0.f;
    if (beg == end) {
#pragma unroll
      for (int u = 0; u < NV; ++u) Vec8<T>::store(g + (size_t)(v + u * vpt) * 8, bs[u]);
      continue;
    }
    const T* x = X + (size_t)(t0 + tl) * d;
    Vec8<T> xv[NV];
#pragma unroll
    for (int u = 0; u < NV; ++u) xv[u] = Vec8<T>::load(x + (size_t)(v + u * vpt) * 8);
    int q = beg;
    for (; q + 2 <= end; q += 2) {
      const int r0 = q < DXC_ROWS ? s_row[q] : tok_row[base + q];
      const int r1 = q + 1 < DXC_ROWS ? s_row[q + 1] : tok_row[base + q + 1];
      Vec8<T> v0[NV], v1[NV];
#pragma unroll
      for (int u = 0; u < NV; ++u) v0[u] = Vec8<T>::load(dXp + (size_t)r0 * d + (size_t)(v + u * vpt) * 8);
#pragma unroll
      for (int u = 0; u < NV; ++u) v1[u] = Vec8<T>::load(dXp + (size_t)r1 * d + (size_t)(v + u * vpt) * 8);
#pragma unroll
      for (int u = 0; u < NV; ++u)
#pragma unroll
        for (int e = 0; e < 8; ++e) bs[u][e] = (bs[u][e] + v0[u].v[e]) + v1[u].v[e];
    }
    if (q < end) {
      const int r = q < DXC_ROWS ? s_row[q] : tok_row[base + q];
      Vec8<T> v0[NV];
#pragma unroll
      for (int u = 0; u < NV; ++u) v0[u] = Vec8<T>::load(dXp + (size_t)r * d + (size_t)(v + u * vpt) * 8);
#pragma unroll
      for (int u = 0; u < NV; ++u)
#pragma unroll
        for (int e = 0; e < 8; ++e) bs[u][e] += v0[u].v[e];
    }
    const float beta = s_beta[tl];
    const float* czt = cz + (size_t)tl * m;
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      const int c0 = (v + u * vpt) * 8;
      float out[8];
      if (GROUP8) {                                // D = 2^d_shift >= 8: the 8 elements share one group
        const float czv = czt[c0 >> d_shift];
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = bs[u][e] + (czv - beta * xv[u].v[e]);
      } else {
        int gi = c0 / D, rem = c0 - gi * D;        // group of the first element, then stepped
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          out[e] = bs[u][e] + (czt[gi] - beta * xv[u].v[e]);
          if (++rem == D) { rem = 0; ++gi; }
        }
      }
      Vec8<T>::store(g + (size_t)c0, out);
    }
  }
}

// Partial dR over chunks of 128 slots of one expert (fixed order inside a chunk):
//   part[i][ch][j] = sum_p w_p Z[t_p][j], w_p = dgate_p sqrt(D)/(a_t b_i);
//   part[i][ch][m] = sum_p dgate_p delta_ti
constexpr int DR_CHUNK = 128;
constexpr int DR_MAXJ = 16;     // m <= 256 * DR_MAXJ
__global__ void __launch_bounds__(256)
affinity_bwd_dr_partial_kernel(const float* __restrict__ Z, const float* __restrict__ delta,
                               const float* __restrict__ xnorm, const float* __restrict__ rnorm,
                               const int32_t* __restrict__ counts,
                               const int32_t* __restrict__ slot_token,
                               const float* __restrict__ dgate, float* __restrict__ part,
                               int E, int m, int C_stride, int nch, float sqD) {
  __shared__ int s_t[DR_CHUNK];
  __shared__ float s_w[DR_CHUNK], s_dd[DR_CHUNK];
  const int i = blockIdx.x, ch = blockIdx.y, tid = threadIdx.x;
  const int n = counts[i];
  const int p0 = ch * DR_CHUNK;
  float* out = part + ((size_t)i * nch + ch) * (m + 1);
  const int np = min(DR_CHUNK, n - p0);
  if (np <= 0) {
    for (int j = tid; j <= m; j += 256) out[j] = 0.f;
    return;
  }
  const float b = rnorm[i];
  if (tid < np) {
    const size_t r = (size_t)i * C_stride + p0 + tid;
    const int t = slot_token[r];
    const float a = xnorm[t], dg = dgate[r];
    const bool dead = (a == 0.f || b == 0.f);
    s_t[tid] = t;
    s_w[tid] = dead ? 0.f : dg * sqD / (a * b);
    s_dd[tid] = dead ? 0.f : dg * delta[(size_t)t * E + i];
  }
  __syncthreads();
  float acc[DR_MAXJ];
#pragma unroll
  for (int u = 0; u < DR_MAXJ; ++u) acc[u] = 0.f;
  float sdd = 0.f;
  // slots in batches of 8: the gathered Z values of a batch are all requested before the first
  // is used; the accumulation order (ascending slot) is unchanged
  for (int p0 = 0; p0 < np; p0 += 8) {
#pragma unroll
    for (int u = 0; u < DR_MAXJ; ++u) {
      const int j = tid + u * 256;
      if (j >= m) break;
      float zv[8];
#pragma unroll
      for (int b = 0; b < 8; ++b) zv[b] = p0 + b < np ? Z[(size_t)s_t[p0 + b] * m + j] : 0.f;
#pragma unroll
      for (int b = 0; b < 8; ++b)
        if (p0 + b < np) acc[u] = fmaf(s_w[p0 + b], zv[b], acc[u]);
    }
#pragma unroll
    for (int b = 0; b < 8; ++b)
      if (p0 + b < np) sdd += s_dd[p0 + b];
  }
#pragma unroll
  for (int u = 0; u < DR_MAXJ; ++u) {
    const int j = tid + u * 256;
    if (j < m) out[j] = acc[u];
  }
  if (tid == 0) out[m] = sdd;
}

// The same partial sums for a dense d delta [T, E] (softmax gate): chunks of DR_DENSE_TOKENS
// consecutive tokens, every expert.  A block takes one chunk and 32 experts at a time: thread j keeps
// column j of the 32 partial rows, so each Z value is loaded once per 32 experts; tokens in ascending
// order (sub-chunks of 128 staged in shared memory).
constexpr int DR_DENSE_TOKENS = 256;
__global__ void __launch_bounds__(256)
affinity_bwd_dr_dense_partial_kernel(const float* __restrict__ Z, const float* __restrict__ delta,
                                     const float* __restrict__ xnorm, const float* __restrict__ rnorm,
                                     const float* __restrict__ ddelta, float* __restrict__ part,
                                     int Ttok, int E, int m, int nch, float sqD) {
  __shared__ __align__(16) float s_w[DR_CHUNK][32];
  __shared__ float s_dd[DR_CHUNK][32];
  const int ch = blockIdx.x, tid = threadIdx.x;
  const int t_beg = ch * DR_DENSE_TOKENS, t_end = min(Ttok, t_beg + DR_DENSE_TOKENS);
  for (int e0 = 0; e0 < E; e0 += 32) {
    for (int j0 = 0; j0 < m; j0 += 256) {
      const int j = j0 + tid;
      float acc[32];
#pragma unroll
      for (int ii = 0; ii < 32; ++ii) acc[ii] = 0.f;
      float sdd = 0.f;
      for (int t0 = t_beg; t0 < t_end; t0 += DR_CHUNK) {
        const int np = min(DR_CHUNK, t_end - t0);
        __syncthreads();
        for (int idx = tid; idx < DR_CHUNK * 32; idx += 256) {
          const int p = idx >> 5, i = e0 + (idx & 31);
          float w = 0.f, dd = 0.f;
          if (p < np && i < E) {
            const int t = t0 + p;
            const float a = xnorm[t], b = rnorm[i], dg = ddelta[(size_t)t * E + i];
            if (a != 0.f && b != 0.f) { w = dg * sqD / (a * b); dd = dg * delta[(size_t)t * E + i]; }
          }
          s_w[p][idx & 31] = w;
          s_dd[p][idx & 31] = dd;
        }
        __syncthreads();
        if (j < m) {
          for (int p = 0; p < np; ++p) {
            const float zv = Z[(size_t)(t0 + p) * m + j];
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4) {
              const float4 w = *reinterpret_cast<const float4*>(&s_w[p][4 * q4]);
              acc[4 * q4] = fmaf(w.x, zv, acc[4 * q4]);         acc[4 * q4 + 1] = fmaf(w.y, zv, acc[4 * q4 + 1]);
              acc[4 * q4 + 2] = fmaf(w.z, zv, acc[4 * q4 + 2]); acc[4 * q4 + 3] = fmaf(w.w, zv, acc[4 * q4 + 3]);
            }
          }
        }
        if (j0 == 0 && tid < 32)
          for (int p = 0; p < np; ++p) sdd += s_dd[p][tid];
      }
      if (j < m) {
#pragma unroll
        for (int ii = 0; ii < 32; ++ii)
          if (e0 + ii < E) part[((size_t)(e0 + ii) * nch + ch) * (m + 1) + j] = acc[ii];
      }
      if (j0 == 0 && tid < 32 && e0 + tid < E) part[((size_t)(e0 + tid) * nch + ch) * (m + 1) + m] = sdd;
    }
  }
}

// dR[i][j] = sum_ch part[i][ch][j] - (sum_ch part[i][ch][m]) R[i][j] / b_i^2, chunks in order.
__global__ void __launch_bounds__(256)
affinity_bwd_dr_final_kernel(const float* __restrict__ part, const float* __restrict__ R,
                             const float* __restrict__ rnorm, float* __restrict__ dR, int m, int nch) {
  const int i = blockIdx.x;
  const float b = rnorm[i];
  const float* base = part + (size_t)i * nch * (m + 1);
  float sdd = 0.f;
#pragma unroll 8
  for (int ch = 0; ch < nch; ++ch) sdd += base[(size_t)ch * (m + 1) + m];
  for (int j = threadIdx.x; j < m; j += 256) {
    float acc = 0.f;
#pragma unroll 8
    for (int ch = 0; ch < nch; ++ch) acc += base[(size_t)ch * (m + 1) + j];
    dR[(size_t)i * m + j] = b == 0.f ? 0.f : acc - sdd * R[(size_t)i * m + j] / (b * b);
  }
}

// ---- host side ---------------------------------------------------------------------------------
static size_t affinity_smem_bytes(int E, int m, int* ldm_out, int* Epad_out) {
  const int ldm = (m + 3) / 4 * 4 + 4, Epad = (E + 3) / 4 * 4;
  *ldm_out = ldm; *Epad_out = Epad;
  return ((size_t)(Epad + AFF_TB) * ldm + AFF_TB + Epad) * sizeof(float);
}

template <class T, int EPL, int TPG>
static etr_status launch_affinity_warp(const etr_config* c, const void* X, const float* R, float* delta,
                                       float* Z, float* xnorm, float* rnorm, etr_stats* stats,
                                       cudaStream_t st, bool* done) {
  const int m = c->d / c->D, ldm = (m + 3) / 4 * 4 + 4;
  *done = false;
  for (int nw = 16; nw >= 8; nw /= 2) {
    const size_t smem = ((size_t)(32 * EPL + nw * TPG) * ldm + 32 * EPL) * sizeof(float);
    if (smem > 220 * 1024) continue;
    auto k = affinity_fwd_warp_kernel<T, EPL, TPG>;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return ETR_ERR_CUDA;
    const int ngroups = ceil_div(c->T, TPG);
    const int grid = std::min(current_sm_count(), ceil_div(ngroups, nw));
    ETR_TIME_BEGIN("affinity_fwd_warp_kernel");
    k<<<grid, nw * 32, smem, st>>>((const T*)X, R, delta, Z, xnorm, rnorm, stats, c->T, c->d, c->D,
                                   c->E, m, ldm);
    ETR_LAUNCH_CHECK();
    *done = true;
    return ETR_OK;
  }
  return ETR_OK;
}

template <class T>
static etr_status affinity_forward_warp(const etr_config* c, const void* X, const float* R, float* delta,
                                        float* Z, float* xnorm, float* rnorm, etr_stats* stats,
                                        cudaStream_t st, bool* done) {
  if (c->E <= 32) return launch_affinity_warp<T, 1, 8>(c, X, R, delta, Z, xnorm, rnorm, stats, st, done);
  if (c->E <= 64) return launch_affinity_warp<T, 2, 8>(c, X, R, delta, Z, xnorm, rnorm, stats, st, done);
  if (c->E <= 128) return launch_affinity_warp<T, 4, 4>(c, X, R, delta, Z, xnorm, rnorm, stats, st, done);
  return launch_affinity_warp<T, 8, 2>(c, X, R, delta, Z, xnorm, rnorm, stats, st, done);
}

template <class T>
static etr_status launch_pool(const etr_config* c, const void* X, float* Z, float* xnorm, cudaStream_t st) {
  constexpr int PE = Raw16<T>::ELEMS;
  const int m = c->d / c->D, grid = ceil_div(c->T, 8), D = c->D;
  ETR_TIME_BEGIN("grap_pool_kernel");
  if (D == PE) grap_pool_kernel<T, 1><<<grid, 256, 0, st>>>((const T*)X, Z, xnorm, c->T, c->d, D, m);
  else if (D == 2 * PE) grap_pool_kernel<T, 2><<<grid, 256, 0, st>>>((const T*)X, Z, xnorm, c->T, c->d, D, m);
  else if (D == 4 * PE) grap_pool_kernel<T, 4><<<grid, 256, 0, st>>>((const T*)X, Z, xnorm, c->T, c->d, D, m);
  else grap_pool_kernel<T, 0><<<grid, 256, 0, st>>>((const T*)X, Z, xnorm, c->T, c->d, D, m);
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

template <int EPL, int TPG>
static etr_status launch_score(const etr_config* c, const float* Z, const float* xnorm, const float* R,
                               float* delta, float* rnorm, etr_stats* stats, cudaStream_t st, bool* done) {
  const int m = c->d / c->D, ldm = (m + 3) / 4 * 4 + 4;
  *done = false;
  for (int nw = 16; nw >= 4; nw /= 2) {
    const size_t smem = ((size_t)(32 * EPL + nw * TPG) * ldm + 32 * EPL) * sizeof(float);
    if (smem > 220 * 1024) continue;
    auto k = affinity_score_kernel<EPL, TPG>;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return ETR_ERR_CUDA;
    const int ngroups = ceil_div(c->T, TPG);
    const int grid = std::min(current_sm_count(), ceil_div(ngroups, nw));
    ETR_TIME_BEGIN("affinity_score_kernel");
    k<<<grid, nw * 32, smem, st>>>(Z, xnorm, R, delta, rnorm, stats, c->T, c->D, c->E, m, ldm);
    ETR_LAUNCH_CHECK();
    *done = true;
    return ETR_OK;
  }
  return ETR_OK;
}

// tiled score kernel: *done is false when the shape is not one it takes
template <int EPT>
static etr_status launch_score_tile(const etr_config* c, const float* Z, const float* xnorm, const float* R,
                                    float* delta, float* rnorm, etr_stats* stats, cudaStream_t st, bool* done) {
  const int m = c->d / c->D, ldm = m + 4;
  *done = false;
  const size_t smem = ((size_t)8 * EPT * ldm + 8 * EPT + (size_t)2 * SC_TM * SC_ZLD) * sizeof(float);
  if (smem > 110 * 1024) return ETR_OK;          // two blocks per SM
  auto k = affinity_score_tile_kernel<EPT>;
  if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return ETR_ERR_CUDA;
  const int grid = std::min(2 * current_sm_count(), ceil_div(c->T, SC_TM));
  ETR_TIME_BEGIN("affinity_score_kernel");
  k<<<grid, 256, smem, st>>>(Z, xnorm, R, delta, rnorm, stats, c->T, c->D, c->E, m, ldm);
  ETR_LAUNCH_CHECK();
  *done = true;
  return ETR_OK;
}

// pool + score as two kernels; *done is false if the score kernel's shared memory does not fit
static etr_status affinity_forward_split(const etr_config* c, const void* X, const float* R, float* delta,
                                         float* Z, float* xnorm, float* rnorm, etr_stats* stats,
                                         cudaStream_t st, bool* done) {
  const int m = c->d / c->D, ldm = (m + 3) / 4 * 4 + 4;
  const int EPL = c->E <= 32 ? 1 : c->E <= 64 ? 2 : c->E <= 128 ? 4 : 8;
  const int TPG = EPL <= 2 ? 8 : EPL == 4 ? 4 : 2;
  *done = false;
  if (((size_t)(32 * EPL + 4 * TPG) * ldm + 32 * EPL) * sizeof(float) > 220 * 1024) return ETR_OK;
  if (c->dtype == ETR_BF16) ETR_TRY(launch_pool<__nv_bfloat16>(c, X, Z, xnorm, st));
  else ETR_TRY(launch_pool<float>(c, X, Z, xnorm, st));
  // The product on the tensor cores wherever its shape rules hold, whatever the token count: a token's
  // affinities must not depend on how a batch is cut (an expert-parallel rank scores its own tokens).
  if (affinity_score_tc_takes(c, Z, R, delta)) {
    ETR_TRY(affinity_score_tc(c, Z, xnorm, R, delta, rnorm, stats, st));
    *done = true;
    return ETR_OK;
  }
  // the tiled form needs a tile of 256 tokens for every SM to pay for its set-up (R and its norms per block)
  if (c->E <= 64 && m % SC_KC == 0 && ceil_div(c->T, SC_TM) >= current_sm_count()) {
    if (c->E <= 16) ETR_TRY(launch_score_tile<2>(c, Z, xnorm, R, delta, rnorm, stats, st, done));
    else if (c->E <= 32) ETR_TRY(launch_score_tile<4>(c, Z, xnorm, R, delta, rnorm, stats, st, done));
    else ETR_TRY(launch_score_tile<8>(c, Z, xnorm, R, delta, rnorm, stats, st, done));
    if (*done) return ETR_OK;
  }
  if (EPL == 1) return launch_score<1, 8>(c, Z, xnorm, R, delta, rnorm, stats, st, done);
  if (EPL == 2) return launch_score<2, 8>(c, Z, xnorm, R, delta, rnorm, stats, st, done);
  if (EPL == 4) return launch_score<4, 4>(c, Z, xnorm, R, delta, rnorm, stats, st, done);
  return launch_score<8, 2>(c, Z, xnorm, R, delta, rnorm, stats, st, done);
}

etr_status affinity_forward(const etr_config* c, const void* X, const float* R, float* delta,
                            float* Z, float* xnorm, float* rnorm, etr_stats* stats,
                            cudaStream_t st) {
  const int m = c->d / c->D;
  bool done = false;
  if (Z != nullptr) {
    ETR_TRY(affinity_forward_split(c, X, R, delta, Z, xnorm, rnorm, stats, st, &done));
    if (done) return ETR_OK;
  }
  if (c->dtype == ETR_BF16)
    ETR_TRY(affinity_forward_warp<__nv_bfloat16>(c, X, R, delta, Z, xnorm, rnorm, stats, st, &done));
  else
    ETR_TRY(affinity_forward_warp<float>(c, X, R, delta, Z, xnorm, rnorm, stats, st, &done));
  if (done) return ETR_OK;
  int ldm, Epad;
  const size_t smem = affinity_smem_bytes(c->E, m, &ldm, &Epad);
  if (smem > 200 * 1024) return ETR_ERR_UNSUPPORTED;
  const int grid = ceil_div(c->T, AFF_TB);
  if (c->dtype == ETR_BF16) {
    auto k = affinity_fwd_kernel<__nv_bfloat16>;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return ETR_ERR_CUDA;
    ETR_TIME_BEGIN("affinity_fwd_kernel");
    k<<<grid, AFF_THREADS, smem, st>>>((const __nv_bfloat16*)X, R, delta, Z, xnorm, rnorm, stats,
                                       c->T, c->d, c->D, c->E, m, ldm, Epad);
  } else {
    auto k = affinity_fwd_kernel<float>;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return ETR_ERR_CUDA;
    ETR_TIME_BEGIN("affinity_fwd_kernel");
    k<<<grid, AFF_THREADS, smem, st>>>((const float*)X, R, delta, Z, xnorm, rnorm, stats, c->T,
                                       c->d, c->D, c->E, m, ldm, Epad);
  }
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

size_t affinity_bwd_workspace_bytes(const etr_config* c) {
  const int m = c->d / c->D;
  const int nch = c->gate_mode == ETR_GATE_SOFTMAX ? std::max(c_stride_of(c) / DR_CHUNK, ceil_div(c->T, DR_DENSE_TOKENS))
                                                   : c_stride_of(c) / DR_CHUNK;
  return (size_t)c->E * nch * (m + 1) * sizeof(float);
}

template <class T>
static etr_status launch_bwd_dx(const etr_config* c, const void* X, const float* R, const float* delta,
                                const float* xnorm, const float* rnorm, const etr_route* rt,
                                const float* dgate, const float* ddelta, const void* dXp_fused, void* dX,
                                etr_stats* stats, size_t smem, cudaStream_t st) {
  (void)stats;
  const int m = c->d / c->D, Cs = c_stride_of(c), grid = ceil_div(c->T, 8);
  auto launch = [&](auto k, const char* name) -> etr_status {
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return ETR_ERR_CUDA;
    ETR_TIME_BEGIN(name);
    k<<<grid, 256, smem, st>>>((const T*)X, R, delta, xnorm, rnorm, rt->tok_ptr, rt->tok_row, dgate, ddelta,
                               (const T*)dXp_fused, (T*)dX, c->T, c->d, c->D, c->E, m, Cs);
    return ETR_OK;
  };
  // chunked form of the fused kernel: as many tokens per block as keep cz within 48 KiB (at most 16)
  int tpb = DXC_MAX_TOKENS;
  while (tpb > 2 && (size_t)tpb * m * sizeof(float) > 48 * 1024) tpb /= 2;
  int d_shift = 0;
  while ((1 << d_shift) < c->D) ++d_shift;
  const bool group8 = c->D >= 8 && (1 << d_shift) == c->D;
  if (dXp_fused && !ddelta && (size_t)tpb * m * sizeof(float) <= 48 * 1024) {
    const size_t csm = (size_t)tpb * m * sizeof(float);
    ETR_TIME_BEGIN("affinity_bwd_dx_fused_kernel");
    auto go = [&](auto k) {
      k<<<ceil_div(c->T, tpb), 256, csm, st>>>((const T*)X, R, delta, xnorm, rnorm, rt->tok_ptr, rt->tok_row, dgate,
                                               (const T*)dXp_fused, (T*)dX, c->T, c->d, c->D, c->E, m, Cs, tpb,
                                               d_shift);
    };
    if (c->d % 16 == 0) {
      if (group8) go(affinity_bwd_dx_chunk_kernel<T, 2, true>);
      else go(affinity_bwd_dx_chunk_kernel<T, 2, false>);
    } else {
      if (group8) go(affinity_bwd_dx_chunk_kernel<T, 1, true>);
      else go(affinity_bwd_dx_chunk_kernel<T, 1, false>);
    }
  } else if (dXp_fused) {
    if (ddelta) ETR_TRY(launch(affinity_bwd_dx_kernel<T, true, true>, "affinity_bwd_dx_fused_kernel"));
    else ETR_TRY(launch(affinity_bwd_dx_kernel<T, true, false>, "affinity_bwd_dx_fused_kernel"));
  } else {
    if (ddelta) ETR_TRY(launch(affinity_bwd_dx_kernel<T, false, true>, "affinity_bwd_dx_kernel"));
    else ETR_TRY(launch(affinity_bwd_dx_kernel<T, false, false>, "affinity_bwd_dx_kernel"));
  }
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

// dXp_fused != nullptr: dX is produced here in one pass (dispatch backward + router gradient).
// ddelta != nullptr: the gradient of the affinities is that dense [T, E] matrix (softmax gate)
// instead of dgate on the selected pairs.
etr_status affinity_backward(const etr_config* c, const void* X, const float* R, const float* delta,
                             const float* Z, const float* xnorm, const float* rnorm,
                             const etr_route* rt, const float* dgate, const float* ddelta,
                             const void* dXp_fused, void* dX, float* dR, void* ws, etr_stats* stats,
                             cudaStream_t st) {
  const int m = c->d / c->D, Cs = c_stride_of(c);
  const int nch = ddelta ? ceil_div(c->T, DR_DENSE_TOKENS) : Cs / DR_CHUNK;
  if (m > 256 * DR_MAXJ) return ETR_ERR_UNSUPPORTED;
  const size_t smem = (size_t)8 * m * sizeof(float);
  if (smem > 200 * 1024) return ETR_ERR_UNSUPPORTED;
  ETR_TRY((c->dtype == ETR_BF16
               ? launch_bwd_dx<__nv_bfloat16>(c, X, R, delta, xnorm, rnorm, rt, dgate, ddelta, dXp_fused, dX, stats, smem, st)
               : launch_bwd_dx<float>(c, X, R, delta, xnorm, rnorm, rt, dgate, ddelta, dXp_fused, dX, stats, smem, st)));
  float* part = (float*)ws;
  if (ddelta) {
    ETR_TIME_BEGIN("affinity_bwd_dr_dense_partial_kernel");
    affinity_bwd_dr_dense_partial_kernel<<<nch, 256, 0, st>>>(Z, delta, xnorm, rnorm, ddelta, part, c->T, c->E,
                                                              m, nch, sqrtf((float)c->D));
  } else {
    ETR_TIME_BEGIN("affinity_bwd_dr_partial_kernel");
    affinity_bwd_dr_partial_kernel<<<dim3(c->E, nch), 256, 0, st>>>(
        Z, delta, xnorm, rnorm, rt->counts, rt->slot_token, dgate, part, c->E, m, Cs, nch,
        sqrtf((float)c->D));
  }
  ETR_LAUNCH_CHECK();
  ETR_TIME_BEGIN("affinity_bwd_dr_final_kernel");
  affinity_bwd_dr_final_kernel<<<c->E, 256, 0, st>>>(part, R, rnorm, dR, m, nch);
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

}  // namespace etr
