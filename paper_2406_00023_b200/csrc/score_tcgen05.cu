// Affinity scores on the tensor cores: delta[t][i] = sqrt(D) <z_t, R_i> / (||x_t|| ||R_i||) for a tile of
// 128 tokens x up to 64 experts per pass, the product <z_t, R_i> as a tcgen05 MMA of kind tf32.
//
// The router decides on these numbers, so they keep fp32 accuracy: every fp32 operand v is split in
// shared memory into hi = v with its low 13 mantissa bits cleared (exactly a tf32 value) and
// lo = (v - hi) cut the same way, and the product is accumulated as hi*hi + hi*lo + lo*hi in fp32
// accumulators in tensor memory.  The products of two tf32 values are exact in fp32; what is dropped is
// lo*lo (2^-22 of a product) and the second cut of lo (2^-24).  Both operand splits are made by a group
// of converter warps between the TMA load and the MMA, in place, so the caller's Z and R stay plain
// fp32 and no scratch memory is needed.
//
// Roles in a CTA of 320 threads: warp 0 lane 0 loads (TMA, 128-byte swizzle: a K block is 32 floats of
// every row), warps 2-5 split, warp 1 lane 0 issues the MMAs, warps 6-9 read the accumulators (two
// stages of four 64-column partial sums: all 512 columns), add them, scale by the norms, store delta
// through a staging tile (whole 128-byte rows) and track the batch maximum.  All waits are bounded; on
// expiry the kernel leaves 0x7c09 in etr_stats.error_word, frees its tensor memory and returns.
#include <algorithm>

#include "common.cuh"
#include "tcgen05_ptx.cuh"

namespace etr {

constexpr int SCT_BM = 128;                         // tokens per tile
constexpr int SCT_BK = 32;                          // floats per K block (one swizzle row)
constexpr int SCT_N = 64;                           // expert columns of the MMA (rows of R past E read as zeros)
constexpr int SCT_STAGES = 4;
constexpr int SCT_THREADS = 320;
constexpr uint32_t SCT_A_BYTES = SCT_BM * SCT_BK * 4;      // 16 KiB
constexpr uint32_t SCT_B_BYTES = SCT_N * SCT_BK * 4;       //  8 KiB
constexpr uint32_t SCT_STAGE_BYTES = 2 * SCT_A_BYTES + 2 * SCT_B_BYTES;      // hi and lo of both
constexpr int SCT_CHAINS = 4;                       // 64-column partial sums of a tile: two chains x {hi*hi + lo*hi, hi*lo}
constexpr uint32_t SCT_TMEM_COLS = 2 * SCT_CHAINS * SCT_N;      // two stages of them: 512 columns

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// v -> (hi, lo), both exactly tf32 values, v = hi + lo up to 2^-24 |v|
__device__ __forceinline__ void split_tf32(float v, float& hi, float& lo) {
  hi = __uint_as_float(__float_as_uint(v) & 0xffffe000u);
  lo = __uint_as_float(__float_as_uint(v - hi) & 0xffffe000u);
}
// The N 16-byte chunks per thread of a tile (chunk ct, ct + 128, ...: consecutive threads, consecutive chunks),
// split in place.  All loads are issued before the first store: the two tiles could alias as far as the
// compiler knows, and a load behind a store would wait for it.
template <int N>
__device__ __forceinline__ void split_chunks(uint8_t* hi_tile, uint8_t* lo_tile, int ct) {
  float4 v[N];
#pragma unroll
  for (int j = 0; j < N; ++j) v[j] = *reinterpret_cast<const float4*>(hi_tile + 16 * (ct + 128 * j));
#pragma unroll
  for (int j = 0; j < N; ++j) {
    float4 h, l;
    split_tf32(v[j].x, h.x, l.x); split_tf32(v[j].y, h.y, l.y); split_tf32(v[j].z, h.z, l.z); split_tf32(v[j].w, h.w, l.w);
    *reinterpret_cast<float4*>(hi_tile + 16 * (ct + 128 * j)) = h;
    *reinterpret_cast<float4*>(lo_tile + 16 * (ct + 128 * j)) = l;
  }
}

__global__ void __launch_bounds__(SCT_THREADS, 1)
affinity_score_tc_kernel(const __grid_constant__ CUtensorMap mapZ, const __grid_constant__ CUtensorMap mapR,
                         const float* __restrict__ R, const float* __restrict__ xnorm, float* __restrict__ delta,
                         float* __restrict__ rnorm, etr_stats* stats, int Ttok, int E, int m, float sqD,
                         uint32_t idesc, long long wait_limit) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[3 * SCT_STAGES + 4];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ float rn[SCT_N];

  volatile int* abort_flag = &abort_flag_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint8_t* tiles = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t tiles_base = smem_u32(tiles);
  const uint32_t full_bar = smem_u32(&bars[0]);                    // [STAGES] the TMA boxes have landed
  const uint32_t conv_bar = smem_u32(&bars[SCT_STAGES]);           // [STAGES] both operands are split
  const uint32_t empty_bar = smem_u32(&bars[2 * SCT_STAGES]);      // [STAGES] the MMAs have read the stage
  const uint32_t tfull_bar = smem_u32(&bars[3 * SCT_STAGES]);      // [2] accumulator complete
  const uint32_t tempty_bar = smem_u32(&bars[3 * SCT_STAGES + 2]); // [2] accumulator read out

  if (tid == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < SCT_STAGES; ++s) {
      mbar_init(full_bar + 8 * s, 1); mbar_init(conv_bar + 8 * s, 128); mbar_init(empty_bar + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar + 8 * a, 1); mbar_init(tempty_bar + 8 * a, 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(SCT_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const uint32_t idesc_wide = (idesc & ~(0x3fu << 17)) | ((uint32_t)(2 * SCT_N >> 3) << 17);      // N = 128
  const int ntiles = (Ttok + SCT_BM - 1) / SCT_BM, nkb = m / SCT_BK;

  if (warp == 0) {
    // ---- TMA producer --------------------------------------------------------------------------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, wait_limit)) { ok = false; break; }
          const uint32_t fb = full_bar + 8 * stage, sa = tiles_base + stage * SCT_STAGE_BYTES;
          mbar_expect_tx(fb, SCT_A_BYTES + SCT_B_BYTES);
          tma_load_2d(sa, &mapZ, fb, kb * SCT_BK, tile * SCT_BM);                 // tokens past T read as zeros
          tma_load_2d(sa + 2 * SCT_A_BYTES, &mapR, fb, kb * SCT_BK, 0);           // experts past E read as zeros
          if (++stage == SCT_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer ------------------------------------------------------------------------------------
    if (lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
        if (!mbar_wait(tempty_bar + 8 * acc, acc_phase ^ 1u, abort_flag, wait_limit)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * SCT_CHAINS * SCT_N);
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(conv_bar + 8 * stage, phase, abort_flag, wait_limit)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_hi = tiles_base + stage * SCT_STAGE_BYTES, a_lo = a_hi + SCT_A_BYTES;
          const uint32_t b_hi = a_hi + 2 * SCT_A_BYTES, b_lo = b_hi + SCT_B_BYTES;
          // 8 floats (32 bytes) per MMA, two MMAs per step: the hi and lo tiles of R lie one behind the other in
          // the stage, so A_hi x [R_hi; R_lo]^T is ONE MMA of 128 expert columns (hi*hi in columns 0-63 of the
          // chain, hi*lo in 64-127), and A_lo x R_hi^T adds lo*hi to columns 0-63.  These are small MMAs whose
          // issue costs about 75 cycles each whatever their width, and the issue lane is the longest stage.
          // Even and odd steps add into different chains (128 columns each), so that consecutive MMAs do not
          // wait for one another's result; the epilogue adds the four 64-column partial sums.
#pragma unroll
          for (int pairk = 0; pairk < SCT_BK / 8; pairk += 2) {
#pragma unroll
            for (int term = 0; term < 2; ++term) {
#pragma unroll
              for (int c = 0; c < 2; ++c) {
                const int kk = pairk + c;
                const uint64_t ad = make_smem_desc((term == 0 ? a_hi : a_lo) + 32 * kk, 16u, 1024u);
                const uint64_t bd = make_smem_desc(b_hi + 32 * kk, 16u, 1024u);
                tc_mma_tf32(d_tmem + (uint32_t)(c * 2 * SCT_N), ad, bd, term == 0 ? idesc_wide : idesc,
                            (kb > 0 || pairk > 0 || term > 0) ? 1u : 0u);
              }
            }
          }
          tc_commit(empty_bar + 8 * stage);
          if (++stage == SCT_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull_bar + 8 * acc);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else if (warp < 6) {
    // ---- converter warps: fp32 -> (hi, lo) in place ---------------------------------------------------
    const int ct = tid - 64;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
      for (int kb = 0; kb < nkb; ++kb) {
        if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag, wait_limit)) { ok = false; break; }
        uint8_t* st = tiles + (size_t)stage * SCT_STAGE_BYTES;
        split_chunks<SCT_A_BYTES / 16 / 128>(st, st + SCT_A_BYTES, ct);
        split_chunks<SCT_B_BYTES / 16 / 128>(st + 2 * SCT_A_BYTES, st + 2 * SCT_A_BYTES + SCT_B_BYTES, ct);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // generic writes -> the MMA's reads
        mbar_arrive(conv_bar + 8 * stage);
        if (++stage == SCT_STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else {
    // ---- epilogue warps: a lane owns a token --------------------------------------------------------------
    const int q = warp & 3;                      // tensor-memory lanes 32 q .. 32 q + 31
    float* stg = reinterpret_cast<float*>(tiles + (size_t)SCT_STAGES * SCT_STAGE_BYTES) + (warp - 6) * 32 * 33;
    // ||R_i|| while the first tile is on its way: a warp per row, lanes over the columns, the same sums
    // as the other score kernels (eight columns per lane requested together)
    for (int i = q; i < SCT_N; i += 4) {
      float acc_q = 0.f;
      if (i < E) {
        const float* row = R + (size_t)i * m;
        for (int j0 = lane; j0 < m; j0 += 256) {
          float v[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) v[u] = j0 + 32 * u < m ? row[j0 + 32 * u] : 0.f;
#pragma unroll
          for (int u = 0; u < 8; ++u) acc_q += v[u] * v[u];
        }
      }
      acc_q = warp_sum(acc_q);
      if (lane == 0) {
        rn[i] = sqrtf(acc_q);
        if (blockIdx.x == 0 && i < E) rnorm[i] = rn[i];
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");      // the four epilogue warps: rn is complete
    int acc = 0;
    uint32_t acc_phase = 0;
    float best = -INFINITY;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
      const int t = tile * SCT_BM + 32 * q + lane;
      const float xn = t < Ttok ? xnorm[t] : 0.f;
      if (!mbar_wait(tfull_bar + 8 * acc, acc_phase, abort_flag, wait_limit)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t)(acc * SCT_CHAINS * SCT_N) + ((uint32_t)(32 * q) << 16);
      uint32_t r[SCT_N];
      tc_ld32(taddr, r);
      tc_ld32(taddr + 32, r + 32);
      tc_wait_ld();
#pragma unroll
      for (int ch = 1; ch < SCT_CHAINS; ++ch) {      // the partial sums of the other accumulators, added in order
        uint32_t p[SCT_N];
        tc_ld32(taddr + ch * SCT_N, p);
        tc_ld32(taddr + ch * SCT_N + 32, p + 32);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < SCT_N; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(p[i]));
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar + 8 * acc);      // the values are in registers
      // scale: delta = sqrt(D) s / (||x|| ||R_i||), 0 where a norm is 0.  A fast division (reciprocal and product,
      // 2 ulp) taken unconditionally and selected afterwards: 64 correctly rounded divisions per token, each behind
      // its own zero test, overlapped with nothing and were the longest stage of the kernel; the result is
      // compared at 1e-5, not to the last bit.
#pragma unroll
      for (int i = 0; i < SCT_N; ++i) {
        const float den = xn * rn[i];
        const float quot = __fdividef(sqD * __uint_as_float(r[i]), den);
        const float v = den == 0.f ? 0.f : quot;
        r[i] = __float_as_uint(v);
        if (i < E && t < Ttok) best = fmaxf(best, v);
      }
      // store: a lane holds a token's row, but 32 lanes writing 32 different rows would send 16 bytes per
      // sector.  The warp turns 32 x 32 blocks through its staging tile (row stride 33 words: no bank
      // conflicts either way) and writes 128 contiguous bytes of one token per instruction.
      const int t_warp = tile * SCT_BM + 32 * q;
#pragma unroll
      for (int half = 0; half < SCT_N / 32; ++half) {
        if (32 * half < E) {
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 32; ++j) stg[lane * 33 + j] = __uint_as_float(r[32 * half + j]);
          __syncwarp();
          const int i = 32 * half + lane;
          const int nrow = min(32, Ttok - t_warp);
          for (int rr = 0; rr < nrow; ++rr)
            if (i < E) delta[(size_t)(t_warp + rr) * E + i] = stg[rr * 33 + lane];
        }
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    uint32_t key = best == -INFINITY ? 0u : ordered_key(best);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
    if (lane == 0 && key) atomicMax(&stats->delta_max_key, key);
  }

  // ---- teardown ---------------------------------------------------------------------------------------
  __syncwarp();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }      // copies still in flight land before the memory is released
    if (tid == 0) atomicExch(&stats->error_word, 0x7c09);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(SCT_TMEM_COLS) : "memory");
  }
}

// fp32 row-major matrix [rows, cols] as a 2-D map (cols, rows), boxes of 32 floats x box_rows, 128-byte swizzle
static etr_status make_map_f32(CUtensorMap* mp, const void* base, int cols, int rows, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return ETR_ERR_CUDA;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
  const cuuint32_t box[2] = {(cuuint32_t)SCT_BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(mp, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? ETR_OK : ETR_ERR_CUDA;
}

bool affinity_score_tc_takes(const etr_config* c, const float* Z, const float* R, const float* delta) {
  const int m = c->d / c->D;
  return c->E <= SCT_N && m % SCT_BK == 0 && aligned16(Z) && aligned16(R) && aligned16(delta);
}

etr_status affinity_score_tc(const etr_config* c, const float* Z, const float* xnorm, const float* R, float* delta,
                             float* rnorm, etr_stats* stats, cudaStream_t st) {
  const int m = c->d / c->D;
  CUtensorMap mapZ, mapR;
  ETR_TRY(make_map_f32(&mapZ, Z, m, c->T, SCT_BM));
  ETR_TRY(make_map_f32(&mapR, R, m, c->E, SCT_N));
  constexpr size_t smem = (size_t)SCT_STAGES * SCT_STAGE_BYTES + 1024 + 4 * 32 * 33 * sizeof(float);      // stages, alignment, staging
  static std::atomic<unsigned long long> attr_done{0};      // one bit per device
  if (!ensure_dyn_smem(affinity_score_tc_kernel, smem, attr_done)) return ETR_ERR_CUDA;
  uint32_t idesc = 0;
  idesc |= 1u << 4;                          // accumulator fp32
  idesc |= 2u << 7;                          // A tf32
  idesc |= 2u << 10;                         // B tf32
  idesc |= (uint32_t)(SCT_N >> 3) << 17;     // both operands K-major
  idesc |= (uint32_t)(SCT_BM >> 4) << 24;
  const int ntiles = ceil_div(c->T, SCT_BM);
  const long long limit = c->wait_limit_cycles > 0 ? (long long)c->wait_limit_cycles : ETR_WAIT_LIMIT_CYCLES;
  ETR_TIME_BEGIN("affinity_score_tc_kernel");
  affinity_score_tc_kernel<<<std::min(ntiles, current_sm_count()), SCT_THREADS, smem, st>>>(
      mapZ, mapR, R, xnorm, delta, rnorm, stats, c->T, c->E, m, sqrtf((float)c->D), idesc, limit);
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

}  // namespace etr
