// Grouped GEMMs of the expert FFN on the 5th-generation tensor cores (bf16 in, fp32
// accumulate in tensor memory).  One persistent, warp-specialised design serves all six
// contractions of the forward and backward pass, in three tile forms:
//
//   tc_grouped_gemm_kernel            one CTA per 128 x 256 tile (cta_group::1), 4-stage ring
//   tc_grouped_gemm_pair_kernel       a cluster of two CTAs per 256 x 256 tile (cta_group::2),
//                                     6-stage ring, two accumulator stages
//   tc_grouped_gemm_pair_wide_kernel  a cluster of two CTAs per 256 x 512 tile: two accumulators
//                                     share the A operand, 4-stage ring, halves released separately
//
//   warp 0      TMA producer: 64x64-element boxes (128-byte swizzle) into the ring
//   warp 1      allocates tensor memory, issues tcgen05.mma (the pair's leader CTA only)
//   warps 2-9   epilogue: tcgen05.ld of the fp32 accumulator, fused SwiGLU / its derivative,
//               bf16 stores (two warps per 32-lane quarter of tensor memory, half of the
//               columns each); it overlaps the next tile's MMAs
//
// Every operand is fetched as 64x64 boxes of its row-major tensor, so one tensor map per
// tensor serves both uses of it: "K-major" (the contraction index is contiguous in memory)
// and "MN-major" (the output index is contiguous: weight-gradient GEMMs, which contract over
// rows, and the data-gradient GEMMs, which read the weights transposed).  Only the
// shared-memory matrix descriptor differs.
//
// Tiles never straddle experts: the per-expert row count is read from `counts` on the
// device, and tiles are dealt round-robin to the CTAs of a persistent grid.  All waits on
// mbarriers are bounded; on expiry the kernel records a code in etr_stats.error_word,
// stops issuing work, releases its tensor memory and returns.
#include "common.cuh"
#include "tcgen05_ptx.cuh"

namespace etr {

constexpr int TC_BM = 128;
constexpr int TC_BK = 64;
constexpr int TC_STAGES = 4;
constexpr int TC_THREADS = 320;        // TMA warp, MMA warp, 8 epilogue warps
constexpr uint32_t TC_BOX_BYTES = 64 * 64 * 2;
constexpr long long TC_WAIT_LIMIT_CYCLES = ETR_WAIT_LIMIT_CYCLES;

enum { TC_EPI_STORE = 0, TC_EPI_SWIGLU = 1, TC_EPI_DSWIGLU = 2 };
enum { TC_DYN_M = 1, TC_DYN_K = 2 };

struct TcParams {
  int a_mn, b_mn;        // 1: operand is MN-major in memory
  int dual_b;            // SwiGLU: accumulator columns [0,128) from B0, [128,256) from B1
  int k1_blocks;         // > 0: K blocks [0,k1) use (A0,B0), the rest (A1,B1)
  int M, N, K;           // per-expert extents (DYN_M: M = C_stride cap; DYN_K: K unused)
  int dyn, E;
  const int32_t* counts;
  __nv_bfloat16* out0; __nv_bfloat16* out1; __nv_bfloat16* out2;
  const __nv_bfloat16* in0; const __nv_bfloat16* in1;
  long long out_bs;      // elements between experts in the outputs (and in0/in1)
  int ld_out;
  uint32_t idesc;
  etr_stats* stats;
  // Row gather (token rearrangement fused into the operand fetch): the rows of one operand are
  // rows of the token matrix X named by slot_token, fetched four at a time by TMA gather.
  // gather 1: the A operand's rows (row r of expert e is token slot_token[e*gather_ld + r]);
  // gather 2: the B operand's K rows (contractions over the expert's rows).  Slots holding -1 fetch
  // row gather_oob, which lies outside X and reads as zeros.  The gathered operand's map is mapA0
  // (gather 1) or mapB0 (gather 2), a 2-D map of X with a one-row box.
  int gather;
  int gather_ld, gather_oob;
  const int32_t* gather_idx;
  // Combine folded into the plain-store epilogue (Top-1 token choice: a token has at most one row, so
  // its output is that row times its gate and needs no sum): besides out0, row r of expert e also goes,
  // scaled, to row sc_tok[e*M + r] of sc_out (skipped where the slot holds -1).  sc_out == nullptr: off.
  const int32_t* sc_tok; const float* sc_gate; __nv_bfloat16* sc_out; int sc_ld;
  long long wait_limit;  // bound of every mbarrier wait, in SM clock cycles
  int out_f32;           // plain-store epilogue: out0 is fp32 (weight gradients with grad_fp32)
};

// ---- PTX wrappers (mbarrier helpers and the bounded wait: common.cuh) ---------------------------
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void load32(const __nv_bfloat16* src, float* v) {
  const uint4* p = reinterpret_cast<const uint4*>(src);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint4 w = p[q];
    const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[8 * q + 2 * i] = __uint_as_float(u[i] << 16);
      v[8 * q + 2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
  }
}

// last_kk: 16-wide MMA steps of the last K block that hold rows in use (contractions over an expert's
// rows: the steps beyond multiply pad rows, which are zero, and are skipped)
struct TileCoord { int e, m0, n0, kblocks, m_lim, last_kk; };

// Warp-cooperative store of a 32-row x 32-column bf16 block whose row `lane` is held by lane
// `lane` as 32 floats.  Written directly, every store instruction would touch 32 rows with 16
// bytes each (half a sector per row).  Instead the block is turned in a per-warp shared-memory
// scratch (32 rows x 80 bytes: the 16-byte pad makes both phases bank-conflict free) so that an
// instruction writes 8 rows x 64 contiguous bytes: whole sectors, half as many of them.
constexpr int TC_SCRATCH_ROW_BYTES = 80;
constexpr int TC_SCRATCH_BYTES = 32 * TC_SCRATCH_ROW_BYTES;      // per epilogue warp
__device__ __forceinline__ void store32_warp(uint8_t* scratch, int lane, int nvalid, __nv_bfloat16* dst,
                                             int ld_out, const float* v) {
  uint4* mine = reinterpret_cast<uint4*>(scratch + lane * TC_SCRATCH_ROW_BYTES);
#pragma unroll
  for (int q = 0; q < 4; ++q)
    mine[q] = make_uint4(pack_bf16(v[8 * q], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                         pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
  __syncwarp();
  const int sub = lane & 3;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = (lane >> 2) + 8 * i;
    const uint4 w = *reinterpret_cast<const uint4*>(scratch + row * TC_SCRATCH_ROW_BYTES + sub * 16);
    if (row < nvalid) *reinterpret_cast<uint4*>(dst + (long long)row * ld_out + sub * 8) = w;
  }
  __syncwarp();
}

// The same turn for 16 raw 32-bit words per lane (64 bytes of a row): a 32 x 32 block already packed
// to bf16, or half of a 32 x 32 block of fp32.  dst is the first row's address, rows ld_bytes apart.
__device__ __forceinline__ void store_rows64(uint8_t* scratch, int lane, int nvalid, char* dst,
                                             long long ld_bytes, const uint32_t* w16) {
  uint4* mine = reinterpret_cast<uint4*>(scratch + lane * TC_SCRATCH_ROW_BYTES);
#pragma unroll
  for (int q = 0; q < 4; ++q) mine[q] = make_uint4(w16[4 * q], w16[4 * q + 1], w16[4 * q + 2], w16[4 * q + 3]);
  __syncwarp();
  const int sub = lane & 3;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = (lane >> 2) + 8 * i;
    const uint4 w = *reinterpret_cast<const uint4*>(scratch + row * TC_SCRATCH_ROW_BYTES + sub * 16);
    if (row < nvalid) *reinterpret_cast<uint4*>(dst + row * ld_bytes + sub * 16) = w;
  }
  __syncwarp();
}
__device__ __forceinline__ void store32_warp_packed(uint8_t* scratch, int lane, int nvalid, __nv_bfloat16* dst,
                                                    int ld_out, const uint32_t* w16) {
  store_rows64(scratch, lane, nvalid, reinterpret_cast<char*>(dst), 2ll * ld_out, w16);
}
// A 32 x 32 block of fp32 accumulators (lane = row, 32 raw words) stored as fp32: two 64-byte halves.
__device__ __forceinline__ void store32_warp_f32(uint8_t* scratch, int lane, int nvalid, float* dst, int ld_out,
                                                 const uint32_t* r32) {
  store_rows64(scratch, lane, nvalid, reinterpret_cast<char*>(dst), 4ll * ld_out, r32);
  store_rows64(scratch, lane, nvalid, reinterpret_cast<char*>(dst) + 64, 4ll * ld_out, r32 + 16);
}
// The combine of a Top-1 layer in the epilogue: the 32 x 32 block just stored (packed bf16, w16 of this
// lane's row) scaled by the row's gate and written to the row of the token the slot holds.  The value
// is formed exactly as the separate kernels would: the stored bf16 output widened, times the gate in
// fp32, rounded to bf16.  Rows turn through the scratch like any store; the token of a row comes from
// the lane that owns it.
__device__ __forceinline__ void scatter32_warp(uint8_t* scratch, int lane, int tok, float gate,
                                               __nv_bfloat16* out, int ld, int col, const uint32_t* w16) {
  uint4* mine = reinterpret_cast<uint4*>(scratch + lane * TC_SCRATCH_ROW_BYTES);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint32_t y[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t w = w16[4 * q + i];
      y[i] = pack_bf16(gate * __uint_as_float(w << 16), gate * __uint_as_float(w & 0xffff0000u));
    }
    mine[q] = make_uint4(y[0], y[1], y[2], y[3]);
  }
  __syncwarp();
  const int sub = lane & 3;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = (lane >> 2) + 8 * i;
    const int t = __shfl_sync(0xffffffffu, tok, row);
    const uint4 w = *reinterpret_cast<const uint4*>(scratch + row * TC_SCRATCH_ROW_BYTES + sub * 16);
    if (t >= 0) *reinterpret_cast<uint4*>(out + (long long)t * ld + col + sub * 8) = w;
  }
  __syncwarp();
}
// 32 zeros at element offset `off` of the output (this lane's row of a block with nothing to contract).
__device__ __forceinline__ void store_zero32(const TcParams& p, long long off) {
  if (p.out_f32) {
    float4* q = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out0) + off);
#pragma unroll
    for (int i = 0; i < 8; ++i) q[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  } else {
    uint4* q = reinterpret_cast<uint4*>(p.out0 + off);
#pragma unroll
    for (int i = 0; i < 4; ++i) q[i] = make_uint4(0, 0, 0, 0);
  }
}

// The reverse turn for the saved activations the SwiGLU derivative reads: fetched as 8 rows x
// 64 contiguous bytes per instruction (regs `t`), later handed to the lane that owns the row.
__device__ __forceinline__ void load32_warp_issue(const __nv_bfloat16* src, int ld, int lane, int nvalid,
                                                  uint4 (&t)[4]) {
  const int sub = lane & 3;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = (lane >> 2) + 8 * i;
    t[i] = row < nvalid ? *reinterpret_cast<const uint4*>(src + (long long)row * ld + sub * 8)
                        : make_uint4(0, 0, 0, 0);
  }
}
__device__ __forceinline__ void load32_warp_turn(uint8_t* scratch, int lane, const uint4 (&t)[4],
                                                 uint4 (&mine)[4]) {
  const int sub = lane & 3;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    *reinterpret_cast<uint4*>(scratch + ((lane >> 2) + 8 * i) * TC_SCRATCH_ROW_BYTES + sub * 16) = t[i];
  __syncwarp();
#pragma unroll
  for (int q = 0; q < 4; ++q)
    mine[q] = *reinterpret_cast<const uint4*>(scratch + lane * TC_SCRATCH_ROW_BYTES + q * 16);
  __syncwarp();
}

// The epilogue of one accumulator tile for one warp: `nch` chunks of 32 columns starting at
// chunk c_beg, read from tensor memory at taddr and stored (or fused with SwiGLU / its
// derivative) at row offset obase.  pg/pu hold the prefetched G and U of the first chunk.
template <int EPI, int BN>
__device__ __forceinline__ void epilogue_chunks(const TcParams& p, int n0, uint32_t taddr, long long obase,
                                                bool row_ok, int c_beg, int nch, uint4 (&pg)[4],
                                                uint4 (&pu)[4], uint8_t* scratch, int lane, int nvalid,
                                                int sc_t = -1, float sc_g = 0.f) {
  const long long wbase = obase - (long long)lane * p.ld_out;     // row 0 of this warp's 32 rows
#pragma unroll 1
  for (int c = c_beg; c < c_beg + nch; ++c) {
    if (n0 + 32 * c >= p.N) break;
    __syncwarp();               // tcgen05.ld is warp-collective: reconverge after masked stores
    uint32_t r0[32];
    float v[32];
    tc_ld32(taddr + 32 * c, r0);
    if (EPI == TC_EPI_SWIGLU) {
      uint32_t r1[32];
      tc_ld32(taddr + BN / 2 + 32 * c, r1);
      tc_wait_ld();
      float hv[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float g = __uint_as_float(r0[i]), u = __uint_as_float(r1[i]);
        hv[i] = __fdividef(g, 1.0f + __expf(-g)) * u;
        v[i] = g;
      }
      store32_warp(scratch, lane, nvalid, p.out0 + wbase + 32 * c, p.ld_out, v);
      store32_warp(scratch, lane, nvalid, p.out2 + wbase + 32 * c, p.ld_out, hv);
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r1[i]);
      store32_warp(scratch, lane, nvalid, p.out1 + wbase + 32 * c, p.ld_out, v);
    } else if (EPI == TC_EPI_DSWIGLU) {
      uint4 cg[4], cu[4];
      load32_warp_turn(scratch, lane, pg, cg);
      load32_warp_turn(scratch, lane, pu, cu);
      if (c + 1 < c_beg + nch && n0 + 32 * (c + 1) < p.N) {
        load32_warp_issue(p.in0 + wbase + 32 * (c + 1), p.ld_out, lane, nvalid, pg);
        load32_warp_issue(p.in1 + wbase + 32 * (c + 1), p.ld_out, lane, nvalid, pu);
      }
      tc_wait_ld();
      {
        float dg[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const uint32_t wg = reinterpret_cast<const uint32_t*>(cg)[i >> 1];
          const uint32_t wu = reinterpret_cast<const uint32_t*>(cu)[i >> 1];
          const float g = (i & 1) ? __uint_as_float(wg & 0xffff0000u) : __uint_as_float(wg << 16);
          const float u = (i & 1) ? __uint_as_float(wu & 0xffff0000u) : __uint_as_float(wu << 16);
          const float dh = __uint_as_float(r0[i]);
          const float sgm = __fdividef(1.0f, 1.0f + __expf(-g));
          dg[i] = dh * u * sgm * (1.0f + g * (1.0f - sgm));
          v[i] = dh * g * sgm;
        }
        store32_warp(scratch, lane, nvalid, p.out0 + wbase + 32 * c, p.ld_out, dg);
        store32_warp(scratch, lane, nvalid, p.out1 + wbase + 32 * c, p.ld_out, v);
      }
    } else {
      tc_wait_ld();
      if (p.out_f32) {
        store32_warp_f32(scratch, lane, nvalid, reinterpret_cast<float*>(p.out0) + wbase + 32 * c, p.ld_out, r0);
      } else if (p.sc_out == nullptr) {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r0[i]);
        store32_warp(scratch, lane, nvalid, p.out0 + wbase + 32 * c, p.ld_out, v);
      } else {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(__uint_as_float(r0[2 * i]), __uint_as_float(r0[2 * i + 1]));
        store32_warp_packed(scratch, lane, nvalid, p.out0 + wbase + 32 * c, p.ld_out, pk);
        scatter32_warp(scratch, lane, sc_t, sc_g, p.sc_out, p.sc_ld, n0 + 32 * c, pk);
      }
    }
  }
}



// Tile index -> coordinates.  tile_prefix[e] = first tile of expert e.
__device__ __forceinline__ bool tile_coord(const TcParams& p, const int* tile_prefix, const int* counts_s,
    int tile, int& e_cur,
                                           int n_tile_cols, TileCoord& tc) {
  if (tile >= tile_prefix[p.E]) return false;
  while (tile >= tile_prefix[e_cur + 1]) ++e_cur;
  const int local = tile - tile_prefix[e_cur];
  const int n_e = counts_s[e_cur];
  int mt_count;
  if (p.dyn == TC_DYN_M) {
    mt_count = (min(n_e, p.M) + TC_BM - 1) / TC_BM;
    tc.kblocks = (p.K + TC_BK - 1) / TC_BK;
    tc.last_kk = TC_BK / 16;
    tc.m_lim = mt_count * TC_BM;
  } else {
    mt_count = (p.M + TC_BM - 1) / TC_BM;
    tc.kblocks = (n_e + TC_BK - 1) / TC_BK;
    tc.last_kk = n_e > 0 ? ((n_e - 1) % TC_BK) / 16 + 1 : TC_BK / 16;
    tc.m_lim = p.M;
  }
  tc.e = e_cur;
  tc.m0 = (local % mt_count) * TC_BM;
  tc.n0 = (local / mt_count) * n_tile_cols;
  (void)n_tile_cols;
  return true;
}

template <int BN, int EPI>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_grouped_gemm_kernel(const __grid_constant__ CUtensorMap mapA0, const __grid_constant__ CUtensorMap mapA1,
                       const __grid_constant__ CUtensorMap mapB0, const __grid_constant__ CUtensorMap mapB1,
                       const TcParams p) {
  constexpr int B_BOXES = BN / 64;
  constexpr uint32_t STAGE_BYTES = (2 + B_BOXES) * TC_BOX_BYTES;
  constexpr int N_TILE_COLS = (EPI == TC_EPI_SWIGLU) ? BN / 2 : BN;
  constexpr uint32_t TMEM_COLS = 512;

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * TC_STAGES + 4];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ int tile_prefix[257];
  __shared__ int s_counts[256];      // the experts' row counts, read from global memory once

  volatile int* abort_flag = &abort_flag_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t full_bar = smem_u32(&bars[0]);                   // [TC_STAGES]
  const uint32_t empty_bar = smem_u32(&bars[TC_STAGES]);          // [TC_STAGES]
  const uint32_t tfull_bar = smem_u32(&bars[2 * TC_STAGES]);      // [2]
  const uint32_t tempty_bar = smem_u32(&bars[2 * TC_STAGES + 2]); // [2]

  // ---- set-up ---------------------------------------------------------------------------------
  for (int e = tid; e < p.E; e += TC_THREADS) s_counts[e] = p.counts[e];
  __syncthreads();
  if (tid == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < TC_STAGES; ++s) { mbar_init(full_bar + 8 * s, 1); mbar_init(empty_bar + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar + 8 * a, 1); mbar_init(tempty_bar + 8 * a, 8); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const int nt = (p.N + N_TILE_COLS - 1) / N_TILE_COLS;
    int acc = 0;
    for (int e = 0; e < p.E; ++e) {
      tile_prefix[e] = acc;
      const int n_e = s_counts[e];
      const int mt = p.dyn == TC_DYN_M ? (min(n_e, p.M) + TC_BM - 1) / TC_BM : (p.M + TC_BM - 1) / TC_BM;
      acc += mt * nt;
    }
    tile_prefix[p.E] = acc;
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    // ---- TMA producer ---------------------------------------------------------------------------
    if (lane == 0) {
      int e_cur = 0, stage = 0;
      uint32_t phase = 0;
      TileCoord tc;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile_coord(p, tile_prefix, s_counts, tile, e_cur, N_TILE_COLS, tc); tile += gridDim.x) {
        for (int kb = 0; kb < tc.kblocks; ++kb) {
          if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
          const uint32_t fb = full_bar + 8 * stage;
          mbar_expect_tx(fb, STAGE_BYTES);
          const bool second = p.k1_blocks > 0 && kb >= p.k1_blocks;
          const int k0 = (second ? kb - p.k1_blocks : kb) * TC_BK;
          const CUtensorMap* ma = second ? &mapA1 : &mapA0;
          const uint32_t sa = tiles_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + 2 * TC_BOX_BYTES;
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            if (p.a_mn) tma_load_3d(sa + j * TC_BOX_BYTES, ma, fb, tc.m0 + 64 * j, k0, tc.e);
            else        tma_load_3d(sa + j * TC_BOX_BYTES, ma, fb, k0, tc.m0 + 64 * j, tc.e);
          }
#pragma unroll
          for (int j = 0; j < B_BOXES; ++j) {
            const CUtensorMap* mb = &mapB0;
            int nn = tc.n0 + 64 * j;
            if (p.dual_b) {
              if (j >= B_BOXES / 2) { mb = &mapB1; nn = tc.n0 + 64 * (j - B_BOXES / 2); }
            } else if (second) {
              mb = &mapB1;
            }
            if (p.b_mn) tma_load_3d(sb + j * TC_BOX_BYTES, mb, fb, nn, k0, tc.e);
            else        tma_load_3d(sb + j * TC_BOX_BYTES, mb, fb, k0, nn, tc.e);
          }
          if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer ------------------------------------------------------------------------------
    if (lane == 0) {
      int e_cur = 0, stage = 0, acc_stage = 0;
      uint32_t phase = 0, acc_phase = 0;
      TileCoord tc;
      bool ok = true;
      const uint32_t a_lbo = p.a_mn ? TC_BOX_BYTES : 16u, b_lbo = p.b_mn ? TC_BOX_BYTES : 16u;
      const uint32_t a_kstep = p.a_mn ? 2048u : 32u, b_kstep = p.b_mn ? 2048u : 32u;
      for (int tile = blockIdx.x; ok && tile_coord(p, tile_prefix, s_counts, tile, e_cur, N_TILE_COLS, tc); tile += gridDim.x) {
        if (tc.kblocks == 0) continue;
        if (!mbar_wait(tempty_bar + 8 * acc_stage, acc_phase ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc_stage * 256);
        for (int kb = 0; kb < tc.kblocks; ++kb) {
          if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.wait_limit)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = tiles_base + stage * STAGE_BYTES;
          const uint32_t sb = sa + 2 * TC_BOX_BYTES;
#pragma unroll
          for (int kk = 0; kk < TC_BK / 16; ++kk) {
            const uint64_t ad = make_smem_desc(sa + kk * a_kstep, a_lbo, 1024u);
            const uint64_t bd = make_smem_desc(sb + kk * b_kstep, b_lbo, 1024u);
            tc_mma(d_tmem, ad, bd, p.idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar + 8 * stage);          // frees the stage when these MMAs retire
          if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull_bar + 8 * acc_stage);        // accumulator complete
        if (++acc_stage == 2) { acc_stage = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---- epilogue warps ---------------------------------------------------------------------------
    const int q = warp & 3;                        // quarter of tensor memory this warp may read
    uint8_t* scratch = smem_raw + (tiles_base - smem_u32(smem_raw)) + TC_STAGES * STAGE_BYTES + (warp - 2) * TC_SCRATCH_BYTES;
    const int half = (warp - 2) >> 2;              // which half of the tile's columns it handles
    constexpr int NCH = N_TILE_COLS / 32 / 2;      // 32-column chunks per warp
    const int row_in_tile = 32 * q + lane;
    int e_cur = 0, acc_stage = 0;
    uint32_t acc_phase = 0;
    TileCoord tc;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile_coord(p, tile_prefix, s_counts, tile, e_cur, N_TILE_COLS, tc); tile += gridDim.x) {
      const int grow = tc.m0 + row_in_tile;
      const bool row_ok = grow < tc.m_lim;
      const int c_beg = half * NCH;
      const long long obase = (long long)tc.e * p.out_bs + (long long)grow * p.ld_out + tc.n0;
      if (tc.kblocks == 0) {        // nothing to contract: the block of the output is zero
        if (row_ok)
          for (int c = c_beg; c < c_beg + NCH && tc.n0 + 32 * c < p.N; ++c) store_zero32(p, obase + 32 * c);
        continue;
      }
      // SwiGLU derivative: the saved G and U of the first chunk are fetched before the
      // accumulator is ready, those of chunk c+1 while chunk c is processed
      uint4 pg[4], pu[4];
      const int nvalid = min(32, max(0, tc.m_lim - (grow - lane)));
      if (EPI == TC_EPI_DSWIGLU && tc.n0 + 32 * c_beg < p.N) {
        const long long wb = obase - (long long)lane * p.ld_out + 32 * c_beg;
        load32_warp_issue(p.in0 + wb, p.ld_out, lane, nvalid, pg);
        load32_warp_issue(p.in1 + wb, p.ld_out, lane, nvalid, pu);
      }
      if (!mbar_wait(tfull_bar + 8 * acc_stage, acc_phase, abort_flag, p.wait_limit)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t)(acc_stage * 256) + ((uint32_t)(32 * q) << 16);
      int sc_t = -1;
      float sc_g = 0.f;
      if (EPI == TC_EPI_STORE && p.sc_out != nullptr && row_ok && grow < p.M) {
        sc_t = p.sc_tok[(long long)tc.e * p.M + grow];
        sc_g = p.sc_gate[(long long)tc.e * p.M + grow];
      }
      epilogue_chunks<EPI, BN>(p, tc.n0, taddr, obase, row_ok, c_beg, NCH, pg, pu, scratch, lane, nvalid, sc_t, sc_g);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar + 8 * acc_stage);
      if (++acc_stage == 2) { acc_stage = 0; acc_phase ^= 1u; }
    }
  }

  // ---- teardown -----------------------------------------------------------------------------------
  __syncwarp();
  if (*abort_flag) {
    // give copies that are still in flight time to land before the CTA's memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }
    if (tid == 0) atomicExch(&p.stats->error_word, 0x7c05);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---- two-CTA form ---------------------------------------------------------------------------------
// The same pipeline on CTA pairs (thread-block cluster of 2, tcgen05 cta_group::2): one MMA covers
// 256 x 256 x 16, each CTA holding its own 128 rows of A, half of the B tile (128 of the 256
// columns) and the accumulator of its 128 rows.  Per CTA and K block only 32 KiB enter shared
// memory instead of 48 KiB, and the tensor core reads half of B from the peer, which takes
// pressure off the shared-memory port; six stages fit.  Only the leader CTA (cluster rank 0)
// issues MMAs.  Both CTAs' TMA loads complete on the leader's "full" barrier; the leader's
// commits are multicast to both CTAs' "empty" and "accumulator full" barriers; the epilogue
// warps of both CTAs arrive on the leader's "accumulator empty" barrier.  No load is multicast.
constexpr int TC2_STAGES = 6;
constexpr uint32_t TC2_STAGE_BYTES = 4 * TC_BOX_BYTES;       // per CTA: 2 boxes of A, 2 of B

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_count_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                  long long limit_cycles) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if ((it & 255u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit_cycles) { *abort_flag = 1; return false; }
    }
  }
}
// TMA load into this CTA's shared memory whose completion is counted on a barrier of the pair
// (cluster address); not a multicast.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster,
                                                 int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// Four rows of a 2-D tensor (one-row box of 64 columns), 4 x 128 bytes written consecutively.
__device__ __forceinline__ void tma_gather4_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster,
                                                 int col, int4 rows) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes.cta_group::2"
      " [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(col), "r"(rows.x), "r"(rows.y), "r"(rows.z), "r"(rows.w)
      : "memory");
}
// Token ids of four consecutive slots, -1 replaced by the out-of-range row.
__device__ __forceinline__ int4 gather_rows(const int32_t* idx, int oob) {
  int4 r = __ldg(reinterpret_cast<const int4*>(idx));
  r.x = r.x < 0 ? oob : r.x; r.y = r.y < 0 ? oob : r.y; r.z = r.z < 0 ? oob : r.z; r.w = r.w < 0 ? oob : r.w;
  return r;
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {      // arrives on `bar` in both CTAs
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// Pair-tile index -> coordinates (256 rows per pair tile).
__device__ __forceinline__ bool tile_coord_pair(const TcParams& p, const int* tile_prefix, const int* counts_s,
    int tile, int& e_cur,
                                                int n_tile_cols, TileCoord& tc) {
  if (tile >= tile_prefix[p.E]) return false;
  while (tile >= tile_prefix[e_cur + 1]) ++e_cur;
  const int local = tile - tile_prefix[e_cur];
  const int n_e = counts_s[e_cur];
  int mt_count;
  if (p.dyn == TC_DYN_M) {
    mt_count = (min(n_e, p.M) + 255) / 256;
    tc.kblocks = (p.K + TC_BK - 1) / TC_BK;
    tc.last_kk = TC_BK / 16;
    tc.m_lim = (min(n_e, p.M) + TC_BM - 1) / TC_BM * TC_BM;
  } else {
    mt_count = (p.M + 255) / 256;
    tc.kblocks = (n_e + TC_BK - 1) / TC_BK;
    tc.last_kk = n_e > 0 ? ((n_e - 1) % TC_BK) / 16 + 1 : TC_BK / 16;
    tc.m_lim = p.M;
  }
  tc.e = e_cur;
  tc.m0 = (local % mt_count) * 256;
  tc.n0 = (local / mt_count) * n_tile_cols;
  return true;
}

// GATHER is TcParams::gather, and CFG the operand modes (a_mn, b_mn, dual_b, two K ranges), as
// compile-time constants: the single-lane producer and MMA loops are on the kernel's critical path,
// and run-time branches cost there even when not taken (6-8 % of a GEMM for the operand modes,
// 10 % per gather branch).  CFG = -1 keeps the run-time forms for combinations without an
// instantiation of their own.
template <int EPI, int GATHER, int CFG>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_grouped_gemm_pair_kernel(const __grid_constant__ CUtensorMap mapA0, const __grid_constant__ CUtensorMap mapA1,
                            const __grid_constant__ CUtensorMap mapB0, const __grid_constant__ CUtensorMap mapB1,
                            const TcParams p) {
  constexpr int BN = 256;
  constexpr int N_TILE_COLS = (EPI == TC_EPI_SWIGLU) ? BN / 2 : BN;
  constexpr uint32_t TMEM_COLS = 512;
  // operand modes as compile-time constants when CFG >= 0 (bit 0 a_mn, 1 b_mn, 2 dual_b, 3 two K ranges)
  const bool A_MN = CFG < 0 ? p.a_mn != 0 : (CFG & 1) != 0, B_MN = CFG < 0 ? p.b_mn != 0 : (CFG & 2) != 0;
  const bool DUAL_B = CFG < 0 ? p.dual_b != 0 : (CFG & 4) != 0, TWO_K = CFG < 0 ? p.k1_blocks > 0 : (CFG & 8) != 0;

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * TC2_STAGES + 4];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ int tile_prefix[257];
  __shared__ int s_counts[256];      // the experts' row counts, read from global memory once

  volatile int* abort_flag = &abort_flag_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = (int)cluster_id_x(), npairs = (int)cluster_count_x();
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t full_bar = smem_u32(&bars[0]);                    // [TC2_STAGES]  used in the leader
  const uint32_t empty_bar = smem_u32(&bars[TC2_STAGES]);          // [TC2_STAGES]  in each CTA
  const uint32_t tfull_bar = smem_u32(&bars[2 * TC2_STAGES]);      // [2]           in each CTA
  const uint32_t tempty_bar = smem_u32(&bars[2 * TC2_STAGES + 2]); // [2]           used in the leader

  for (int e = tid; e < p.E; e += TC_THREADS) s_counts[e] = p.counts[e];
  __syncthreads();
  if (tid == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < TC2_STAGES; ++s) { mbar_init(full_bar + 8 * s, 1); mbar_init(empty_bar + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar + 8 * a, 1); mbar_init(tempty_bar + 8 * a, 16); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const int nt = (p.N + N_TILE_COLS - 1) / N_TILE_COLS;
    int acc = 0;
    for (int e = 0; e < p.E; ++e) {
      tile_prefix[e] = acc;
      const int n_e = s_counts[e];
      const int mt = p.dyn == TC_DYN_M ? (min(n_e, p.M) + 255) / 256 : (p.M + 255) / 256;
      acc += mt * nt;
    }
    tile_prefix[p.E] = acc;
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                 // both CTAs' barriers exist before any remote arrive
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const uint32_t leader_full = map_to_cta(full_bar, 0);
  const uint32_t leader_tempty = map_to_cta(tempty_bar, 0);

  if (warp == 0) {
    // ---- TMA producer (both CTAs) ---------------------------------------------------------------
    // Without a gather lane 0 works alone.  With one, the whole warp walks the loop: lane l
    // fetches rows 4l..4l+3 of the gathered operand's 128 (gather 1) or, for the two 64-column
    // boxes of a K block, rows 4(l%16)..+3 of box l/16 (gather 2); lane 0 issues the rest.
    if (lane == 0 || GATHER) {
      int e_cur = 0, stage = 0;
      uint32_t phase = 0;
      TileCoord tc;
      bool ok = true;
      for (int tile = pair; ok && tile_coord_pair(p, tile_prefix, s_counts, tile, e_cur, N_TILE_COLS, tc); tile += npairs) {
        const int m0c = tc.m0 + 128 * (int)rank;
        const int32_t* gidx = p.gather_idx + (size_t)tc.e * p.gather_ld;
        int4 rows_a = make_int4(0, 0, 0, 0), rows_b = make_int4(0, 0, 0, 0);
        if (GATHER == 1)      // a CTA's 128 rows lie inside the expert's C_stride slots or all past them
          rows_a = m0c < p.M ? gather_rows(gidx + m0c + 4 * lane, p.gather_oob)
                             : make_int4(p.gather_oob, p.gather_oob, p.gather_oob, p.gather_oob);
        if (GATHER == 2 && tc.kblocks > 0) rows_b = gather_rows(gidx + 4 * (lane & 15), p.gather_oob);
        for (int kb = 0; kb < tc.kblocks; ++kb) {
          int4 rows_next = rows_b;
          if (GATHER == 2 && kb + 1 < tc.kblocks)
            rows_next = gather_rows(gidx + (kb + 1) * TC_BK + 4 * (lane & 15), p.gather_oob);
          if (!mbar_wait_cluster(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
          if (rank == 0 && lane == 0) mbar_expect_tx(full_bar + 8 * stage, 2 * TC2_STAGE_BYTES);
          const uint32_t fb = leader_full + 8 * stage;
          const bool second = TWO_K && kb >= p.k1_blocks;
          const int k0 = (second ? kb - p.k1_blocks : kb) * TC_BK;
          const CUtensorMap* ma = second ? &mapA1 : &mapA0;
          const CUtensorMap* mb = DUAL_B ? (rank ? &mapB1 : &mapB0) : (second ? &mapB1 : &mapB0);
          const int nb = DUAL_B ? tc.n0 : tc.n0 + 128 * (int)rank;
          const uint32_t sa = tiles_base + stage * TC2_STAGE_BYTES;
          const uint32_t sb = sa + 2 * TC_BOX_BYTES;
          if (GATHER == 1) tma_gather4_pair(sa + 512u * lane, &mapA0, fb, k0, rows_a);
          if (GATHER == 2)
            tma_gather4_pair(sb + (lane >> 4) * TC_BOX_BYTES + 512u * (lane & 15), &mapB0, fb,
                             nb + 64 * (lane >> 4), rows_b);
          if (lane == 0) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              if (GATHER != 1) {
                if (A_MN) tma_load_3d_pair(sa + j * TC_BOX_BYTES, ma, fb, m0c + 64 * j, k0, tc.e);
                else        tma_load_3d_pair(sa + j * TC_BOX_BYTES, ma, fb, k0, m0c + 64 * j, tc.e);
              }
              if (GATHER != 2) {
                if (B_MN) tma_load_3d_pair(sb + j * TC_BOX_BYTES, mb, fb, nb + 64 * j, k0, tc.e);
                else        tma_load_3d_pair(sb + j * TC_BOX_BYTES, mb, fb, k0, nb + 64 * j, tc.e);
              }
            }
          }
          rows_b = rows_next;
          if (++stage == TC2_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer (leader CTA only) --------------------------------------------------------------
    if (lane == 0 && rank == 0) {
      int e_cur = 0, stage = 0, acc_stage = 0;
      uint32_t phase = 0, acc_phase = 0;
      TileCoord tc;
      bool ok = true;
      const uint32_t a_lbo = A_MN ? TC_BOX_BYTES : 16u, b_lbo = B_MN ? TC_BOX_BYTES : 16u;
      const uint32_t a_kstep = A_MN ? 2048u : 32u, b_kstep = B_MN ? 2048u : 32u;
      for (int tile = pair; ok && tile_coord_pair(p, tile_prefix, s_counts, tile, e_cur, N_TILE_COLS, tc); tile += npairs) {
        if (tc.kblocks == 0) continue;
        if (!mbar_wait_cluster(tempty_bar + 8 * acc_stage, acc_phase ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc_stage * 256);
        // A contraction over the expert's rows (operand modes 3, or the generic form) ends in a K block
        // whose last 16-wide steps may hold pad rows only: that block is peeled off the loop and runs
        // just the steps with rows in use (the skipped ones would add zeros).  The loop itself stays
        // free of the test: anything extra in it shows in the GEMM time.
        constexpr bool PEEL = CFG < 0 || CFG == 3;
        const int nloop = PEEL ? tc.kblocks - 1 : tc.kblocks;
        for (int kb = 0; kb < nloop; ++kb) {
          if (!mbar_wait_cluster(full_bar + 8 * stage, phase, abort_flag, p.wait_limit)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = tiles_base + stage * TC2_STAGE_BYTES;
          const uint32_t sb = sa + 2 * TC_BOX_BYTES;
#pragma unroll
          for (int kk = 0; kk < TC_BK / 16; ++kk) {
            const uint64_t ad = make_smem_desc(sa + kk * a_kstep, a_lbo, 1024u);
            const uint64_t bd = make_smem_desc(sb + kk * b_kstep, b_lbo, 1024u);
            tc_mma_pair(d_tmem, ad, bd, p.idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit_pair(empty_bar + 8 * stage);      // frees the stage in both CTAs
          if (++stage == TC2_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (PEEL && ok) {
          if (!mbar_wait_cluster(full_bar + 8 * stage, phase, abort_flag, p.wait_limit)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = tiles_base + stage * TC2_STAGE_BYTES;
          const uint32_t sb = sa + 2 * TC_BOX_BYTES;
#pragma unroll
          for (int kk = 0; kk < TC_BK / 16; ++kk) {
            if (kk < tc.last_kk) {
              const uint64_t ad = make_smem_desc(sa + kk * a_kstep, a_lbo, 1024u);
              const uint64_t bd = make_smem_desc(sb + kk * b_kstep, b_lbo, 1024u);
              tc_mma_pair(d_tmem, ad, bd, p.idesc, (nloop > 0 || kk > 0) ? 1u : 0u);
            }
          }
          tc_commit_pair(empty_bar + 8 * stage);
          if (++stage == TC2_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(tfull_bar + 8 * acc_stage);    // accumulators complete in both CTAs
        if (++acc_stage == 2) { acc_stage = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ---- epilogue warps (both CTAs, own 128 rows) -----------------------------------------------------
    const int q = warp & 3;
    uint8_t* scratch = smem_raw + (tiles_base - smem_u32(smem_raw)) + TC2_STAGES * TC2_STAGE_BYTES + (warp - 2) * TC_SCRATCH_BYTES;
    const int half = (warp - 2) >> 2;
    constexpr int NCH = N_TILE_COLS / 32 / 2;
    const int row_in_tile = 128 * (int)rank + 32 * q + lane;
    int e_cur = 0, acc_stage = 0;
    uint32_t acc_phase = 0;
    TileCoord tc;
    bool ok = true;
    for (int tile = pair; ok && tile_coord_pair(p, tile_prefix, s_counts, tile, e_cur, N_TILE_COLS, tc); tile += npairs) {
      const int grow = tc.m0 + row_in_tile;
      const bool row_ok = grow < tc.m_lim;
      const int c_beg = half * NCH;
      const long long obase = (long long)tc.e * p.out_bs + (long long)grow * p.ld_out + tc.n0;
      if (tc.kblocks == 0) {
        if (row_ok)
          for (int c = c_beg; c < c_beg + NCH && tc.n0 + 32 * c < p.N; ++c) store_zero32(p, obase + 32 * c);
        continue;
      }
      uint4 pg[4], pu[4];
      const int nvalid = min(32, max(0, tc.m_lim - (grow - lane)));
      if (EPI == TC_EPI_DSWIGLU && tc.n0 + 32 * c_beg < p.N) {
        const long long wb = obase - (long long)lane * p.ld_out + 32 * c_beg;
        load32_warp_issue(p.in0 + wb, p.ld_out, lane, nvalid, pg);
        load32_warp_issue(p.in1 + wb, p.ld_out, lane, nvalid, pu);
      }
      if (!mbar_wait_cluster(tfull_bar + 8 * acc_stage, acc_phase, abort_flag, p.wait_limit)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t)(acc_stage * 256) + ((uint32_t)(32 * q) << 16);
      int sc_t = -1;
      float sc_g = 0.f;
      if (EPI == TC_EPI_STORE && p.sc_out != nullptr && row_ok && grow < p.M) {
        sc_t = p.sc_tok[(long long)tc.e * p.M + grow];
        sc_g = p.sc_gate[(long long)tc.e * p.M + grow];
      }
      epilogue_chunks<EPI, BN>(p, tc.n0, taddr, obase, row_ok, c_beg, NCH, pg, pu, scratch, lane, nvalid, sc_t, sc_g);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * acc_stage);
      if (++acc_stage == 2) { acc_stage = 0; acc_phase ^= 1u; }
    }
  }

  // ---- teardown: neither CTA leaves while the other may still touch its barriers or memory -------
  __syncwarp();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }
    if (tid == 0) atomicExch(&p.stats->error_word, 0x7c06);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---- CTA-pair kernel, two output tiles per pass ------------------------------------------------------
// Same pair as above, but one pass covers 256 rows x 2 adjacent column tiles: the A boxes of a K
// block are fetched once and multiplied into two accumulators (tensor-memory columns [0,256) and
// [256,512)), so a K block moves 48 KiB per CTA for twice the flops of the 32 KiB above: a
// quarter less operand traffic from L2 per flop.  The price is that all of tensor memory is one
// tile's accumulator: the next tile's MMAs wait for the epilogue.  To hide most of that, the
// epilogue drains and releases the two halves separately, and the MMA warp runs the first K
// blocks of the next tile into half 0 alone (those stages stay held) until half 1 is free.
constexpr int TCW_STAGES = 4;
constexpr uint32_t TCW_STAGE_BYTES = 6 * TC_BOX_BYTES;       // per CTA: 2 boxes of A, 2 + 2 of B
constexpr int TCW_LEAD = TCW_STAGES - 1;                     // K blocks half 0 may run ahead of half 1

__device__ __forceinline__ bool tile_coord_wide(const TcParams& p, const int* tile_prefix, const int* counts_s,
    int tile, int& e_cur,
                                                int n_tile_cols, TileCoord& tc) {
  if (tile >= tile_prefix[p.E]) return false;
  while (tile >= tile_prefix[e_cur + 1]) ++e_cur;
  const int local = tile - tile_prefix[e_cur];
  const int n_e = counts_s[e_cur];
  int mt_count;
  if (p.dyn == TC_DYN_M) {
    mt_count = (min(n_e, p.M) + 255) / 256;
    tc.kblocks = (p.K + TC_BK - 1) / TC_BK;
    tc.last_kk = TC_BK / 16;
    tc.m_lim = (min(n_e, p.M) + TC_BM - 1) / TC_BM * TC_BM;
  } else {
    mt_count = (p.M + 255) / 256;
    tc.kblocks = (n_e + TC_BK - 1) / TC_BK;
    tc.last_kk = n_e > 0 ? ((n_e - 1) % TC_BK) / 16 + 1 : TC_BK / 16;
    tc.m_lim = p.M;
  }
  tc.e = e_cur;
  tc.m0 = (local % mt_count) * 256;
  tc.n0 = (local / mt_count) * 2 * n_tile_cols;
  return true;
}

template <int EPI, int GATHER, int CFG>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_grouped_gemm_pair_wide_kernel(const __grid_constant__ CUtensorMap mapA0, const __grid_constant__ CUtensorMap mapA1,
                                 const __grid_constant__ CUtensorMap mapB0, const __grid_constant__ CUtensorMap mapB1,
                                 const TcParams p) {
  constexpr int BN = 256;
  constexpr int N_TILE_COLS = (EPI == TC_EPI_SWIGLU) ? BN / 2 : BN;
  constexpr uint32_t TMEM_COLS = 512;
  // operand modes as compile-time constants when CFG >= 0 (bit 0 a_mn, 1 b_mn, 2 dual_b, 3 two K ranges)
  const bool A_MN = CFG < 0 ? p.a_mn != 0 : (CFG & 1) != 0, B_MN = CFG < 0 ? p.b_mn != 0 : (CFG & 2) != 0;
  const bool DUAL_B = CFG < 0 ? p.dual_b != 0 : (CFG & 4) != 0, TWO_K = CFG < 0 ? p.k1_blocks > 0 : (CFG & 8) != 0;

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * TCW_STAGES + 3];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ int tile_prefix[257];
  __shared__ int s_counts[256];      // the experts' row counts, read from global memory once

  volatile int* abort_flag = &abort_flag_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = (int)cluster_id_x(), npairs = (int)cluster_count_x();
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t full_bar = smem_u32(&bars[0]);                    // [TCW_STAGES]  used in the leader
  const uint32_t empty_bar = smem_u32(&bars[TCW_STAGES]);          // [TCW_STAGES]  in each CTA
  const uint32_t tfull_bar = smem_u32(&bars[2 * TCW_STAGES]);      // [1]           in each CTA
  const uint32_t tempty_bar = smem_u32(&bars[2 * TCW_STAGES + 1]); // [2]           used in the leader

  for (int e = tid; e < p.E; e += TC_THREADS) s_counts[e] = p.counts[e];
  __syncthreads();
  if (tid == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < TCW_STAGES; ++s) { mbar_init(full_bar + 8 * s, 1); mbar_init(empty_bar + 8 * s, 1); }
    mbar_init(tfull_bar, 1);
    for (int a = 0; a < 2; ++a) mbar_init(tempty_bar + 8 * a, 16);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const int nt = (p.N + 2 * N_TILE_COLS - 1) / (2 * N_TILE_COLS);
    int acc = 0;
    for (int e = 0; e < p.E; ++e) {
      tile_prefix[e] = acc;
      const int n_e = s_counts[e];
      const int mt = p.dyn == TC_DYN_M ? (min(n_e, p.M) + 255) / 256 : (p.M + 255) / 256;
      acc += mt * nt;
    }
    tile_prefix[p.E] = acc;
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                 // both CTAs' barriers exist before any remote arrive
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const uint32_t leader_full = map_to_cta(full_bar, 0);
  const uint32_t leader_tempty = map_to_cta(tempty_bar, 0);

  if (warp == 0) {
    // ---- TMA producer (both CTAs) ---------------------------------------------------------------
    // Lane 0 alone, or with a gathered A operand the whole warp (lane l fetches rows 4l..4l+3 of
    // the CTA's 128 rows of A; lane 0 also issues the B boxes).
    if (lane == 0 || GATHER) {
      int e_cur = 0, stage = 0;
      uint32_t phase = 0;
      TileCoord tc;
      bool ok = true;
      for (int tile = pair; ok && tile_coord_wide(p, tile_prefix, s_counts, tile, e_cur, N_TILE_COLS, tc); tile += npairs) {
        const int m0c = tc.m0 + 128 * (int)rank;
        const bool two = tc.n0 + N_TILE_COLS < p.N;
        int4 rows_a = make_int4(0, 0, 0, 0);
        if (GATHER == 1)
          rows_a = m0c < p.M ? gather_rows(p.gather_idx + (size_t)tc.e * p.gather_ld + m0c + 4 * lane, p.gather_oob)
                             : make_int4(p.gather_oob, p.gather_oob, p.gather_oob, p.gather_oob);
        for (int kb = 0; kb < tc.kblocks; ++kb) {
          if (!mbar_wait_cluster(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
          if (rank == 0 && lane == 0) mbar_expect_tx(full_bar + 8 * stage, 2 * (two ? 6 : 4) * TC_BOX_BYTES);
          const uint32_t fb = leader_full + 8 * stage;
          const bool second = TWO_K && kb >= p.k1_blocks;
          const int k0 = (second ? kb - p.k1_blocks : kb) * TC_BK;
          const CUtensorMap* ma = second ? &mapA1 : &mapA0;
          const CUtensorMap* mb = DUAL_B ? (rank ? &mapB1 : &mapB0) : (second ? &mapB1 : &mapB0);
          const uint32_t sa = tiles_base + stage * TCW_STAGE_BYTES;
          if (GATHER == 1) tma_gather4_pair(sa + 512u * lane, &mapA0, fb, k0, rows_a);
          if (lane == 0) {
            if (GATHER != 1) {
#pragma unroll
              for (int j = 0; j < 2; ++j) {
                if (A_MN) tma_load_3d_pair(sa + j * TC_BOX_BYTES, ma, fb, m0c + 64 * j, k0, tc.e);
                else        tma_load_3d_pair(sa + j * TC_BOX_BYTES, ma, fb, k0, m0c + 64 * j, tc.e);
              }
            }
            for (int hf = 0; hf < (two ? 2 : 1); ++hf) {
              const uint32_t sb = sa + (2 + 2 * hf) * TC_BOX_BYTES;
              const int nh = tc.n0 + hf * N_TILE_COLS;
              const int nb = DUAL_B ? nh : nh + 128 * (int)rank;
#pragma unroll
              for (int j = 0; j < 2; ++j) {
                if (B_MN) tma_load_3d_pair(sb + j * TC_BOX_BYTES, mb, fb, nb + 64 * j, k0, tc.e);
                else        tma_load_3d_pair(sb + j * TC_BOX_BYTES, mb, fb, k0, nb + 64 * j, tc.e);
              }
            }
          }
          if (++stage == TCW_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer (leader CTA only) --------------------------------------------------------------
    if (lane == 0 && rank == 0) {
      int e_cur = 0, stage = 0;
      uint32_t phase = 0, acc_phase = 0;
      TileCoord tc;
      bool ok = true;
      const uint32_t a_lbo = A_MN ? TC_BOX_BYTES : 16u, b_lbo = B_MN ? TC_BOX_BYTES : 16u;
      const uint32_t a_kstep = A_MN ? 2048u : 32u, b_kstep = B_MN ? 2048u : 32u;
      // one K block of one half: 4 MMAs of 256 x 256 x 16
      auto issue = [&](int st, int hf, bool first_block) {
        const uint32_t sa = tiles_base + st * TCW_STAGE_BYTES;
        const uint32_t sb = sa + (2 + 2 * hf) * TC_BOX_BYTES;
#pragma unroll
        for (int kk = 0; kk < TC_BK / 16; ++kk) {
          const uint64_t ad = make_smem_desc(sa + kk * a_kstep, a_lbo, 1024u);
          const uint64_t bd = make_smem_desc(sb + kk * b_kstep, b_lbo, 1024u);
          tc_mma_pair(tmem_base + (uint32_t)(hf * 256), ad, bd, p.idesc, (!first_block || kk > 0) ? 1u : 0u);
        }
      };
      for (int tile = pair; ok && tile_coord_wide(p, tile_prefix, s_counts, tile, e_cur, N_TILE_COLS, tc); tile += npairs) {
        if (tc.kblocks == 0) continue;
        const bool two = tc.n0 + N_TILE_COLS < p.N;
        if (!mbar_wait_cluster(tempty_bar, acc_phase ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
        tc_fence_after();
        // Lead-in: half 0 of the first K blocks while the epilogue still drains half 1.
        const int lead = two ? min(TCW_LEAD, tc.kblocks) : 0;
        int st = stage;
        uint32_t ph = phase;
        for (int kb = 0; kb < lead; ++kb) {
          if (!mbar_wait_cluster(full_bar + 8 * st, ph, abort_flag, p.wait_limit)) { ok = false; break; }
          tc_fence_after();
          issue(st, 0, kb == 0);
          if (++st == TCW_STAGES) { st = 0; ph ^= 1u; }
        }
        if (!ok) break;
        if (!mbar_wait_cluster(tempty_bar + 8, acc_phase ^ 1u, abort_flag, p.wait_limit)) { ok = false; break; }
        tc_fence_after();
        for (int kb = 0; kb < tc.kblocks; ++kb) {
          if (kb >= lead) {
            if (!mbar_wait_cluster(full_bar + 8 * stage, phase, abort_flag, p.wait_limit)) { ok = false; break; }
            tc_fence_after();
            issue(stage, 0, kb == 0);
          }
          if (two) issue(stage, 1, kb == 0);
          tc_commit_pair(empty_bar + 8 * stage);      // frees the stage in both CTAs
          if (++stage == TCW_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(tfull_bar);                    // both accumulators complete in both CTAs
        acc_phase ^= 1u;
      }
    }
  } else {
    // ---- epilogue warps (both CTAs, own 128 rows) -----------------------------------------------------
    const int q = warp & 3;
    uint8_t* scratch = smem_raw + (tiles_base - smem_u32(smem_raw)) + TCW_STAGES * TCW_STAGE_BYTES + (warp - 2) * TC_SCRATCH_BYTES;
    const int half = (warp - 2) >> 2;
    constexpr int NCH = N_TILE_COLS / 32 / 2;
    const int row_in_tile = 128 * (int)rank + 32 * q + lane;
    int e_cur = 0;
    uint32_t acc_phase = 0;
    TileCoord tc;
    bool ok = true;
    for (int tile = pair; ok && tile_coord_wide(p, tile_prefix, s_counts, tile, e_cur, N_TILE_COLS, tc); tile += npairs) {
      const int grow = tc.m0 + row_in_tile;
      const bool row_ok = grow < tc.m_lim;
      const int c_beg = half * NCH;
      const bool two = tc.n0 + N_TILE_COLS < p.N;
      const long long obase = (long long)tc.e * p.out_bs + (long long)grow * p.ld_out + tc.n0;
      if (tc.kblocks == 0) {
        if (row_ok)
          for (int hf = 0; hf < (two ? 2 : 1); ++hf)
            for (int c = c_beg; c < c_beg + NCH && tc.n0 + hf * N_TILE_COLS + 32 * c < p.N; ++c)
              store_zero32(p, obase + hf * N_TILE_COLS + 32 * c);
        continue;
      }
      uint4 pg[4], pu[4];
      const int nvalid = min(32, max(0, tc.m_lim - (grow - lane)));
      if (EPI == TC_EPI_DSWIGLU && tc.n0 + 32 * c_beg < p.N) {
        const long long wb = obase - (long long)lane * p.ld_out + 32 * c_beg;
        load32_warp_issue(p.in0 + wb, p.ld_out, lane, nvalid, pg);
        load32_warp_issue(p.in1 + wb, p.ld_out, lane, nvalid, pu);
      }
      int sc_t = -1;
      float sc_g = 0.f;
      if (EPI == TC_EPI_STORE && p.sc_out != nullptr && row_ok && grow < p.M) {
        sc_t = p.sc_tok[(long long)tc.e * p.M + grow];
        sc_g = p.sc_gate[(long long)tc.e * p.M + grow];
      }
      if (!mbar_wait_cluster(tfull_bar, acc_phase, abort_flag, p.wait_limit)) { ok = false; break; }
      tc_fence_after();
      if (EPI == TC_EPI_STORE && !p.out_f32) {
        // Plain stores: empty each half into registers (packed bf16) and release it at once;
        // the turn through the scratch and the global stores follow while the MMAs run on.
        static_assert(EPI != TC_EPI_STORE || NCH == 4, "four chunks of 32 columns per warp and half");
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t pk[NCH][16];
          const int n0h = tc.n0 + hf * N_TILE_COLS;
          const bool live = hf == 0 || two;
          if (live) {
            const uint32_t taddr = tmem_base + (uint32_t)(hf * 256) + ((uint32_t)(32 * q) << 16);
            uint32_t r[NCH][32];
#pragma unroll
            for (int c = 0; c < NCH; ++c) tc_ld32(taddr + 32 * (c_beg + c), r[c]);
            tc_wait_ld();
#pragma unroll
            for (int c = 0; c < NCH; ++c)
#pragma unroll
              for (int i = 0; i < 16; ++i)
                pk[c][i] = pack_bf16(__uint_as_float(r[c][2 * i]), __uint_as_float(r[c][2 * i + 1]));
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * hf);
          if (live) {
            const long long wb = obase - (long long)lane * p.ld_out + hf * N_TILE_COLS;
#pragma unroll
            for (int c = 0; c < NCH; ++c)
              if (n0h + 32 * (c_beg + c) < p.N)
              {
                store32_warp_packed(scratch, lane, nvalid, p.out0 + wb + 32 * (c_beg + c), p.ld_out, pk[c]);
                if (p.sc_out != nullptr)
                  scatter32_warp(scratch, lane, sc_t, sc_g, p.sc_out, p.sc_ld, n0h + 32 * (c_beg + c), pk[c]);
              }
          }
        }
      } else if (EPI == TC_EPI_SWIGLU) {
        // Fused SwiGLU: G and U of a half are read, H computed, and all three packed to bf16 in
        // registers before the half is released; the stores follow.
        static_assert(EPI != TC_EPI_SWIGLU || NCH == 2, "two chunks of 32 gate columns per warp and half");
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t pk[NCH][3][16];
          const int n0h = tc.n0 + hf * N_TILE_COLS;
          const bool live = hf == 0 || two;
          if (live) {
            const uint32_t taddr = tmem_base + (uint32_t)(hf * 256) + ((uint32_t)(32 * q) << 16);
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
              uint32_t r0[32], r1[32];
              tc_ld32(taddr + 32 * (c_beg + c), r0);
              tc_ld32(taddr + BN / 2 + 32 * (c_beg + c), r1);
              tc_wait_ld();
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const float g0 = __uint_as_float(r0[2 * i]), g1 = __uint_as_float(r0[2 * i + 1]);
                const float u0 = __uint_as_float(r1[2 * i]), u1 = __uint_as_float(r1[2 * i + 1]);
                pk[c][0][i] = pack_bf16(g0, g1);
                pk[c][1][i] = pack_bf16(u0, u1);
                pk[c][2][i] = pack_bf16(__fdividef(g0, 1.0f + __expf(-g0)) * u0, __fdividef(g1, 1.0f + __expf(-g1)) * u1);
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * hf);
          if (live) {
            const long long wb = obase - (long long)lane * p.ld_out + hf * N_TILE_COLS;
#pragma unroll
            for (int c = 0; c < NCH; ++c)
              if (n0h + 32 * (c_beg + c) < p.N) {
                store32_warp_packed(scratch, lane, nvalid, p.out0 + wb + 32 * (c_beg + c), p.ld_out, pk[c][0]);
                store32_warp_packed(scratch, lane, nvalid, p.out2 + wb + 32 * (c_beg + c), p.ld_out, pk[c][2]);
                store32_warp_packed(scratch, lane, nvalid, p.out1 + wb + 32 * (c_beg + c), p.ld_out, pk[c][1]);
              }
          }
        }
      } else {
        for (int hf = 0; hf < 2; ++hf) {
          if (hf == 0 || two) {
            const int n0h = tc.n0 + hf * N_TILE_COLS;
            const long long ob = obase + hf * N_TILE_COLS;
            if (EPI == TC_EPI_DSWIGLU && hf == 1 && n0h + 32 * c_beg < p.N) {
              const long long wb = ob - (long long)lane * p.ld_out + 32 * c_beg;
              load32_warp_issue(p.in0 + wb, p.ld_out, lane, nvalid, pg);
              load32_warp_issue(p.in1 + wb, p.ld_out, lane, nvalid, pu);
            }
            const uint32_t taddr = tmem_base + (uint32_t)(hf * 256) + ((uint32_t)(32 * q) << 16);
            epilogue_chunks<EPI, BN>(p, n0h, taddr, ob, row_ok, c_beg, NCH, pg, pu, scratch, lane, nvalid, sc_t, sc_g);
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * hf);
        }
      }
      acc_phase ^= 1u;
    }
  }

  // ---- teardown: neither CTA leaves while the other may still touch its barriers or memory -------
  __syncwarp();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }
    if (tid == 0) atomicExch(&p.stats->error_word, 0x7c07);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---- host side --------------------------------------------------------------------------------------
// Row-major bf16 tensor [E, rows, cols] as a 3-D map (cols, rows, E), 64x64 boxes, 128-byte swizzle.
static etr_status make_map(CUtensorMap* m, const void* base, int cols, int rows, int E) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return ETR_ERR_CUDA;
  const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)E};
  const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)cols * 2 * (cuuint64_t)rows};
  const cuuint32_t box[3] = {64, 64, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? ETR_OK : ETR_ERR_CUDA;
}

// Row-major bf16 token matrix [T, d] as a 2-D map (d, T) with a one-row box of 64 columns, for row
// gathers; rows at or past T read as zeros.
static etr_status make_gather_map(CUtensorMap* m, const void* base, int cols, int rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return ETR_ERR_CUDA;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {64, 1};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? ETR_OK : ETR_ERR_CUDA;
}

static uint32_t make_idesc(int a_mn, int b_mn, int n, int m_instr = TC_BM) {
  uint32_t d = 0;
  d |= 1u << 4;                     // accumulator fp32
  d |= 1u << 7;                     // A bf16
  d |= 1u << 10;                    // B bf16
  d |= (uint32_t)(a_mn ? 1 : 0) << 15;
  d |= (uint32_t)(b_mn ? 1 : 0) << 16;
  d |= (uint32_t)(n >> 3) << 17;
  d |= (uint32_t)(m_instr >> 4) << 24;
  return d;
}

static int sm_count() { return current_sm_count(); }

template <int BN, int EPI>
static etr_status tc_launch(const char* name, const CUtensorMap& a0, const CUtensorMap& a1,
                            const CUtensorMap& b0, const CUtensorMap& b1, TcParams p, int max_tiles,
                            cudaStream_t st) {
  constexpr size_t smem = (size_t)TC_STAGES * (2 + BN / 64) * TC_BOX_BYTES + 1024 + 8 * TC_SCRATCH_BYTES;
  auto k = tc_grouped_gemm_kernel<BN, EPI>;
  static std::atomic<unsigned long long> attr_done{0};      // one bit per device
  if (!ensure_dyn_smem(k, smem, attr_done)) return ETR_ERR_CUDA;
  p.idesc = make_idesc(p.a_mn, p.b_mn, BN);
  const int grid = max_tiles < sm_count() ? (max_tiles < 1 ? 1 : max_tiles) : sm_count();
  ETR_TIME_BEGIN(name);
  k<<<grid, TC_THREADS, smem, st>>>(a0, a1, b0, b1, p);
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

template <int EPI, int GATHER, int CFG>
static etr_status tc_launch_pair_cfg(const char* name, const CUtensorMap& a0, const CUtensorMap& a1,
                                 const CUtensorMap& b0, const CUtensorMap& b1, TcParams p, int max_tiles,
                                 cudaStream_t st) {
  constexpr size_t smem = (size_t)TC2_STAGES * TC2_STAGE_BYTES + 1024 + 8 * TC_SCRATCH_BYTES;
  auto k = tc_grouped_gemm_pair_kernel<EPI, GATHER, CFG>;
  static std::atomic<unsigned long long> attr_done{0};      // one bit per device
  if (!ensure_dyn_smem(k, smem, attr_done)) return ETR_ERR_CUDA;
  p.idesc = make_idesc(p.a_mn, p.b_mn, 256, 256);
  const int pairs_max = sm_count() / 2;
  const int pairs = max_tiles < pairs_max ? (max_tiles < 1 ? 1 : max_tiles) : pairs_max;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ETR_TIME_BEGIN(name);
  if (cudaLaunchKernelEx(&cfg, k, a0, a1, b0, b1, p) != cudaSuccess) { timing_end(st); return ETR_ERR_CUDA; }
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

template <int EPI, int GATHER, int CFG>
static etr_status tc_launch_pair_wide_cfg(const char* name, const CUtensorMap& a0, const CUtensorMap& a1,
                                      const CUtensorMap& b0, const CUtensorMap& b1, TcParams p, int max_tiles,
                                      cudaStream_t st) {
  constexpr size_t smem = (size_t)TCW_STAGES * TCW_STAGE_BYTES + 1024 + 8 * TC_SCRATCH_BYTES;
  auto k = tc_grouped_gemm_pair_wide_kernel<EPI, GATHER, CFG>;
  static std::atomic<unsigned long long> attr_done{0};      // one bit per device
  if (!ensure_dyn_smem(k, smem, attr_done)) return ETR_ERR_CUDA;
  p.idesc = make_idesc(p.a_mn, p.b_mn, 256, 256);
  const int pairs_max = sm_count() / 2;
  const int pairs = max_tiles < pairs_max ? (max_tiles < 1 ? 1 : max_tiles) : pairs_max;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ETR_TIME_BEGIN(name);
  if (cudaLaunchKernelEx(&cfg, k, a0, a1, b0, b1, p) != cudaSuccess) { timing_end(st); return ETR_ERR_CUDA; }
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}


// The operand modes each epilogue is used with get their own instantiation; anything else runs the
// generic one (CFG = -1).
template <int EPI, int GATHER>
static etr_status tc_launch_pair(const char* name, const CUtensorMap& a0, const CUtensorMap& a1,
                                 const CUtensorMap& b0, const CUtensorMap& b1, TcParams p, int max_tiles,
                                 cudaStream_t st) {
  const int cfg = (p.a_mn ? 1 : 0) | (p.b_mn ? 2 : 0) | (p.dual_b ? 4 : 0) | (p.k1_blocks > 0 ? 8 : 0);
  constexpr int C0 = EPI == TC_EPI_SWIGLU ? 4 : EPI == TC_EPI_DSWIGLU ? 2 : 0;      // first use
  constexpr int C1 = EPI == TC_EPI_STORE ? 3 : C0, C2 = EPI == TC_EPI_STORE ? 10 : C0;
  if (cfg == C0) return tc_launch_pair_cfg<EPI, GATHER, C0>(name, a0, a1, b0, b1, p, max_tiles, st);
  if (cfg == C1) return tc_launch_pair_cfg<EPI, GATHER, C1>(name, a0, a1, b0, b1, p, max_tiles, st);
  if (cfg == C2) return tc_launch_pair_cfg<EPI, GATHER, C2>(name, a0, a1, b0, b1, p, max_tiles, st);
  return tc_launch_pair_cfg<EPI, GATHER, -1>(name, a0, a1, b0, b1, p, max_tiles, st);
}
template <int EPI, int GATHER>
static etr_status tc_launch_pair_wide(const char* name, const CUtensorMap& a0, const CUtensorMap& a1,
                                      const CUtensorMap& b0, const CUtensorMap& b1, TcParams p, int max_tiles,
                                      cudaStream_t st) {
  const int cfg = (p.a_mn ? 1 : 0) | (p.b_mn ? 2 : 0) | (p.dual_b ? 4 : 0) | (p.k1_blocks > 0 ? 8 : 0);
  constexpr int C0 = EPI == TC_EPI_SWIGLU ? 4 : EPI == TC_EPI_DSWIGLU ? 2 : 0;
  constexpr int C2 = EPI == TC_EPI_STORE ? 10 : C0;
  if (cfg == C0) return tc_launch_pair_wide_cfg<EPI, GATHER, C0>(name, a0, a1, b0, b1, p, max_tiles, st);
  if (cfg == C2) return tc_launch_pair_wide_cfg<EPI, GATHER, C2>(name, a0, a1, b0, b1, p, max_tiles, st);
  return tc_launch_pair_wide_cfg<EPI, GATHER, -1>(name, a0, a1, b0, b1, p, max_tiles, st);
}

// The three forms of one contraction; max_tiles is an upper bound counted in 128-row tiles of one
// column tile (it only caps the grid for small problems).
enum TcForm { TC_FORM_SINGLE, TC_FORM_PAIR, TC_FORM_PAIR_WIDE };

// Which form runs one contraction.  A forced gemm_impl decides alone.  Otherwise (AUTO) the wide
// pair form is taken where its saving in operand traffic outweighs its exposed epilogue: plain
// stores whose row extent is the expert's token count (down, dXp), and the fused SwiGLU when the
// contraction is long (>= 48 K blocks); and only when the launch has at least four rounds of wide
// tiles per CTA pair at full capacity, since a wide tile is twice the unit of work (small layers
// fall back to the single-CTA form for those stores, see below).  Weight
// gradients (short contraction over the expert's rows, large outputs) and the SwiGLU derivative
// (its epilogue also fetches G and U) measured faster on 256 x 256 tiles.
static TcForm tc_form_of(const etr_config* c, int epi, const TcParams& p) {
  if (p.gather) {      // the pair kernels fetch gathered rows; wide only where it is chosen anyway
    if (c->gemm_impl == ETR_GEMM_TCGEN05_2CTA_WIDE && p.gather == 1) return TC_FORM_PAIR_WIDE;
    if (c->gemm_impl != ETR_GEMM_AUTO || p.gather == 2) return TC_FORM_PAIR;
  }
  if (c->gemm_impl == ETR_GEMM_TCGEN05) return TC_FORM_SINGLE;
  if (c->gemm_impl == ETR_GEMM_TCGEN05_2CTA) return TC_FORM_PAIR;
  if (c->gemm_impl == ETR_GEMM_TCGEN05_2CTA_WIDE) return TC_FORM_PAIR_WIDE;
  if (p.dyn != TC_DYN_M || epi == TC_EPI_DSWIGLU) return TC_FORM_PAIR;
  if (epi == TC_EPI_SWIGLU && ceil_div(p.K, TC_BK) < 48) return TC_FORM_PAIR;
  const int cols = epi == TC_EPI_SWIGLU ? 256 : 512;
  const long long rounds = 4ll * (sm_count() / 2);
  const long long wide_tiles = (long long)p.E * ceil_div(p.M, 256) * ceil_div(p.N, cols);
  if (wide_tiles >= rounds) return TC_FORM_PAIR_WIDE;
  // Few tiles (small layers): for the plain stores, 128-row tiles on single CTAs balance better and
  // pad the expert's rows to 128 instead of 256.
  const long long pair_tiles = (long long)p.E * ceil_div(p.M, 256) * ceil_div(p.N, 256);
  return (epi == TC_EPI_STORE && pair_tiles < rounds && !p.gather) ? TC_FORM_SINGLE : TC_FORM_PAIR;
}
template <int EPI>
static etr_status tc_run(TcForm form, const char* name, const CUtensorMap& a0, const CUtensorMap& a1,
                         const CUtensorMap& b0, const CUtensorMap& b1, const TcParams& p, int max_tiles,
                         cudaStream_t st) {
  // gathered operands exist for the SwiGLU GEMM (A rows) and the plain-store weight gradients (K rows)
  if (form == TC_FORM_PAIR_WIDE) {
    if (EPI == TC_EPI_SWIGLU && p.gather == 1)
      return tc_launch_pair_wide<EPI, EPI == TC_EPI_SWIGLU ? 1 : 0>(name, a0, a1, b0, b1, p, (max_tiles + 1) / 2, st);
    if (p.gather) return ETR_ERR_UNSUPPORTED;
    return tc_launch_pair_wide<EPI, 0>(name, a0, a1, b0, b1, p, (max_tiles + 1) / 2, st);
  }
  if (form == TC_FORM_PAIR) {
    if (EPI == TC_EPI_SWIGLU && p.gather == 1)
      return tc_launch_pair<EPI, EPI == TC_EPI_SWIGLU ? 1 : 0>(name, a0, a1, b0, b1, p, (max_tiles + 1) / 2, st);
    if (EPI == TC_EPI_STORE && p.gather == 2)
      return tc_launch_pair<EPI, EPI == TC_EPI_STORE ? 2 : 0>(name, a0, a1, b0, b1, p, (max_tiles + 1) / 2, st);
    if (p.gather) return ETR_ERR_UNSUPPORTED;
    return tc_launch_pair<EPI, 0>(name, a0, a1, b0, b1, p, (max_tiles + 1) / 2, st);
  }
  if (p.gather) return ETR_ERR_UNSUPPORTED;
  return tc_launch<256, EPI>(name, a0, a1, b0, b1, p, max_tiles, st);
}

static TcParams tc_params(const etr_config* c) {
  TcParams p = {};
  p.wait_limit = c->wait_limit_cycles > 0 ? (long long)c->wait_limit_cycles : TC_WAIT_LIMIT_CYCLES;
  return p;
}

size_t tc_workspace_bytes(const etr_config*) { return 0; }
bool tc_available() { return true; }

etr_status tc_ffn_forward(const etr_config* c, const etr_route* rt, const void* Xp, const void* Xtok, const void* W1g,
                          const void* W1u, const void* W2, void* G, void* U, void* H, void* O,
                          etr_stats* stats, void*, void* Y_top1, cudaStream_t st) {
  const int d = c->d, h = c->h, Cs = c_stride_of(c), E = c->E;
  CUtensorMap mXp, mW1g, mW1u, mW2, mH;
  if (Xtok) ETR_TRY(make_gather_map(&mXp, Xtok, d, c->T));
  else ETR_TRY(make_map(&mXp, Xp, d, Cs, E));
  ETR_TRY(make_map(&mW1g, W1g, d, h, E));
  ETR_TRY(make_map(&mW1u, W1u, d, h, E));
  ETR_TRY(make_map(&mW2, W2, h, d, E));
  ETR_TRY(make_map(&mH, H, h, Cs, E));
  const int mt = Cs / TC_BM;
  {  // G, U, H = SwiGLU(Xp W1g^T, Xp W1u^T)
    TcParams p = tc_params(c);
    if (Xtok) { p.gather = 1; p.gather_ld = Cs; p.gather_oob = c->T; p.gather_idx = rt->slot_token; }
    p.dual_b = 1; p.M = Cs; p.N = h; p.K = d; p.dyn = TC_DYN_M; p.E = E; p.counts = rt->counts;
    p.out0 = (__nv_bfloat16*)G; p.out1 = (__nv_bfloat16*)U; p.out2 = (__nv_bfloat16*)H;
    p.out_bs = (long long)Cs * h; p.ld_out = h; p.stats = stats;
    ETR_TRY((tc_run<TC_EPI_SWIGLU>(tc_form_of(c, TC_EPI_SWIGLU, p), "tc_gemm_swiglu", mXp, mXp, mW1g, mW1u, p,
                                           E * mt * ceil_div(h, 128), st)));
  }
  {  // O = H W2^T
    TcParams p = tc_params(c);
    p.M = Cs; p.N = d; p.K = h; p.dyn = TC_DYN_M; p.E = E; p.counts = rt->counts;
    p.out0 = (__nv_bfloat16*)O; p.out_bs = (long long)Cs * d; p.ld_out = d; p.stats = stats;
    if (Y_top1) {      // Top-1: the combine in this epilogue (the caller has zeroed the rows of unrouted tokens)
      p.sc_tok = rt->slot_token; p.sc_gate = rt->gate; p.sc_out = (__nv_bfloat16*)Y_top1; p.sc_ld = d;
    }
    ETR_TRY((tc_run<TC_EPI_STORE>(tc_form_of(c, TC_EPI_STORE, p), "tc_gemm_down", mH, mH, mW2, mW2, p, E * mt * ceil_div(d, 256), st)));
  }
  return ETR_OK;
}

etr_status tc_ffn_backward(const etr_config* c, const etr_route* rt, const void* dO, const void* Xp,
                           const void* Xtok, const void* G, const void* U, const void* H, const void* W1g,
                           const void* W1u, const void* W2, void* dG, void* dU, void* dXp, void* dW1g,
                           void* dW1u, void* dW2, etr_stats* stats, void*, cudaStream_t st) {
  const int d = c->d, h = c->h, Cs = c_stride_of(c), E = c->E;
  CUtensorMap mdO, mXp, mH, mdG, mdU, mW1g, mW1u, mW2;
  ETR_TRY(make_map(&mdO, dO, d, Cs, E));
  if (Xtok) ETR_TRY(make_gather_map(&mXp, Xtok, d, c->T));
  else ETR_TRY(make_map(&mXp, Xp, d, Cs, E));
  ETR_TRY(make_map(&mH, H, h, Cs, E));
  ETR_TRY(make_map(&mdG, dG, h, Cs, E));
  ETR_TRY(make_map(&mdU, dU, h, Cs, E));
  ETR_TRY(make_map(&mW1g, W1g, d, h, E));
  ETR_TRY(make_map(&mW1u, W1u, d, h, E));
  ETR_TRY(make_map(&mW2, W2, h, d, E));
  const int mt = Cs / TC_BM;
  {  // dH = dO W2 (W2 read with its output index contiguous), then dG, dU
    TcParams p = tc_params(c);
    p.b_mn = 1; p.M = Cs; p.N = h; p.K = d; p.dyn = TC_DYN_M; p.E = E; p.counts = rt->counts;
    p.out0 = (__nv_bfloat16*)dG; p.out1 = (__nv_bfloat16*)dU;
    p.in0 = (const __nv_bfloat16*)G; p.in1 = (const __nv_bfloat16*)U;
    p.out_bs = (long long)Cs * h; p.ld_out = h; p.stats = stats;
    ETR_TRY((tc_run<TC_EPI_DSWIGLU>(tc_form_of(c, TC_EPI_DSWIGLU, p), "tc_gemm_dswiglu", mdO, mdO, mW2, mW2, p,
                                            E * mt * ceil_div(h, 256), st)));
  }
  {  // dXp = dG W1g + dU W1u: one contraction over 2h
    TcParams p = tc_params(c);
    p.b_mn = 1; p.k1_blocks = ceil_div(h, TC_BK); p.M = Cs; p.N = d; p.K = 2 * h; p.dyn = TC_DYN_M;
    p.E = E; p.counts = rt->counts;
    p.out0 = (__nv_bfloat16*)dXp; p.out_bs = (long long)Cs * d; p.ld_out = d; p.stats = stats;
    ETR_TRY((tc_run<TC_EPI_STORE>(tc_form_of(c, TC_EPI_STORE, p), "tc_gemm_dxp", mdG, mdU, mW1g, mW1u, p,
                                          E * mt * ceil_div(d, 256), st)));
  }
  {  // dW2 = dO^T H: contraction over the expert's rows, both operands MN-major
    TcParams p = tc_params(c);
    p.a_mn = 1; p.b_mn = 1; p.M = d; p.N = h; p.dyn = TC_DYN_K; p.E = E; p.counts = rt->counts;
    p.out0 = (__nv_bfloat16*)dW2; p.out_bs = (long long)d * h; p.ld_out = h; p.stats = stats;
    p.out_f32 = c->grad_fp32 != 0;
    ETR_TRY((tc_run<TC_EPI_STORE>(tc_form_of(c, TC_EPI_STORE, p), "tc_gemm_dw2", mdO, mdO, mH, mH, p,
                                          E * ceil_div(d, TC_BM) * ceil_div(h, 256), st)));
  }
  for (int which = 0; which < 2; ++which) {  // dW1g = dG^T Xp, dW1u = dU^T Xp
    TcParams p = tc_params(c);
    p.a_mn = 1; p.b_mn = 1; p.M = h; p.N = d; p.dyn = TC_DYN_K; p.E = E; p.counts = rt->counts;
    if (Xtok) { p.gather = 2; p.gather_ld = Cs; p.gather_oob = c->T; p.gather_idx = rt->slot_token; }
    p.out0 = (__nv_bfloat16*)(which ? dW1u : dW1g); p.out_bs = (long long)h * d; p.ld_out = d; p.stats = stats;
    p.out_f32 = c->grad_fp32 != 0;
    const CUtensorMap& ma = which ? mdU : mdG;
    ETR_TRY((tc_run<TC_EPI_STORE>(tc_form_of(c, TC_EPI_STORE, p), "tc_gemm_dw1", ma, ma, mXp, mXp, p,
                                          E * ceil_div(h, TC_BM) * ceil_div(d, 256), st)));
  }
  return ETR_OK;
}

// The pipeline's bounded wait exercised on its own: thread 0 waits on an mbarrier that nothing ever
// arrives on (no TMA, no tensor memory, nothing in flight), gives up after `limit` cycles and leaves
// the code 0x7c08 in error_word, exactly as a GEMM kernel would; the kernel then returns normally.
__global__ void __launch_bounds__(32) tc_wait_selftest_kernel(etr_stats* stats, long long limit) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag_s;
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (threadIdx.x == 0 && !mbar_wait(smem_u32(&bar), 0u, &abort_flag_s, limit))
    atomicExch(&stats->error_word, 0x7c08);
}

etr_status tc_wait_selftest(etr_stats* stats, long long limit, cudaStream_t st) {
  ETR_TIME_BEGIN("tc_wait_selftest_kernel");
  tc_wait_selftest_kernel<<<1, 32, 0, st>>>(stats, limit);
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

}  // namespace etr
