// Softmax-gate variant and load statistics.
//
// The default gate of a selected pair (t, i) is the raw affinity delta_ti.  In the variant the
// gate is the softmax of token t's affinities over all E experts (the example gate of the general
// MoE equation); the softmax couples all experts of a token, so its backward produces a dense
// d delta [T, E] instead of the sparse (route, dgate) pair.  One warp per token throughout; sums
// run in a fixed lane order, so results are deterministic.
#include "common.cuh"

namespace etr {

// lse[t] = log sum_j exp(delta_tj); gate[r] = exp(delta_ti - lse[t]) for every row r of token t.
__global__ void __launch_bounds__(256)
gate_softmax_kernel(const float* __restrict__ delta, const int32_t* __restrict__ tok_ptr,
                    const int32_t* __restrict__ tok_row, float* __restrict__ gate,
                    float* __restrict__ lse, int Ttok, int E, int C_stride) {
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= Ttok) return;
  const float* dt = delta + (size_t)t * E;
  float mx = -INFINITY;
  for (int j = lane; j < E; j += 32) mx = fmaxf(mx, dt[j]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float s = 0.f;
  for (int j = lane; j < E; j += 32) s += expf(dt[j] - mx);
  s = warp_sum(s);
  const float l = mx + logf(s);
  if (lane == 0) lse[t] = l;
  for (int q = tok_ptr[t] + lane; q < tok_ptr[t + 1]; q += 32) {
    const int r = tok_row[q];
    gate[r] = expf(dt[r / C_stride] - l);
  }
}

// s_t = sum over the token's rows of dgate[r] gate[r];
// ddelta[t][j] = p_tj (g_tj - s_t), p_tj = exp(delta_tj - lse[t]), g_tj = dgate of the row of (t, j)
// if selected, else 0.
__global__ void __launch_bounds__(256)
gate_softmax_bwd_kernel(const float* __restrict__ delta, const float* __restrict__ lse,
                        const int32_t* __restrict__ tok_ptr, const int32_t* __restrict__ tok_row,
                        const float* __restrict__ gate, const float* __restrict__ dgate,
                        float* __restrict__ ddelta, int Ttok, int E, int C_stride) {
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= Ttok) return;
  const int beg = tok_ptr[t], end = tok_ptr[t + 1];
  float* out = ddelta + (size_t)t * E;
  if (beg == end) {               // no selected expert: no gradient reaches this token's affinities
    for (int j = lane; j < E; j += 32) out[j] = 0.f;
    return;
  }
  float s = 0.f;
  for (int q = beg + lane; q < end; q += 32) {
    const int r = tok_row[q];
    s = fmaf(dgate[r], gate[r], s);
  }
  s = warp_sum(s);
  const float l = lse[t];
  const float* dt = delta + (size_t)t * E;
  for (int j = lane; j < E; j += 32) out[j] = -expf(dt[j] - l) * s;
  __syncwarp();
  for (int q = beg + lane; q < end; q += 32) {
    const int r = tok_row[q];
    out[r / C_stride] = gate[r] * (dgate[r] - s);
  }
}

// load[i] = counts[i] / T; gate_mean[i] = (sum of the gates of expert i's rows) / T.  One block
// per expert; a fixed-shape tree reduction.
__global__ void __launch_bounds__(256)
load_stats_kernel(const int32_t* __restrict__ counts, const float* __restrict__ gate,
                  float* __restrict__ load, float* __restrict__ gate_mean, int Ttok, int C_stride) {
  __shared__ float red[8];
  const int i = blockIdx.x, tid = threadIdx.x;
  const int n = counts[i];
  float s = 0.f;
  for (int p = tid; p < n; p += 256) s += gate[(size_t)i * C_stride + p];
  s = warp_sum(s);
  if ((tid & 31) == 0) red[tid >> 5] = s;
  __syncthreads();
  if (tid == 0) {
    float a = 0.f;
    for (int w = 0; w < 8; ++w) a += red[w];
    load[i] = (float)n / (float)Ttok;
    gate_mean[i] = a / (float)Ttok;
  }
}

etr_status gate_softmax_forward(const etr_config* c, const float* delta, const etr_route* rt, float* lse,
                                cudaStream_t st) {
  ETR_TIME_BEGIN("gate_softmax_kernel");
  gate_softmax_kernel<<<ceil_div(c->T, 8), 256, 0, st>>>(delta, rt->tok_ptr, rt->tok_row, rt->gate, lse,
                                                         c->T, c->E, c_stride_of(c));
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

etr_status gate_softmax_backward(const etr_config* c, const float* delta, const float* lse,
                                 const etr_route* rt, const float* dgate, float* ddelta, cudaStream_t st) {
  ETR_TIME_BEGIN("gate_softmax_bwd_kernel");
  gate_softmax_bwd_kernel<<<ceil_div(c->T, 8), 256, 0, st>>>(delta, lse, rt->tok_ptr, rt->tok_row, rt->gate,
                                                             dgate, ddelta, c->T, c->E, c_stride_of(c));
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

etr_status load_stats_launch(const etr_config* c, const etr_route* rt, float* load, float* gate_mean,
                             cudaStream_t st) {
  ETR_TIME_BEGIN("load_stats_kernel");
  load_stats_kernel<<<c->E, 256, 0, st>>>(rt->counts, rt->gate, load, gate_mean, c->T, c_stride_of(c));
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

}  // namespace etr
