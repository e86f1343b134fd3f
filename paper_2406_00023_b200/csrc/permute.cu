// Token rearrangement and gate-weighted combine, forward and backward.  All four kernels
// are pure streaming: 16-byte vectors, one pass over every byte they must touch.
#include "common.cuh"

namespace etr {

// Xp[r,:] = X[slot_token[r],:] for rows in use; pad rows (up to the next multiple of 128
// after counts[i]) are zero-filled; rows beyond are left alone.  One warp per row.
template <class T>
__global__ void __launch_bounds__(256)
dispatch_kernel(const T* __restrict__ X, const int32_t* __restrict__ counts,
                const int32_t* __restrict__ slot_token, T* __restrict__ Xp, int d, int C_stride,
                int n_rows) {
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= n_rows) return;
  const int i = r / C_stride, p = r - i * C_stride;
  const int lim = (counts[i] + 127) & ~127;
  if (p >= lim) return;
  const int t = slot_token[r];
  uint4* dst = reinterpret_cast<uint4*>(Xp + (size_t)r * d);
  const int nv = d * (int)sizeof(T) / 16;
  if (t >= 0) {
    const uint4* src = reinterpret_cast<const uint4*>(X + (size_t)t * d);
#pragma unroll 4
    for (int v = lane; v < nv; v += 32) dst[v] = __ldg(src + v);
  } else {
    for (int v = lane; v < nv; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
  }
}

// Y[t,:] = sum_{r in rows(t)} gate[r] O[r,:]   (gate == nullptr: plain sum, used for dX).
// A block takes COMBINE_TOKENS consecutive tokens.  It first copies their row lists and gates to
// shared memory (two rounds of dependent loads for the whole chunk instead of two per token), then
// every thread owns NV groups of 8 consecutive elements of a token, 1/NV of a row apart, and walks
// the token's rows two at a time: 2 NV independent 16-byte loads in flight per thread, none of them
// waiting for an index.  Rows are added in list order (the result does not depend on the chunking).
constexpr int COMBINE_TOKENS = 8;
constexpr int COMBINE_ROWS = 512;     // row entries held in shared memory; later ones are read in place

template <class T, int NV>
__global__ void __launch_bounds__(256)
combine_kernel(const T* __restrict__ O, const float* __restrict__ gate,
               const int32_t* __restrict__ tok_ptr, const int32_t* __restrict__ tok_row,
               T* __restrict__ Y, int Ttok, int d) {
  __shared__ int s_ptr[COMBINE_TOKENS + 1];
  __shared__ int s_row[COMBINE_ROWS];
  __shared__ float s_gate[COMBINE_ROWS];
  const int tid = threadIdx.x;
  const int t0 = blockIdx.x * COMBINE_TOKENS;
  const int nt = min(COMBINE_TOKENS, Ttok - t0);
  if (tid <= nt) s_ptr[tid] = tok_ptr[t0 + tid];
  __syncthreads();
  const int base = s_ptr[0];
  const int staged = min(s_ptr[nt] - base, COMBINE_ROWS);
  for (int i = tid; i < staged; i += 256) {
    const int r = tok_row[base + i];
    s_row[i] = r;
    s_gate[i] = gate ? gate[r] : 1.0f;
  }
  __syncthreads();
  auto entry = [&](int q, int& r, float& g) {
    if (q < COMBINE_ROWS) { r = s_row[q]; g = s_gate[q]; }
    else { r = tok_row[base + q]; g = gate ? gate[r] : 1.0f; }
  };
  const int vpt = d / 8 / NV;                       // threads per token
  for (int w = tid; w < nt * vpt; w += 256) {
    const int tl = w / vpt, v = w - tl * vpt;
    const int end = s_ptr[tl + 1] - base;
    float acc[NV][8];
#pragma unroll
    for (int u = 0; u < NV; ++u)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[u][e] = 0.f;
    int q = s_ptr[tl] - base;
    for (; q + 2 <= end; q += 2) {
      int r0, r1;
      float g0, g1;
      entry(q, r0, g0);
      entry(q + 1, r1, g1);
      Vec8<T> o0[NV], o1[NV];
#pragma unroll
      for (int u = 0; u < NV; ++u) o0[u] = Vec8<T>::load(O + (size_t)r0 * d + (size_t)(v + u * vpt) * 8);
#pragma unroll
      for (int u = 0; u < NV; ++u) o1[u] = Vec8<T>::load(O + (size_t)r1 * d + (size_t)(v + u * vpt) * 8);
#pragma unroll
      for (int u = 0; u < NV; ++u)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[u][e] = fmaf(g1, o1[u].v[e], fmaf(g0, o0[u].v[e], acc[u][e]));
    }
    if (q < end) {
      int r;
      float g;
      entry(q, r, g);
      Vec8<T> o[NV];
#pragma unroll
      for (int u = 0; u < NV; ++u) o[u] = Vec8<T>::load(O + (size_t)r * d + (size_t)(v + u * vpt) * 8);
#pragma unroll
      for (int u = 0; u < NV; ++u)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[u][e] = fmaf(g, o[u].v[e], acc[u][e]);
    }
#pragma unroll
    for (int u = 0; u < NV; ++u)
      Vec8<T>::store(Y + (size_t)(t0 + tl) * d + (size_t)(v + u * vpt) * 8, acc[u]);
  }
}

// dO[r,:] = gate[r] dY[t(r),:], dgate[r] = <dY[t(r),:], O[r,:]>; pad rows zero.  Warp per row.
template <class T>
__global__ void __launch_bounds__(256)
combine_bwd_kernel(const T* __restrict__ dY, const T* __restrict__ O,
                   const int32_t* __restrict__ counts, const int32_t* __restrict__ slot_token,
                   const float* __restrict__ gate, T* __restrict__ dO, float* __restrict__ dgate,
                   int d, int C_stride, int n_rows) {
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= n_rows) return;
  const int i = r / C_stride, p = r - i * C_stride;
  const int lim = (counts[i] + 127) & ~127;
  if (p >= lim) return;
  const int t = slot_token[r];
  T* dst = dO + (size_t)r * d;
  if (t < 0) {
    const int nv = d * (int)sizeof(T) / 16;
    for (int v = lane; v < nv; v += 32) reinterpret_cast<uint4*>(dst)[v] = make_uint4(0, 0, 0, 0);
    if (lane == 0) dgate[r] = 0.f;
    return;
  }
  const float g = gate[r];
  const T* gy = dY + (size_t)t * d;
  const T* o = O + (size_t)r * d;
  float dot = 0.f;
#pragma unroll 2
  for (int v = lane; v < d / 8; v += 32) {
    Vec8<T> a = Vec8<T>::load(gy + v * 8), b = Vec8<T>::load(o + v * 8);
    float out[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { out[e] = g * a.v[e]; dot = fmaf(a.v[e], b.v[e], dot); }
    Vec8<T>::store(dst + v * 8, out);
  }
  dot = warp_sum(dot);
  if (lane == 0) dgate[r] = dot;
}

// Y[t,:] = 0 for tokens without a row (the part of the combine that the fused Top-1 epilogue of the
// down GEMM leaves over).  One warp per token.
__global__ void __launch_bounds__(256)
zero_unrouted_kernel(const int32_t* __restrict__ tok_ptr, uint4* __restrict__ Y, int Ttok, int row_vec) {
  const int t = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= Ttok || tok_ptr[t] != tok_ptr[t + 1]) return;
  uint4* dst = Y + (size_t)t * row_vec;
  for (int v = lane; v < row_vec; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
}

etr_status zero_unrouted_rows(const etr_config* c, const etr_route* rt, void* Y, cudaStream_t st) {
  ETR_TIME_BEGIN("zero_unrouted_kernel");
  zero_unrouted_kernel<<<ceil_div(c->T, 8), 256, 0, st>>>(rt->tok_ptr, (uint4*)Y, c->T,
                                                          (int)((size_t)c->d * elem_bytes(c->dtype) / 16));
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

template <class T>
static etr_status permute_launch(int which, const etr_config* c, const etr_route* rt, const void* a,
                                 const void* b, void* out, float* dgate, cudaStream_t st) {
  const int Cs = c_stride_of(c), n_rows = c->E * Cs;
  switch (which) {
    case 0:
      ETR_TIME_BEGIN("dispatch_kernel");
      dispatch_kernel<T><<<ceil_div(n_rows, 8), 256, 0, st>>>((const T*)a, rt->counts, rt->slot_token,
                                                             (T*)out, c->d, Cs, n_rows);
      break;
    case 1:
    case 3: {
      const float* g = which == 1 ? rt->gate : nullptr;
      ETR_TIME_BEGIN("combine_kernel");
      const unsigned grid = (unsigned)ceil_div(c->T, COMBINE_TOKENS);
      if (c->d % 16 == 0)
        combine_kernel<T, 2><<<grid, 256, 0, st>>>((const T*)a, g, rt->tok_ptr, rt->tok_row, (T*)out, c->T, c->d);
      else
        combine_kernel<T, 1><<<grid, 256, 0, st>>>((const T*)a, g, rt->tok_ptr, rt->tok_row, (T*)out, c->T, c->d);
      break;
    }
    case 2:
      ETR_TIME_BEGIN("combine_bwd_kernel");
      combine_bwd_kernel<T><<<ceil_div(n_rows, 8), 256, 0, st>>>(
          (const T*)a, (const T*)b, rt->counts, rt->slot_token, rt->gate, (T*)out, dgate, c->d, Cs, n_rows);
      break;
  }
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

static etr_status permute_dispatch(int which, const etr_config* c, const etr_route* rt, const void* a,
                                   const void* b, void* out, float* dgate, cudaStream_t st) {
  return c->dtype == ETR_BF16 ? permute_launch<__nv_bfloat16>(which, c, rt, a, b, out, dgate, st)
                              : permute_launch<float>(which, c, rt, a, b, out, dgate, st);
}

etr_status dispatch_forward(const etr_config* c, const void* X, const etr_route* rt, void* Xp, cudaStream_t st) {
  return permute_dispatch(0, c, rt, X, nullptr, Xp, nullptr, st);
}
etr_status combine_forward(const etr_config* c, const etr_route* rt, const void* O, void* Y, cudaStream_t st) {
  return permute_dispatch(1, c, rt, O, nullptr, Y, nullptr, st);
}
etr_status combine_backward(const etr_config* c, const etr_route* rt, const void* dY, const void* O,
                            void* dO, float* dgate, cudaStream_t st) {
  return permute_dispatch(2, c, rt, dY, O, dO, dgate, st);
}
etr_status dispatch_backward(const etr_config* c, const etr_route* rt, const void* dXp, void* dX, cudaStream_t st) {
  return permute_dispatch(3, c, rt, dXp, nullptr, dX, nullptr, st);
}


// fp32 -> bf16 (round to nearest even), eight values per thread: the expert weights of a layer that keeps
// fp32 master weights, rounded once per pass for the GEMMs.
__global__ void __launch_bounds__(256) cast_f32_to_bf16_kernel(const float4* __restrict__ src, uint4* __restrict__ dst,
                                                               size_t n8) {
  for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < n8; i += (size_t)gridDim.x * 256) {
    const float4 a = src[2 * i], b = src[2 * i + 1];
    const __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x, a.y), p1 = __floats2bfloat162_rn(a.z, a.w);
    const __nv_bfloat162 p2 = __floats2bfloat162_rn(b.x, b.y), p3 = __floats2bfloat162_rn(b.z, b.w);
    dst[i] = make_uint4(*reinterpret_cast<const uint32_t*>(&p0), *reinterpret_cast<const uint32_t*>(&p1),
                        *reinterpret_cast<const uint32_t*>(&p2), *reinterpret_cast<const uint32_t*>(&p3));
  }
}

etr_status cast_f32_to_bf16(const void* src, void* dst, size_t n, cudaStream_t st) {
  if (src == nullptr || dst == nullptr) return ETR_ERR_ARG;
  if (n % 8 != 0) return ETR_ERR_SHAPE;
  if (!aligned16(src) || !aligned16(dst)) return ETR_ERR_ALIGN;
  const size_t n8 = n / 8;
  const size_t want = (n8 + 255) / 256, cap = (size_t)current_sm_count() * 16;
  ETR_TIME_BEGIN("cast_weights_kernel");
  cast_f32_to_bf16_kernel<<<(unsigned)(want < cap ? (want ? want : 1) : cap), 256, 0, st>>>((const float4*)src,
                                                                                            (uint4*)dst, n8);
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

}  // namespace etr
