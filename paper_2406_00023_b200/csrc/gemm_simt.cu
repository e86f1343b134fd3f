// Grouped GEMMs of the expert FFN on the CUDA cores (fp32 accumulate).  This is the path
// for fp32 layers and the cross-check for the tensor-core kernels; the bf16 layer runs on
// gemm_tcgen05.cu.  One generic kernel: 64x64x16 tiles, 4x4 outputs per thread, operands
// addressed by (row stride, column stride) so the same code serves K-major and MN-major
// inputs; blockIdx.z is the expert and the row (or contraction) extent comes from counts.
#include "common.cuh"

namespace etr {

struct Operand {
  const void* ptr;
  long long batch_stride;   // elements between experts
  int s_row, s_col;         // element (r,c) at ptr[batch*batch_stride + r*s_row + c*s_col]
};

enum { EPI_STORE = 0, EPI_SWIGLU = 1, EPI_DSWIGLU = 2 };
enum { DYN_NONE = 0, DYN_M = 1, DYN_K = 2 };

struct GemmArgs {
  Operand A[2], B[2];       // A: [M,K], B: [K,N]
  int npair;
  void* out0; void* out1; void* out2;   // STORE: C | SWIGLU: G,U,H | DSWIGLU: dG,dU
  const void* in0; const void* in1;     // DSWIGLU: G,U
  int M, N, K, ld_out;
  long long out_bs;
  const int32_t* counts;
  int dyn, m_cap;
  int out_f32;              // STORE: C is fp32 whatever T is (weight gradients with grad_fp32)
};

__device__ inline float silu_f(float v) { return v / (1.0f + expf(-v)); }
__device__ inline float sigmoid_f(float v) { return 1.0f / (1.0f + expf(-v)); }

template <class T, int EPI>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs g) {
  constexpr int BM = 64, BN = 64, BK = 16;
  constexpr bool SEP = (EPI == EPI_SWIGLU);
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int e = blockIdx.z;
  int M = g.M, K = g.K;
  if (g.dyn == DYN_M) M = min(g.m_cap, (g.counts[e] + 127) & ~127);
  if (g.dyn == DYN_K) K = g.counts[e];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (m0 >= M) return;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc0[4][4] = {}, acc1[4][4] = {};

  for (int pr = 0; pr < g.npair; ++pr) {
    const T* A = (const T*)g.A[pr].ptr + (long long)e * g.A[pr].batch_stride;
    const T* B = (const T*)g.B[pr].ptr + (long long)e * g.B[pr].batch_stride;
    const int sAr = g.A[pr].s_row, sAc = g.A[pr].s_col, sBr = g.B[pr].s_row, sBc = g.B[pr].s_col;
    for (int k0 = 0; k0 < K; k0 += BK) {
      for (int idx = tid; idx < BM * BK; idx += 256) {
        int mm, kk;
        if (sAc == 1) { kk = idx % BK; mm = idx / BK; } else { mm = idx % BM; kk = idx / BM; }
        const int gm = m0 + mm, gk = k0 + kk;
        As[kk][mm] = (gm < M && gk < K) ? to_f32<T>(A[(long long)gm * sAr + (long long)gk * sAc]) : 0.f;
      }
      for (int idx = tid; idx < BN * BK; idx += 256) {
        int nn, kk;
        if (sBr == 1) { kk = idx % BK; nn = idx / BK; } else { nn = idx % BN; kk = idx / BN; }
        const int gn = n0 + nn, gk = k0 + kk;
        Bs[kk][nn] = (gn < g.N && gk < K) ? to_f32<T>(B[(long long)gk * sBr + (long long)gn * sBc]) : 0.f;
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) {
        const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
        const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
        const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
        if (SEP && pr == 1) {
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc1[i][j] = fmaf(av[i], bv[j], acc1[i][j]);
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc0[i][j] = fmaf(av[i], bv[j], acc0[i][j]);
        }
      }
      __syncthreads();
    }
  }

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= g.N) continue;
      const long long o = (long long)e * g.out_bs + (long long)gm * g.ld_out + gn;
      if (EPI == EPI_STORE) {
        if (g.out_f32) ((float*)g.out0)[o] = acc0[i][j];
        else ((T*)g.out0)[o] = from_f32<T>(acc0[i][j]);
      } else if (EPI == EPI_SWIGLU) {
        const float gg = acc0[i][j], uu = acc1[i][j];
        ((T*)g.out0)[o] = from_f32<T>(gg);
        ((T*)g.out1)[o] = from_f32<T>(uu);
        ((T*)g.out2)[o] = from_f32<T>(silu_f(gg) * uu);
      } else {
        const float dh = acc0[i][j];
        const float gg = to_f32<T>(((const T*)g.in0)[o]), uu = to_f32<T>(((const T*)g.in1)[o]);
        const float s = sigmoid_f(gg);
        ((T*)g.out0)[o] = from_f32<T>(dh * uu * s * (1.0f + gg * (1.0f - s)));
        ((T*)g.out1)[o] = from_f32<T>(dh * gg * s);
      }
    }
  }
}

template <class T, int EPI>
static etr_status launch(const GemmArgs& g, int E, cudaStream_t st) {
  dim3 grid(ceil_div(g.N, 64), ceil_div(g.dyn == DYN_M ? g.m_cap : g.M, 64), E);
  ETR_TIME_BEGIN("gemm_simt_kernel");
  gemm_simt_kernel<T, EPI><<<grid, 256, 0, st>>>(g);
  ETR_LAUNCH_CHECK();
  return ETR_OK;
}

template <class T>
static etr_status ffn_forward_t(const etr_config* c, const etr_route* rt, const void* Xp,
                                const void* W1g, const void* W1u, const void* W2, void* G, void* U,
                                void* H, void* O, cudaStream_t st) {
  const int d = c->d, h = c->h, Cs = c_stride_of(c), E = c->E;
  GemmArgs g = {};
  g.counts = rt->counts; g.dyn = DYN_M; g.m_cap = Cs;
  // G,U,H = swiglu(Xp W1g^T, Xp W1u^T): A = Xp [rows,d]; B(k,n) = W1[n,k]
  g.A[0] = g.A[1] = {Xp, (long long)Cs * d, d, 1};
  g.B[0] = {W1g, (long long)h * d, 1, d};
  g.B[1] = {W1u, (long long)h * d, 1, d};
  g.npair = 2; g.M = Cs; g.N = h; g.K = d; g.ld_out = h; g.out_bs = (long long)Cs * h;
  g.out0 = G; g.out1 = U; g.out2 = H;
  ETR_TRY((launch<T, EPI_SWIGLU>(g, E, st)));
  // O = H W2^T: B(k,n) = W2[n,k]
  GemmArgs o = {};
  o.counts = rt->counts; o.dyn = DYN_M; o.m_cap = Cs;
  o.A[0] = {H, (long long)Cs * h, h, 1};
  o.B[0] = {W2, (long long)d * h, 1, h};
  o.npair = 1; o.M = Cs; o.N = d; o.K = h; o.ld_out = d; o.out_bs = (long long)Cs * d; o.out0 = O;
  return launch<T, EPI_STORE>(o, E, st);
}

template <class T>
static etr_status ffn_backward_t(const etr_config* c, const etr_route* rt, const void* dO,
                                 const void* Xp, const void* G, const void* U, const void* H,
                                 const void* W1g, const void* W1u, const void* W2, void* dG,
                                 void* dU, void* dXp, void* dW1g, void* dW1u, void* dW2,
                                 cudaStream_t st) {
  const int d = c->d, h = c->h, Cs = c_stride_of(c), E = c->E;
  {  // dH = dO W2 -> dG, dU.  B(k,n) = W2[k,n]
    GemmArgs g = {};
    g.counts = rt->counts; g.dyn = DYN_M; g.m_cap = Cs;
    g.A[0] = {dO, (long long)Cs * d, d, 1};
    g.B[0] = {W2, (long long)d * h, h, 1};
    g.npair = 1; g.M = Cs; g.N = h; g.K = d; g.ld_out = h; g.out_bs = (long long)Cs * h;
    g.out0 = dG; g.out1 = dU; g.in0 = G; g.in1 = U;
    ETR_TRY((launch<T, EPI_DSWIGLU>(g, E, st)));
  }
  {  // dXp = dG W1g + dU W1u.  B(k,n) = W1[k,n]
    GemmArgs g = {};
    g.counts = rt->counts; g.dyn = DYN_M; g.m_cap = Cs;
    g.A[0] = {dG, (long long)Cs * h, h, 1};
    g.A[1] = {dU, (long long)Cs * h, h, 1};
    g.B[0] = {W1g, (long long)h * d, d, 1};
    g.B[1] = {W1u, (long long)h * d, d, 1};
    g.npair = 2; g.M = Cs; g.N = d; g.K = h; g.ld_out = d; g.out_bs = (long long)Cs * d; g.out0 = dXp;
    ETR_TRY((launch<T, EPI_STORE>(g, E, st)));
  }
  {  // dW2[a,b] = sum_r dO[r,a] H[r,b]: A(m,k) = dO[k,m], B(k,n) = H[k,n]
    GemmArgs g = {};
    g.counts = rt->counts; g.dyn = DYN_K;
    g.A[0] = {dO, (long long)Cs * d, 1, d};
    g.B[0] = {H, (long long)Cs * h, h, 1};
    g.npair = 1; g.M = d; g.N = h; g.K = 0; g.ld_out = h; g.out_bs = (long long)d * h; g.out0 = dW2;
    g.out_f32 = c->grad_fp32 != 0;
    ETR_TRY((launch<T, EPI_STORE>(g, E, st)));
  }
  for (int which = 0; which < 2; ++which) {  // dW1[b,c] = sum_r dG[r,b] Xp[r,c]
    GemmArgs g = {};
    g.counts = rt->counts; g.dyn = DYN_K;
    g.A[0] = {which ? dU : dG, (long long)Cs * h, 1, h};
    g.B[0] = {Xp, (long long)Cs * d, d, 1};
    g.npair = 1; g.M = h; g.N = d; g.K = 0; g.ld_out = d; g.out_bs = (long long)h * d;
    g.out0 = which ? dW1u : dW1g;
    g.out_f32 = c->grad_fp32 != 0;
    ETR_TRY((launch<T, EPI_STORE>(g, E, st)));
  }
  return ETR_OK;
}

etr_status simt_ffn_forward(const etr_config* c, const etr_route* rt, const void* Xp, const void* W1g,
                            const void* W1u, const void* W2, void* G, void* U, void* H, void* O,
                            cudaStream_t st) {
  return c->dtype == ETR_BF16
             ? ffn_forward_t<__nv_bfloat16>(c, rt, Xp, W1g, W1u, W2, G, U, H, O, st)
             : ffn_forward_t<float>(c, rt, Xp, W1g, W1u, W2, G, U, H, O, st);
}

etr_status simt_ffn_backward(const etr_config* c, const etr_route* rt, const void* dO, const void* Xp,
                             const void* G, const void* U, const void* H, const void* W1g,
                             const void* W1u, const void* W2, void* dG, void* dU, void* dXp,
                             void* dW1g, void* dW1u, void* dW2, cudaStream_t st) {
  return c->dtype == ETR_BF16
             ? ffn_backward_t<__nv_bfloat16>(c, rt, dO, Xp, G, U, H, W1g, W1u, W2, dG, dU, dXp, dW1g, dW1u, dW2, st)
             : ffn_backward_t<float>(c, rt, dO, Xp, G, U, H, W1g, W1u, W2, dG, dU, dXp, dW1g, dW1u, dW2, st);
}

}  // namespace etr
