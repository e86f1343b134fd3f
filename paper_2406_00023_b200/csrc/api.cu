// C ABI of libetr: argument checks, buffer carving, stage wrappers, whole-layer calls.
#include <atomic>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include "common.cuh"

namespace etr {

static_assert(sizeof(etr_config) == 112 && sizeof(etr_stats) == 64, "layouts the bindings rely on");

static std::atomic<long long> g_launches{0};
void note_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// ---- optional per-kernel timing: one CUDA event pair per launch, on the launch stream ----
struct TimingRecord { const char* name; cudaEvent_t beg, end; };
static std::mutex g_timing_mu;
static bool g_timing_on = false;
static std::vector<TimingRecord> g_records;
static std::vector<cudaEvent_t> g_event_pool;

static cudaEvent_t take_event() {
  if (!g_event_pool.empty()) { cudaEvent_t e = g_event_pool.back(); g_event_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}
void timing_begin(const char* name, cudaStream_t st) {
  if (!g_timing_on) return;
  std::lock_guard<std::mutex> lk(g_timing_mu);
  TimingRecord r{name, take_event(), take_event()};
  if (r.beg) cudaEventRecord(r.beg, st);
  g_records.push_back(r);
}
void timing_end(cudaStream_t st) {
  if (!g_timing_on) return;
  std::lock_guard<std::mutex> lk(g_timing_mu);
  if (!g_records.empty() && g_records.back().end) cudaEventRecord(g_records.back().end, st);
}

static bool use_tc(const etr_config* c) {
  if (c->gemm_impl == ETR_GEMM_SIMT) return false;
  if (c->gemm_impl >= ETR_GEMM_TCGEN05 && c->gemm_impl <= ETR_GEMM_TCGEN05_2CTA_WIDE) return true;
  return c->dtype == ETR_BF16 && tc_available();
}

// Token rearrangement fused into the GEMM operand fetch (layer calls, tensor-core path only).
static bool fuse_dispatch(const etr_config* c) {
  return use_tc(c) && c->fuse_dispatch == ETR_FUSE_ON;
}

// Combine folded into the down GEMM's epilogue (layer calls, tensor-core path): only where it is exact,
// Top-1 token choice, in which a token has at most one row and its output needs no sum.
static bool fuse_combine(const etr_config* c) {
  return use_tc(c) && c->fuse_combine != ETR_FUSE_OFF && c->k == 1 && resolve_mode(c) == ETR_MODE_TCR;
}

// bf16 activations with fp32 expert weights (master weights of mixed-precision training): the GEMMs take
// both operands in one 16-bit type, so every call that multiplies by the weights first rounds them to bf16
// (round to nearest even) into the tail of the workspace, and the weight gradients come back in fp32.
static bool mixed_weights(const etr_config* c) { return c->dtype == ETR_BF16 && c->weight_dtype == ETR_F32; }
static size_t scratch_bytes(const etr_config* c) {      // the part of ws the stages use from offset 0
  size_t w = select_workspace_bytes(c);
  w = w > affinity_bwd_workspace_bytes(c) ? w : affinity_bwd_workspace_bytes(c);
  if (use_tc(c)) w = w > tc_workspace_bytes(c) ? w : tc_workspace_bytes(c);
  return align_up(w, 256);
}
static size_t weight_elems(const etr_config* c) { return (size_t)c->E * c->d * c->h; }
struct ExpertWeights { const void *W1g, *W1u, *W2; };
// The weights the kernels read: the caller's, or their bf16 copies behind the scratch part of ws
// (written here when `cast`, otherwise taken as an earlier call on the same ws left them).
static etr_status kernel_weights(const etr_config* c, const void* W1g, const void* W1u, const void* W2, void* ws,
                                 bool cast, ExpertWeights* out, cudaStream_t st) {
  *out = ExpertWeights{W1g, W1u, W2};
  if (!mixed_weights(c)) return ETR_OK;
  if (ws == nullptr) return ETR_ERR_ARG;
  const size_t n = weight_elems(c);
  char* base = (char*)ws + scratch_bytes(c);
  void* dst[3] = {base, base + 2 * n, base + 4 * n};
  const void* src[3] = {W1g, W1u, W2};
  if (cast)
    for (int i = 0; i < 3; ++i) ETR_TRY(cast_f32_to_bf16(src[i], dst[i], n, st));
  *out = ExpertWeights{dst[0], dst[1], dst[2]};
  return ETR_OK;
}
// The configuration the GEMM stages see under mixed weights: bf16 weights, fp32 weight gradients.
static etr_config gemm_config(const etr_config* c) {
  etr_config g = *c;
  if (mixed_weights(c)) { g.weight_dtype = ETR_BF16; g.grad_fp32 = 1; }
  return g;
}

static etr_status check_ptrs(std::initializer_list<const void*> ps) {
  for (const void* p : ps) {
    if (p == nullptr) return ETR_ERR_ARG;
    if (!aligned16(p)) return ETR_ERR_ALIGN;
  }
  return ETR_OK;
}

static etr_status check_route(const etr_route* r) {
  if (r == nullptr) return ETR_ERR_ARG;
  return check_ptrs({r->topk_idx, r->counts, r->slot_token, r->gate, r->tok_ptr, r->tok_row});
}

struct Carver {
  char* base; size_t off;
  void* take(size_t bytes) {
    off = align_up(off, 256);
    void* p = base ? base + off : nullptr;
    off += bytes;
    return p;
  }
};

static void carve(const etr_config* c, int staging, char* base, etr_buffers* b, size_t* total) {
  const size_t T = c->T, E = c->E, d = c->d, h = c->h, m = c->d / c->D, k = c->k;
  const size_t rows = E * (size_t)c_stride_of(c), eb = elem_bytes(c->dtype);
  size_t ws = 0;
  etr_workspace_bytes(c, &ws);
  Carver cv{base, 0};
  etr_buffers t;
  memset(&t, 0, sizeof(t));
  t.stats = (etr_stats*)cv.take(sizeof(etr_stats));
  t.route.topk_idx = (int32_t*)cv.take(T * k * 4);
  t.route.counts = (int32_t*)cv.take(E * 4);
  t.route.slot_token = (int32_t*)cv.take(rows * 4);
  t.route.gate = (float*)cv.take(rows * 4);
  t.route.tok_ptr = (int32_t*)cv.take((T + 1) * 4);
  t.route.tok_row = (int32_t*)cv.take(rows * 4);
  t.delta = (float*)cv.take(T * E * 4);
  t.Z = (float*)cv.take(T * m * 4);
  t.xnorm = (float*)cv.take(T * 4);
  t.rnorm = (float*)cv.take(E * 4);
  t.Xp = cv.take(rows * d * eb);
  t.G = cv.take(rows * h * eb);
  t.U = cv.take(rows * h * eb);
  t.H = cv.take(rows * h * eb);
  t.O = cv.take(rows * d * eb);
  t.dO = cv.take(rows * d * eb);
  t.dG = cv.take(rows * h * eb);
  t.dU = cv.take(rows * h * eb);
  t.dXp = cv.take(rows * d * eb);
  t.dgate = (float*)cv.take(rows * 4);
  t.ws = cv.take(ws);
  t.ws_bytes = ws;
  if (staging) {
    t.X_dev = cv.take(T * d * eb);
    t.dY_dev = cv.take(T * d * eb);
    t.Y_dev = cv.take(T * d * eb);
    t.dX_dev = cv.take(T * d * eb);
  }
  if (c->gate_mode == ETR_GATE_SOFTMAX) {
    t.lse = (float*)cv.take(T * 4);
    t.ddelta = (float*)cv.take(T * E * 4);
  }
  if (b) *b = t;
  *total = align_up(cv.off, 256);
}

}  // namespace etr

using namespace etr;

extern "C" {

const char* etr_status_string(etr_status s) {
  switch (s) {
    case ETR_OK: return "ok";
    case ETR_ERR_ARG: return "bad argument (NULL pointer, non-positive size or bad enum)";
    case ETR_ERR_SHAPE: return "sizes violate the shape rules";
    case ETR_ERR_ALIGN: return "pointer not 16-byte aligned";
    case ETR_ERR_WORKSPACE: return "buffer too small";
    case ETR_ERR_CUDA: return "CUDA call failed";
    case ETR_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case ETR_ERR_UNSUPPORTED: return "unsupported configuration";
  }
  return "unknown status";
}

etr_status etr_validate(const etr_config* c) {
  if (c == nullptr) return ETR_ERR_ARG;
  if (c->T < 1 || c->d < 1 || c->D < 1 || c->E < 1 || c->k < 1 || c->h < 1 || c->capacity < 1)
    return ETR_ERR_ARG;
  if (c->dtype != ETR_F32 && c->dtype != ETR_BF16) return ETR_ERR_ARG;
  if (c->mode < ETR_MODE_AUTO || c->mode > ETR_MODE_ECR) return ETR_ERR_ARG;
  if (c->gemm_impl < ETR_GEMM_AUTO || c->gemm_impl > ETR_GEMM_TCGEN05_2CTA_WIDE) return ETR_ERR_ARG;
  if (c->fuse_dispatch < ETR_FUSE_AUTO || c->fuse_dispatch > ETR_FUSE_ON) return ETR_ERR_ARG;
  if (c->fuse_combine < ETR_FUSE_AUTO || c->fuse_combine > ETR_FUSE_ON) return ETR_ERR_ARG;
  if (c->gate_mode != ETR_GATE_AFFINITY && c->gate_mode != ETR_GATE_SOFTMAX) return ETR_ERR_ARG;
  if (c->weight_dtype != ETR_F32 && c->weight_dtype != ETR_BF16) return ETR_ERR_ARG;
  if (c->threshold_mode < 0 || c->threshold_mode > (ETR_THRESHOLD_EXPERT | ETR_THRESHOLD_TOKEN)) return ETR_ERR_ARG;
  if (c->threshold_mode != ETR_THRESHOLD_OFF && (c->threshold_tau != c->threshold_tau ||
                                                  c->threshold_tau_token != c->threshold_tau_token))
    return ETR_ERR_ARG;                                   // NaN thresholds
  if (c->wait_limit_cycles < 0) return ETR_ERR_ARG;
  if (c->weight_dtype != c->dtype && !(c->dtype == ETR_BF16 && c->weight_dtype == ETR_F32)) return ETR_ERR_UNSUPPORTED;
  if (c->d % c->D != 0 || c->d % 8 != 0 || c->h % 8 != 0) return ETR_ERR_SHAPE;
  if (c->k > c->E || c->E > 256 || c->E > c->d / c->D) return ETR_ERR_SHAPE;
  if ((long long)c->T * c->E >= (1ll << 31)) return ETR_ERR_SHAPE;
  if ((long long)c->E * c_stride_of(c) >= (1ll << 31)) return ETR_ERR_SHAPE;
  if (use_tc(c)) {
    if (c->dtype != ETR_BF16) return ETR_ERR_UNSUPPORTED;
    if (c->d % 64 != 0 || c->h % 64 != 0) return ETR_ERR_UNSUPPORTED;
  }
  return ETR_OK;
}

int32_t etr_c_stride(const etr_config* c) { return c ? c_stride_of(c) : 0; }

etr_status etr_workspace_bytes(const etr_config* c, size_t* bytes) {
  if (bytes == nullptr) return ETR_ERR_ARG;
  ETR_TRY(etr_validate(c));
  *bytes = scratch_bytes(c) + (mixed_weights(c) ? align_up(3 * 2 * weight_elems(c), 256) : 0);
  return ETR_OK;
}

etr_status etr_buffers_bytes(const etr_config* c, int with_host_staging, size_t* bytes) {
  if (bytes == nullptr) return ETR_ERR_ARG;
  ETR_TRY(etr_validate(c));
  carve(c, with_host_staging, nullptr, nullptr, bytes);
  return ETR_OK;
}

etr_status etr_buffers_bind(const etr_config* c, int with_host_staging, void* base, size_t bytes,
                            etr_buffers* out) {
  if (base == nullptr || out == nullptr) return ETR_ERR_ARG;
  ETR_TRY(etr_validate(c));
  if (reinterpret_cast<uintptr_t>(base) & 255u) return ETR_ERR_ALIGN;
  size_t need = 0;
  carve(c, with_host_staging, nullptr, nullptr, &need);
  if (bytes < need) return ETR_ERR_WORKSPACE;
  carve(c, with_host_staging, (char*)base, out, &need);
  return ETR_OK;
}

etr_status etr_layout(const etr_config* c, int with_host_staging, etr_layout_info* out) {
  if (out == nullptr) return ETR_ERR_ARG;
  ETR_TRY(etr_validate(c));
  etr_buffers b;
  size_t total = 0;
  char* const base = reinterpret_cast<char*>(uintptr_t(256));      // any aligned non-null base: only differences are kept
  carve(c, with_host_staging, base, &b, &total);
  auto off = [&](const void* p) -> size_t { return p ? (size_t)(reinterpret_cast<const char*>(p) - base) : 0; };
  memset(out, 0, sizeof(*out));
  out->C_stride = c_stride_of(c);
  out->total_bytes = total;
  out->ws_bytes = b.ws_bytes;
  out->stats = off(b.stats);
  out->topk_idx = off(b.route.topk_idx); out->counts = off(b.route.counts); out->slot_token = off(b.route.slot_token);
  out->gate = off(b.route.gate); out->tok_ptr = off(b.route.tok_ptr); out->tok_row = off(b.route.tok_row);
  out->delta = off(b.delta); out->Z = off(b.Z); out->xnorm = off(b.xnorm); out->rnorm = off(b.rnorm);
  out->Xp = off(b.Xp); out->G = off(b.G); out->U = off(b.U); out->H = off(b.H); out->O = off(b.O);
  out->dO = off(b.dO); out->dG = off(b.dG); out->dU = off(b.dU); out->dXp = off(b.dXp); out->dgate = off(b.dgate);
  out->ws = off(b.ws);
  out->X_dev = off(b.X_dev); out->dY_dev = off(b.dY_dev); out->Y_dev = off(b.Y_dev); out->dX_dev = off(b.dX_dev);
  out->lse = off(b.lse); out->ddelta = off(b.ddelta);
  return ETR_OK;
}

etr_status etr_affinity(const etr_config* c, const void* X, const float* R, float* delta, float* Z,
                        float* xnorm, float* rnorm, etr_stats* stats, void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({X, R, delta, xnorm, rnorm, stats}));
  if (Z && !aligned16(Z)) return ETR_ERR_ALIGN;
  return affinity_forward(c, X, R, delta, Z, xnorm, rnorm, stats, (cudaStream_t)stream);
}

etr_status etr_select(const etr_config* c, const float* delta, etr_stats* stats,
                      const etr_route* route, void* ws, void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({delta, stats, ws}));
  ETR_TRY(check_route(route));
  return select_forward(c, delta, stats, route, ws, (cudaStream_t)stream);
}

etr_status etr_dispatch(const etr_config* c, const void* X, const etr_route* route, void* Xp,
                        void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({X, Xp}));
  ETR_TRY(check_route(route));
  return dispatch_forward(c, X, route, Xp, (cudaStream_t)stream);
}

etr_status etr_expert_ffn(const etr_config* c, const etr_route* route, const void* Xp,
                          const void* W1g, const void* W1u, const void* W2, void* G, void* U,
                          void* H, void* O, etr_stats* stats, void* ws, void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({Xp, W1g, W1u, W2, G, U, H, O}));
  ETR_TRY(check_route(route));
  ExpertWeights w;
  ETR_TRY(kernel_weights(c, W1g, W1u, W2, ws, true, &w, (cudaStream_t)stream));
  const etr_config g = gemm_config(c);
  if (use_tc(c)) {
    ETR_TRY(check_ptrs({stats, ws}));
    return tc_ffn_forward(&g, route, Xp, nullptr, w.W1g, w.W1u, w.W2, G, U, H, O, stats, ws, nullptr,
                          (cudaStream_t)stream);
  }
  return simt_ffn_forward(&g, route, Xp, w.W1g, w.W1u, w.W2, G, U, H, O, (cudaStream_t)stream);
}

etr_status etr_combine(const etr_config* c, const etr_route* route, const void* O, void* Y,
                       void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({O, Y}));
  ETR_TRY(check_route(route));
  return combine_forward(c, route, O, Y, (cudaStream_t)stream);
}

etr_status etr_combine_bwd(const etr_config* c, const etr_route* route, const void* dY,
                           const void* O, void* dO, float* dgate, void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({dY, O, dO, dgate}));
  ETR_TRY(check_route(route));
  return combine_backward(c, route, dY, O, dO, dgate, (cudaStream_t)stream);
}

// cast_weights: under mixed weights, round the fp32 weights to bf16 now (false: an earlier call on the same
// ws, the layer's forward pass, already left them there).
static etr_status expert_ffn_bwd(const etr_config* c, const etr_route* route, const void* dO,
                                 const void* Xp, const void* G, const void* U, const void* H,
                                 const void* W1g, const void* W1u, const void* W2, void* dG, void* dU,
                                 void* dXp, void* dW1g, void* dW1u, void* dW2, etr_stats* stats,
                                 void* ws, bool cast_weights, void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({dO, Xp, G, U, H, W1g, W1u, W2, dG, dU, dXp, dW1g, dW1u, dW2}));
  ETR_TRY(check_route(route));
  ExpertWeights w;
  ETR_TRY(kernel_weights(c, W1g, W1u, W2, ws, cast_weights, &w, (cudaStream_t)stream));
  const etr_config g = gemm_config(c);
  if (use_tc(c)) {
    ETR_TRY(check_ptrs({stats, ws}));
    return tc_ffn_backward(&g, route, dO, Xp, nullptr, G, U, H, w.W1g, w.W1u, w.W2, dG, dU, dXp, dW1g, dW1u, dW2,
                           stats, ws, (cudaStream_t)stream);
  }
  return simt_ffn_backward(&g, route, dO, Xp, G, U, H, w.W1g, w.W1u, w.W2, dG, dU, dXp, dW1g, dW1u, dW2,
                           (cudaStream_t)stream);
}

etr_status etr_expert_ffn_bwd(const etr_config* c, const etr_route* route, const void* dO,
                              const void* Xp, const void* G, const void* U, const void* H,
                              const void* W1g, const void* W1u, const void* W2, void* dG, void* dU,
                              void* dXp, void* dW1g, void* dW1u, void* dW2, etr_stats* stats,
                              void* ws, void* stream) {
  return expert_ffn_bwd(c, route, dO, Xp, G, U, H, W1g, W1u, W2, dG, dU, dXp, dW1g, dW1u, dW2, stats, ws, true,
                        stream);
}

etr_status etr_dispatch_bwd(const etr_config* c, const etr_route* route, const void* dXp, void* dX,
                            void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({dXp, dX}));
  ETR_TRY(check_route(route));
  return dispatch_backward(c, route, dXp, dX, (cudaStream_t)stream);
}

etr_status etr_select_bwd(const etr_config* c, const etr_route* route, const float* dgate) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({dgate}));
  return check_route(route);
}

etr_status etr_affinity_bwd(const etr_config* c, const void* X, const float* R, const float* delta,
                            const float* Z, const float* xnorm, const float* rnorm,
                            const etr_route* route, const float* dgate, void* dX, float* dR,
                            void* ws, void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({X, R, delta, Z, xnorm, rnorm, dgate, dX, dR, ws}));
  ETR_TRY(check_route(route));
  return affinity_backward(c, X, R, delta, Z, xnorm, rnorm, route, dgate, nullptr, nullptr, dX, dR, ws, nullptr,
                           (cudaStream_t)stream);
}

etr_status etr_gate_softmax(const etr_config* c, const float* delta, const etr_route* route, float* lse,
                            void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({delta, lse}));
  ETR_TRY(check_route(route));
  return gate_softmax_forward(c, delta, route, lse, (cudaStream_t)stream);
}

etr_status etr_gate_softmax_bwd(const etr_config* c, const float* delta, const float* lse,
                                const etr_route* route, const float* dgate, float* ddelta,
                                void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({delta, lse, dgate, ddelta}));
  ETR_TRY(check_route(route));
  return gate_softmax_backward(c, delta, lse, route, dgate, ddelta, (cudaStream_t)stream);
}

etr_status etr_affinity_bwd_dense(const etr_config* c, const void* X, const float* R, const float* delta,
                                  const float* Z, const float* xnorm, const float* rnorm,
                                  const etr_route* route, const float* ddelta, void* dX, float* dR,
                                  void* ws, void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({X, R, delta, Z, xnorm, rnorm, ddelta, dX, dR, ws}));
  ETR_TRY(check_route(route));
  return affinity_backward(c, X, R, delta, Z, xnorm, rnorm, route, nullptr, ddelta, nullptr, dX, dR, ws, nullptr,
                           (cudaStream_t)stream);
}

etr_status etr_load_stats(const etr_config* c, const etr_route* route, float* load, float* gate_mean,
                          void* stream) {
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({load, gate_mean}));
  ETR_TRY(check_route(route));
  return load_stats_launch(c, route, load, gate_mean, (cudaStream_t)stream);
}

etr_status etr_layer_forward(const etr_config* c, const void* X, const float* R, const void* W1g,
                             const void* W1u, const void* W2, const etr_buffers* b, void* Y,
                             void* stream) {
  if (b == nullptr) return ETR_ERR_ARG;
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({b->stats}));
  if (cudaMemsetAsync(b->stats, 0, sizeof(etr_stats), (cudaStream_t)stream) != cudaSuccess)
    return ETR_ERR_CUDA;
  ETR_TRY(etr_affinity(c, X, R, b->delta, b->Z, b->xnorm, b->rnorm, b->stats, stream));
  ETR_TRY(etr_select(c, b->delta, b->stats, &b->route, b->ws, stream));
  if (c->gate_mode == ETR_GATE_SOFTMAX) ETR_TRY(etr_gate_softmax(c, b->delta, &b->route, b->lse, stream));
  const bool fc = fuse_combine(c);
  if (fc) {                     // Top-1: Y is written by the down GEMM's epilogue; tokens without a row get zeros here
    ETR_TRY(check_ptrs({Y}));
    ETR_TRY(zero_unrouted_rows(c, &b->route, Y, (cudaStream_t)stream));
  }
  if (fuse_dispatch(c) || fc) {
    const bool fd = fuse_dispatch(c);      // the first GEMM gathers its rows from X: no Xp
    ETR_TRY(check_ptrs({X, W1g, W1u, W2, b->G, b->U, b->H, b->O, b->ws}));
    if (!fd) ETR_TRY(etr_dispatch(c, X, &b->route, b->Xp, stream));
    ExpertWeights w;
    ETR_TRY(kernel_weights(c, W1g, W1u, W2, b->ws, true, &w, (cudaStream_t)stream));
    const etr_config g = gemm_config(c);
    ETR_TRY(tc_ffn_forward(&g, &b->route, fd ? nullptr : b->Xp, fd ? X : nullptr, w.W1g, w.W1u, w.W2, b->G, b->U,
                           b->H, b->O, b->stats, b->ws, fc ? Y : nullptr, (cudaStream_t)stream));
  } else {
    ETR_TRY(etr_dispatch(c, X, &b->route, b->Xp, stream));
    ETR_TRY(etr_expert_ffn(c, &b->route, b->Xp, W1g, W1u, W2, b->G, b->U, b->H, b->O, b->stats, b->ws,
                           stream));
  }
  return fc ? ETR_OK : etr_combine(c, &b->route, b->O, Y, stream);
}

etr_status etr_layer_backward(const etr_config* c, const void* X, const float* R, const void* W1g,
                              const void* W1u, const void* W2, const void* dY, const etr_buffers* b,
                              void* dX, float* dR, void* dW1g, void* dW1u, void* dW2, void* stream) {
  if (b == nullptr) return ETR_ERR_ARG;
  ETR_TRY(etr_combine_bwd(c, &b->route, dY, b->O, b->dO, b->dgate, stream));
  if (fuse_dispatch(c)) {
    ETR_TRY(etr_validate(c));
    ETR_TRY(check_ptrs({X, b->dO, b->G, b->U, b->H, W1g, W1u, W2, b->dG, b->dU, b->dXp, dW1g, dW1u, dW2,
                        b->stats, b->ws}));
    ExpertWeights w;
    ETR_TRY(kernel_weights(c, W1g, W1u, W2, b->ws, false, &w, (cudaStream_t)stream));
    const etr_config g = gemm_config(c);
    ETR_TRY(tc_ffn_backward(&g, &b->route, b->dO, nullptr, X, b->G, b->U, b->H, w.W1g, w.W1u, w.W2, b->dG, b->dU,
                            b->dXp, dW1g, dW1u, dW2, b->stats, b->ws, (cudaStream_t)stream));
  } else {
    ETR_TRY(expert_ffn_bwd(c, &b->route, b->dO, b->Xp, b->G, b->U, b->H, W1g, W1u, W2, b->dG, b->dU,
                           b->dXp, dW1g, dW1u, dW2, b->stats, b->ws, false, stream));
  }
  // dispatch backward and the router gradient in one pass over dX
  ETR_TRY(etr_select_bwd(c, &b->route, b->dgate));
  ETR_TRY(check_ptrs({X, R, dX, dR, b->dXp, b->ws}));
  const float* ddelta = nullptr;
  if (c->gate_mode == ETR_GATE_SOFTMAX) {
    ETR_TRY(etr_gate_softmax_bwd(c, b->delta, b->lse, &b->route, b->dgate, b->ddelta, stream));
    ddelta = b->ddelta;
  }
  return affinity_backward(c, X, R, b->delta, b->Z, b->xnorm, b->rnorm, &b->route, b->dgate, ddelta,
                           b->dXp, dX, dR, b->ws, b->stats, (cudaStream_t)stream);
}

// Side streams and events for the host-buffer step (host-side objects, created once per device).
struct HostSlotEvents { cudaEvent_t x_ready, dy_ready, fwd_done, bwd_done, y_down, dx_down; bool used; };
struct HostStepCtx {
  cudaStream_t up = nullptr, down = nullptr;
  cudaEvent_t dy_ready = nullptr, fwd_done = nullptr, y_done = nullptr, start = nullptr;
  HostSlotEvents slot[ETR_HOST_SLOTS] = {};
};
static std::mutex g_ctx_mu;
static HostStepCtx g_ctx[64];

static etr_status host_step_ctx(HostStepCtx** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ETR_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_ctx_mu);
  HostStepCtx& c = g_ctx[dev];
  if (c.up == nullptr) {
    if (cudaStreamCreateWithFlags(&c.up, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&c.down, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&c.dy_ready, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c.fwd_done, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c.y_done, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c.start, cudaEventDisableTiming) != cudaSuccess)
      return ETR_ERR_CUDA;
    for (auto& sl : c.slot) {
      cudaEvent_t* ev[6] = {&sl.x_ready, &sl.dy_ready, &sl.fwd_done, &sl.bwd_done, &sl.y_down, &sl.dx_down};
      for (cudaEvent_t* e : ev)
        if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return ETR_ERR_CUDA;
      sl.used = false;
    }
  }
  *out = &c;
  return ETR_OK;
}

#define ETR_CUDA(expr) do { if ((expr) != cudaSuccess) return ETR_ERR_CUDA; } while (0)

etr_status etr_layer_step_host(const etr_config* c, const void* X_host, const void* dY_host,
                               const float* R, const void* W1g, const void* W1u, const void* W2,
                               const etr_buffers* b, void* Y_host, void* dX_host, float* dR,
                               void* dW1g, void* dW1u, void* dW2, void* stream) {
  if (b == nullptr || X_host == nullptr || dY_host == nullptr || Y_host == nullptr || dX_host == nullptr)
    return ETR_ERR_ARG;
  ETR_TRY(etr_validate(c));
  if (!b->X_dev || !b->dY_dev || !b->Y_dev || !b->dX_dev) return ETR_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  HostStepCtx* hc = nullptr;
  ETR_TRY(host_step_ctx(&hc));
  const size_t bytes = (size_t)c->T * c->d * elem_bytes(c->dtype);
  // dY goes up on a side stream while X is copied and the forward pass runs; Y comes down on
  // another side stream while the backward pass runs.
  ETR_CUDA(cudaEventRecord(hc->start, st));
  ETR_CUDA(cudaStreamWaitEvent(hc->up, hc->start, 0));
  ETR_CUDA(cudaMemcpyAsync(b->X_dev, X_host, bytes, cudaMemcpyHostToDevice, st));
  ETR_CUDA(cudaMemcpyAsync(b->dY_dev, dY_host, bytes, cudaMemcpyHostToDevice, hc->up));
  ETR_CUDA(cudaEventRecord(hc->dy_ready, hc->up));
  ETR_TRY(etr_layer_forward(c, b->X_dev, R, W1g, W1u, W2, b, b->Y_dev, stream));
  ETR_CUDA(cudaEventRecord(hc->fwd_done, st));
  ETR_CUDA(cudaStreamWaitEvent(hc->down, hc->fwd_done, 0));
  ETR_CUDA(cudaMemcpyAsync(Y_host, b->Y_dev, bytes, cudaMemcpyDeviceToHost, hc->down));
  ETR_CUDA(cudaEventRecord(hc->y_done, hc->down));
  ETR_CUDA(cudaStreamWaitEvent(st, hc->dy_ready, 0));
  ETR_TRY(etr_layer_backward(c, b->X_dev, R, W1g, W1u, W2, b->dY_dev, b, b->dX_dev, dR, dW1g, dW1u,
                             dW2, stream));
  ETR_CUDA(cudaMemcpyAsync(dX_host, b->dX_dev, bytes, cudaMemcpyDeviceToHost, st));
  ETR_CUDA(cudaStreamWaitEvent(st, hc->y_done, 0));
  ETR_CUDA(cudaStreamSynchronize(st));
  return ETR_OK;
}

etr_status etr_layer_step_host_begin(const etr_config* c, const void* X_host, const void* dY_host,
                                     const float* R, const void* W1g, const void* W1u, const void* W2,
                                     const etr_buffers* b, const etr_host_slot* sg, int32_t slot,
                                     void* Y_host, void* dX_host, float* dR, void* dW1g, void* dW1u,
                                     void* dW2, void* stream) {
  if (b == nullptr || sg == nullptr || X_host == nullptr || dY_host == nullptr || Y_host == nullptr ||
      dX_host == nullptr || slot < 0 || slot >= ETR_HOST_SLOTS)
    return ETR_ERR_ARG;
  ETR_TRY(etr_validate(c));
  ETR_TRY(check_ptrs({sg->X_dev, sg->dY_dev, sg->Y_dev, sg->dX_dev}));
  cudaStream_t st = (cudaStream_t)stream;
  HostStepCtx* hc = nullptr;
  ETR_TRY(host_step_ctx(&hc));
  HostSlotEvents& ev = hc->slot[slot];
  const size_t bytes = (size_t)c->T * c->d * elem_bytes(c->dtype);
  // Upload stream: both inputs, X first.  The staging was last read by the backward pass of the
  // previous step on this slot (a wait on an event never recorded is a no-op).
  ETR_CUDA(cudaStreamWaitEvent(hc->up, ev.bwd_done, 0));
  ETR_CUDA(cudaMemcpyAsync(sg->X_dev, X_host, bytes, cudaMemcpyHostToDevice, hc->up));
  ETR_CUDA(cudaEventRecord(ev.x_ready, hc->up));
  ETR_CUDA(cudaMemcpyAsync(sg->dY_dev, dY_host, bytes, cudaMemcpyHostToDevice, hc->up));
  ETR_CUDA(cudaEventRecord(ev.dy_ready, hc->up));
  // Compute stream: forward once X is up and the slot's previous Y has left; backward once dY is
  // up and the slot's previous dX has left.
  ETR_CUDA(cudaStreamWaitEvent(st, ev.x_ready, 0));
  ETR_CUDA(cudaStreamWaitEvent(st, ev.y_down, 0));
  ETR_TRY(etr_layer_forward(c, sg->X_dev, R, W1g, W1u, W2, b, sg->Y_dev, stream));
  ETR_CUDA(cudaEventRecord(ev.fwd_done, st));
  ETR_CUDA(cudaStreamWaitEvent(st, ev.dy_ready, 0));
  ETR_CUDA(cudaStreamWaitEvent(st, ev.dx_down, 0));
  ETR_TRY(etr_layer_backward(c, sg->X_dev, R, W1g, W1u, W2, sg->dY_dev, b, sg->dX_dev, dR, dW1g, dW1u,
                             dW2, stream));
  ETR_CUDA(cudaEventRecord(ev.bwd_done, st));
  // Download stream: each result as soon as its pass is done.
  ETR_CUDA(cudaStreamWaitEvent(hc->down, ev.fwd_done, 0));
  ETR_CUDA(cudaMemcpyAsync(Y_host, sg->Y_dev, bytes, cudaMemcpyDeviceToHost, hc->down));
  ETR_CUDA(cudaEventRecord(ev.y_down, hc->down));
  ETR_CUDA(cudaStreamWaitEvent(hc->down, ev.bwd_done, 0));
  ETR_CUDA(cudaMemcpyAsync(dX_host, sg->dX_dev, bytes, cudaMemcpyDeviceToHost, hc->down));
  ETR_CUDA(cudaEventRecord(ev.dx_down, hc->down));
  ev.used = true;
  return ETR_OK;
}

etr_status etr_layer_step_host_wait(int32_t slot) {
  if (slot < 0 || slot >= ETR_HOST_SLOTS) return ETR_ERR_ARG;
  HostStepCtx* hc = nullptr;
  ETR_TRY(host_step_ctx(&hc));
  if (!hc->slot[slot].used) return ETR_OK;
  ETR_CUDA(cudaEventSynchronize(hc->slot[slot].dx_down));      // recorded after y_down on the same stream
  return ETR_OK;
}

etr_status etr_read_stats(const etr_stats* dev, etr_stats* host, void* stream) {
  if (dev == nullptr || host == nullptr) return ETR_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(host, dev, sizeof(etr_stats), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return ETR_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return ETR_ERR_CUDA;
  return host->error_word ? ETR_ERR_TIMEOUT : ETR_OK;
}

etr_status etr_selftest_bounded_wait(etr_stats* stats, int64_t limit_cycles, void* stream) {
  if (stats == nullptr || limit_cycles < 1 || limit_cycles > 4000000000ll) return ETR_ERR_ARG;
  if (!aligned16(stats)) return ETR_ERR_ALIGN;
  return tc_wait_selftest(stats, (long long)limit_cycles, (cudaStream_t)stream);
}

etr_status etr_read_status(const etr_stats* dev, etr_stats* host, void* stream) {
  return etr_read_stats(dev, host, stream);
}

int64_t etr_launch_count(void) { return (int64_t)g_launches.load(); }

etr_status etr_timing_enable(int on) {
  std::lock_guard<std::mutex> lk(g_timing_mu);
  for (auto& r : g_records) { g_event_pool.push_back(r.beg); g_event_pool.push_back(r.end); }
  g_records.clear();
  g_timing_on = on != 0;
  return ETR_OK;
}

int64_t etr_timing_collect(char* names, size_t names_bytes, float* ms, int64_t max_records) {
  std::lock_guard<std::mutex> lk(g_timing_mu);
  int64_t n = 0;
  size_t off = 0;
  if (names && names_bytes) names[0] = 0;
  for (auto& r : g_records) {
    if (n >= max_records) break;
    float t = -1.f;
    if (!r.beg || !r.end || cudaEventSynchronize(r.end) != cudaSuccess ||
        cudaEventElapsedTime(&t, r.beg, r.end) != cudaSuccess)
      t = -1.f;
    const size_t len = strlen(r.name);
    if (!names || off + len + 2 > names_bytes) break;
    memcpy(names + off, r.name, len);
    names[off + len] = '\n';
    names[off + len + 1] = 0;
    off += len + 1;
    if (ms) ms[n] = t;
    ++n;
  }
  for (auto& r : g_records) { g_event_pool.push_back(r.beg); g_event_pool.push_back(r.end); }
  g_records.clear();
  return n;
}

}  // extern "C"
