/*
 * libetr — forward and backward pass of an Expert-Token Resonance (ETR) MoE layer
 * (arXiv 2406.00023) on one NVIDIA B200 (sm_100a).
 *
 * Plain C ABI.  Unless a parameter says "host", every data pointer is DEVICE memory
 * owned by the caller; the library allocates no device memory.  `stream` is a
 * cudaStream_t passed as void* (NULL = default stream); every call only enqueues work
 * on it and returns without synchronising, except etr_read_stats and
 * etr_layer_step_host.
 *
 * Notation (the paper's in brackets): T tokens [s], d hidden size, D GrAP group size,
 * m = d/D pooled width, E experts [n], k experts per token [l], C per-expert capacity,
 * h FFN hidden size.
 *
 * Layouts: row-major, innermost index contiguous.
 *   X, Y, dY, dX [T,d]      R, dR [E,m] fp32        delta [T,E] fp32      Z [T,m] fp32
 *   W1g, W1u [E,h,d]        W2 [E,d,h]              (gradients: same shape; `dtype`, or fp32 with grad_fp32)
 *   Xp, O, dO, dXp [E*C_stride, d]                  G, U, H, dG, dU [E*C_stride, h]
 * C_stride = capacity rounded up to a multiple of 128.  Expert i owns rows
 * [i*C_stride, (i+1)*C_stride); the first counts[i] of them are in use.  Rows from
 * counts[i] up to the next multiple of 128 are kept zero by the library ("pad rows");
 * rows beyond that are never read or written.
 * Activations and expert weights are `dtype` (fp32 or bf16); routing tensors are fp32,
 * maps are int32.  All accumulation is fp32.
 *
 * Requirements checked on the host before anything is launched (ETR_ERR_* otherwise):
 *   d % D == 0, d % 8 == 0, h % 8 == 0, 1 <= k <= E <= 256, E <= m, 1 <= capacity,
 *   T >= 1, T*E < 2^31, data pointers 16-byte aligned and non-NULL.
 *   bf16 tensor-core path: d % 64 == 0 and h % 64 == 0 (else ETR_ERR_UNSUPPORTED).
 *
 * Errors: every function returns an etr_status.  Argument errors are reported before
 * any launch.  A launch failure maps to ETR_ERR_CUDA.  Device-side problems (a bounded
 * wait in the GEMM pipeline that ran out) never trap: the kernel records a code in
 * etr_stats.error_word, stops issuing work and returns; etr_read_stats reports it as
 * ETR_ERR_TIMEOUT.  The bound of those waits is cfg->wait_limit_cycles (default about two
 * seconds); etr_selftest_bounded_wait exercises the path on its own.
 */
#ifndef ETR_H_
#define ETR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ETR_OK = 0,
  ETR_ERR_ARG = 1,          /* NULL pointer, non-positive size, bad enum */
  ETR_ERR_SHAPE = 2,        /* sizes violate the divisibility / range rules above */
  ETR_ERR_ALIGN = 3,        /* a data pointer is not 16-byte aligned */
  ETR_ERR_WORKSPACE = 4,    /* caller-provided buffer too small */
  ETR_ERR_CUDA = 5,         /* CUDA runtime / driver call failed */
  ETR_ERR_TIMEOUT = 6,      /* a bounded device-side wait expired (see etr_stats) */
  ETR_ERR_UNSUPPORTED = 7   /* valid request the library has no kernel for */
} etr_status;

typedef enum { ETR_F32 = 0, ETR_BF16 = 1 } etr_dtype;
typedef enum { ETR_MODE_AUTO = 0, ETR_MODE_TCR = 1, ETR_MODE_ECR = 2 } etr_mode;
/* Grouped-GEMM kernel of the expert FFN.  TCGEN05: one CTA per 128 x 256 tile; TCGEN05_2CTA: a CTA
 * pair per 256 x 256 tile; TCGEN05_2CTA_WIDE: a CTA pair per 256 x 512 tile (two accumulators
 * sharing the A operand). */
typedef enum { ETR_GEMM_AUTO = 0, ETR_GEMM_SIMT = 1, ETR_GEMM_TCGEN05 = 2, ETR_GEMM_TCGEN05_2CTA = 3,
               ETR_GEMM_TCGEN05_2CTA_WIDE = 4 } etr_gemm_impl;

/* etr_layer_forward/backward on the tensor-core path can skip the token rearrangement: the first
 * FFN GEMM and the W1 weight-gradient GEMMs then fetch their token rows straight from X with TMA
 * row gathers (four rows per request, named by slot_token), and buf->Xp is neither written nor
 * read.  The stage calls are unaffected.  ETR_FUSE_AUTO lets the library choose. */
typedef enum { ETR_FUSE_AUTO = 0, ETR_FUSE_OFF = 1, ETR_FUSE_ON = 2 } etr_fuse;
/* fuse_combine: in etr_layer_forward on the tensor-core path with Top-1 token choice (k = 1, the
 * routing of the paper's efficiency runs) every token has at most one row, so the gate-weighted sum
 * of the general MoE equation has a single term and the down GEMM's epilogue writes gate * O straight
 * to the token's row of Y; the combine kernel does not run (tokens without a row get their zeros from
 * a small fill kernel).  Same bits as the separate combine.  AUTO and ON enable it wherever that
 * condition holds, OFF never; with k >= 2 or expert choice a token's rows lie in different experts'
 * tiles and the sum stays in etr_combine, whose fixed order keeps the result deterministic. */

/* Gate of a selected pair (t, i).  AFFINITY (default): the raw affinity delta_ti (the affinity-score
 * equation of "Cost-Efficient Sparse Expert-Token Affinity", whose matrix the paper also uses as the
 * gating weight).  SOFTMAX: p_ti = exp(delta_ti) / sum_j exp(delta_tj)
 * over all E experts of the token, the example gate of the general MoE equation; its backward
 * gives every expert of a routed token a gradient (a dense d delta), see etr_gate_softmax_bwd. */
typedef enum { ETR_GATE_AFFINITY = 0, ETR_GATE_SOFTMAX = 1 } etr_gate;

/* Number of kept candidates limited by the accumulated affinity ("Routing Strategy", the sentence
 * that introduces the expert-side equation: how many tokens an expert takes depends on the sum of
 * their affinity scores; "Training Strategy": that number adapts during training).  The paper gives
 * no rule, so this is a reading: walking a candidate list in descending affinity, the
 * candidate of rank j is kept while the sum of the j-1 affinities before it is still below tau (and
 * j is within the capacity C, resp. k).  EXPERT applies it to every expert's candidate tokens (both
 * modes), TOKEN to every token's experts (token choice only: a token then takes 1..k experts and
 * the unused entries of topk_idx hold -1); the flags combine.  Sums are taken on affinities
 * quantised to multiples of 2^-32 (round to nearest), as 64-bit integers, so they do not depend on
 * the order of summation.  tau = +infinity reproduces the plain selection; tau <= 0 keeps nothing. */
typedef enum { ETR_THRESHOLD_OFF = 0, ETR_THRESHOLD_EXPERT = 1, ETR_THRESHOLD_TOKEN = 2 } etr_threshold;

/* Immutable description of one layer call (host struct, passed by pointer). */
typedef struct etr_config {
  int32_t T, d, D, E, k, h;
  int32_t capacity;           /* upper bound on rows per expert, ceil(cf*T*k/E) */
  int32_t c_floor;            /* lower clamp of the adaptive bound (>= 1) */
  int32_t adaptive;           /* 0: C = capacity.  1: C = clamp(ceil(C_min), c_floor, capacity) */
  float delta_max_override;   /* < 0: use this batch's max affinity; >= 0: use this value */
  int64_t step, switch_step;  /* ETR_MODE_AUTO: token choice while step < switch_step */
  int32_t mode;               /* etr_mode */
  int32_t dtype;              /* etr_dtype of activations and expert weights */
  int32_t gemm_impl;          /* etr_gemm_impl; AUTO = CTA-pair tcgen05 for bf16, SIMT for fp32 */
  int32_t fuse_dispatch;      /* etr_fuse: token rearrangement fused into the GEMM operand fetch */
  int32_t gate_mode;          /* etr_gate: what weighs an expert's output in the combine */
  int32_t grad_fp32;          /* != 0: dW1g, dW1u, dW2 are written as fp32 (same shapes) whatever `dtype` is;
                                 0: in `dtype`.  The accumulation is fp32 either way. */
  int32_t weight_dtype;       /* etr_dtype of W1g, W1u, W2: equal to `dtype`, or ETR_F32 under dtype = ETR_BF16
                                 (fp32 master weights).  The GEMMs take both operands in one 16-bit type,
                                 so in the mixed case every call that multiplies by the weights
                                 (etr_expert_ffn, etr_expert_ffn_bwd, etr_layer_forward) first rounds them to
                                 bf16, nearest even, into the tail of ws (etr_workspace_bytes grows by
                                 3 E d h 2 bytes), dW1g, dW1u, dW2 are written as fp32 whatever grad_fp32
                                 says, and etr_layer_backward reads the copies etr_layer_forward left in
                                 buf->ws (same buffers, weights unchanged in between).  Results equal those of
                                 a bf16 layer with grad_fp32 on weights rounded beforehand, bit for bit.
                                 bf16 weights under fp32 activations: ETR_ERR_UNSUPPORTED */
  int32_t threshold_mode;     /* etr_threshold flags: selections also cut by a running sum of affinities */
  float threshold_tau;        /* ETR_THRESHOLD_EXPERT: the sum at which an expert stops taking tokens */
  float threshold_tau_token;  /* ETR_THRESHOLD_TOKEN: the sum at which a token stops taking experts */
  int64_t wait_limit_cycles;  /* bound of every device-side wait of the GEMM pipeline, in SM clock
                                 cycles; 0 = the default, about two seconds */
  int32_t fuse_combine;       /* etr_fuse: the combine folded into the down GEMM's epilogue (see below) */
  int32_t reserved0;
} etr_config;

/* Per-call scalars produced and consumed on the device (device struct, 64 bytes). */
typedef struct etr_stats {
  int32_t mode;               /* etr_mode actually used */
  int32_t C;                  /* capacity actually used */
  int32_t dropped;            /* candidate (token,expert) pairs cut by the capacity */
  int32_t unrouted;           /* tokens that ended up in no expert */
  float delta_max;            /* max affinity of this batch */
  uint32_t delta_max_key;     /* order-preserving integer image of delta_max */
  int32_t error_word;         /* 0, or a code left by a kernel that gave up a wait */
  int32_t rows_total;         /* sum of counts */
  int32_t reserved[8];
} etr_stats;

/* Routing maps (host struct of device pointers). */
typedef struct etr_route {
  int32_t* topk_idx;          /* [T,k]  token choice: experts by descending affinity; -1 in expert choice */
  int32_t* counts;            /* [E]    rows in use per expert */
  int32_t* slot_token;        /* [E*C_stride] token id held by each row, -1 if unused */
  float* gate;                /* [E*C_stride] affinity of that (token, expert) pair, 0 if unused */
  int32_t* tok_ptr;           /* [T+1]  CSR: rows of token t are tok_row[tok_ptr[t] .. tok_ptr[t+1]) */
  int32_t* tok_row;           /* [E*C_stride] row ids, ascending expert order inside a token */
} etr_route;

/* Every device buffer a forward+backward needs besides inputs, parameters and outputs
 * (host struct of device pointers).  etr_buffers_bind carves them out of one block. */
typedef struct etr_buffers {
  etr_stats* stats;
  etr_route route;
  float* delta;               /* [T,E] */
  float* Z;                   /* [T,m] pooled tokens, saved for the router gradient */
  float* xnorm;               /* [T] */
  float* rnorm;               /* [E] */
  void* Xp; void* G; void* U; void* H; void* O;          /* forward activations */
  void* dO; void* dG; void* dU; void* dXp; float* dgate; /* backward activations */
  void* ws;                   /* scratch, ws_bytes long */
  size_t ws_bytes;
  /* staging used only by etr_layer_step_host */
  void* X_dev; void* dY_dev; void* Y_dev; void* dX_dev;
  /* softmax gate only (NULL otherwise): per-token log-sum-exp [T] and the dense d delta [T,E] */
  float* lse; float* ddelta;
} etr_buffers;

const char* etr_status_string(etr_status s);

/* Checks a config against the rules in the header comment. */
etr_status etr_validate(const etr_config* cfg);

/* C_stride for a config (capacity rounded up to 128). */
int32_t etr_c_stride(const etr_config* cfg);

/* Scratch bytes the calls below need in `ws` (max over all of them). */
etr_status etr_workspace_bytes(const etr_config* cfg, size_t* bytes);

/* Size of one block holding every etr_buffers member, and the carving of such a block
 * (base must be 256-byte aligned).  with_host_staging != 0 also reserves X_dev, dY_dev,
 * Y_dev, dX_dev. */
etr_status etr_buffers_bytes(const etr_config* cfg, int with_host_staging, size_t* bytes);
etr_status etr_buffers_bind(const etr_config* cfg, int with_host_staging, void* base, size_t bytes,
                            etr_buffers* out);

/* The same carving as plain numbers, for callers that place the buffers themselves: C_stride, the
 * size of the block, and the byte offset of every etr_buffers member from a 256-byte aligned base
 * (members a config does not use have offset 0 and size 0: the host staging without
 * with_host_staging, lse and ddelta without the softmax gate).  etr_buffers_bind(base) equals
 * base + these offsets. */
typedef struct etr_layout_info {
  int32_t C_stride;
  int32_t reserved;
  size_t total_bytes, ws_bytes;
  size_t stats, topk_idx, counts, slot_token, gate, tok_ptr, tok_row;
  size_t delta, Z, xnorm, rnorm, Xp, G, U, H, O, dO, dG, dU, dXp, dgate, ws;
  size_t X_dev, dY_dev, Y_dev, dX_dev, lse, ddelta;
} etr_layout_info;
etr_status etr_layout(const etr_config* cfg, int with_host_staging, etr_layout_info* out);

/* ---- forward stages ---------------------------------------------------------------- */

/* GrAP pooling and cosine affinity ("Cost-Efficient Sparse Expert-Token Affinity": the
 * W_aff equations and delta_ti = cos(x_t, w_i)), generalised to learned embeddings:
 *   z_t = avgpool_D(x_t);  delta_ti = sqrt(D) <z_t, R_i> / (||x_t|| ||R_i||), 0 if a norm is 0.
 * Writes delta, xnorm, rnorm, optionally Z (NULL to skip), and raises
 * stats->delta_max_key to the batch maximum.  stats must have been zeroed by the caller
 * (etr_layer_forward does it) — the call only ever raises the key.
 * Arithmetic: fp32 throughout.  With Z given, E <= 64 and 32 | d/D the products <z_t, R_i> run on the
 * tensor cores as tf32 MMAs on operands split into two tf32 parts each (hi*hi + hi*lo + lo*hi in an fp32
 * accumulator: what is dropped is 2^-22 of a product), otherwise as fp32 FMAs; either way within 1e-5 of
 * the exact quotient relative to max(|delta|, rms(delta)).  A token's affinities depend on that token,
 * R and the shape (d, D, E) only, not on T or on which other tokens share the batch. */
etr_status etr_affinity(const etr_config* cfg, const void* X, const float* R, float* delta,
                        float* Z, float* xnorm, float* rnorm, etr_stats* stats, void* stream);

/* Bidirectional selection ("Routing Strategy": Top-l experts per token, then each expert
 * keeps C of its assigned tokens, highest affinity first) under the capacity
 *   C = capacity, or clamp(ceil((1/E) exp{d dm^2/(2-dm^2)}), c_floor, capacity) when adaptive
 * (Remark of "Dynamic Lower Bound Module for Expert Capacity"), dm = delta_max_override
 * or the batch maximum left in stats by etr_affinity.  Mode: cfg->mode, or from step.
 * Ties go to the lower index.  Kept tokens of an expert are stored in ascending token
 * order.  Fills every member of route and stats->{mode,C,dropped,unrouted,delta_max,
 * rows_total} (each is set by the call, not added to: selecting again on the same stats, e.g.
 * at another step of a sweep, needs no clearing in between; delta_max_key and error_word are
 * left as they are).  ws: etr_workspace_bytes. */
etr_status etr_select(const etr_config* cfg, const float* delta, etr_stats* stats,
                      const etr_route* route, void* ws, void* stream);

/* etr_select for callers that cannot allocate device memory (the paper has no counterpart;
 * this is a deployment variant of the call above, same results bit for bit).
 *
 * Some hosts of this library may not call cudaMalloc at all: code running inside another
 * framework's stream callback or memory-pool-managed region, plugins loaded into a process
 * whose device memory was fully handed to a pool at start-up, or real-time loops where an
 * allocation (an implicit device synchronisation) is forbidden.  They pass delta, stats and
 * the route outputs as usual, and the T*E 32-bit keys that etr_select keeps in `ws` live
 * instead in a fixed array inside the library image.
 *
 * Limit: T*E <= ETR_SELECT_STATIC_MAX_ENTRIES (16 MiB of keys plus 640 KiB of scan scratch,
 * enough for every workload up to T=65536, E=64); larger problems return ETR_ERR_WORKSPACE
 * and launch nothing.  Every GPU that loads the library carries those bytes until the process
 * ends.
 * The call itself allocates and frees nothing.  Its first use on a device looks up the
 * array's device address (once per device, with that device current); make that first call
 * outside any stream capture.  The address is kept for the life of the process: after a
 * cudaDeviceReset of that device it is stale, and the library must be reloaded before the call
 * is used there again.
 * All calls share the one array, which keeps whatever the previous call left in it: the
 * selection overwrites every entry it later reads, so nothing needs clearing, but two calls
 * whose kernels overlap on the same GPU (different streams, or threads) race on it — keep
 * such calls ordered. */
#define ETR_SELECT_STATIC_MAX_ENTRIES (4u * 1024u * 1024u)
etr_status etr_select_static(const etr_config* cfg, const float* delta, etr_stats* stats,
                             const etr_route* route, void* stream);

/* Token rearrangement: Xp[r,:] = X[slot_token[r],:] for rows in use, 0 for pad rows. */
etr_status etr_dispatch(const etr_config* cfg, const void* X, const etr_route* route, void* Xp,
                        void* stream);

/* Expert networks as a grouped GEMM over the rows in use (SwiGLU FFN, no bias):
 *   G = Xp W1g_i^T, U = Xp W1u_i^T, H = silu(G) * U, O = H W2_i^T   for expert i's rows.
 * G, U, H are kept for the backward pass. */
etr_status etr_expert_ffn(const etr_config* cfg, const etr_route* route, const void* Xp,
                          const void* W1g, const void* W1u, const void* W2,
                          void* G, void* U, void* H, void* O, etr_stats* stats, void* ws,
                          void* stream);

/* Gate-weighted sum of the general MoE form, MoE(x) = sum_t sum_i G_i(x_t) E_i(x_t), with
 * the affinity as the gate:  Y[t,:] = sum_{r in rows(t)} gate[r] O[r,:]  (0 if no rows). */
etr_status etr_combine(const etr_config* cfg, const etr_route* route, const void* O, void* Y,
                       void* stream);

/* ---- backward stages (the paper states no backward; these are the derivatives of the
 *      forward definitions above with the selection held constant) -------------------- */

/* dO[r,:] = gate[r] dY[t(r),:];  dgate[r] = <dY[t(r),:], O[r,:]>;  pad rows get 0. */
etr_status etr_combine_bwd(const etr_config* cfg, const etr_route* route, const void* dY,
                           const void* O, void* dO, float* dgate, void* stream);

/* dH = dO W2_i;  dG = dH*U*s*(1+G*(1-s)), dU = dH*G*s with s = sigmoid(G);
 * dXp = dG W1g_i + dU W1u_i;  dW2_i = dO^T H;  dW1g_i = dG^T Xp;  dW1u_i = dU^T Xp.
 * Experts with no rows get zero weight gradients.  dW1g, dW1u, dW2 are `dtype`, or fp32 when
 * cfg->grad_fp32 is set (the fp32 accumulators stored unrounded). */
etr_status etr_expert_ffn_bwd(const etr_config* cfg, const etr_route* route, const void* dO,
                              const void* Xp, const void* G, const void* U, const void* H,
                              const void* W1g, const void* W1u, const void* W2,
                              void* dG, void* dU, void* dXp,
                              void* dW1g, void* dW1u, void* dW2, etr_stats* stats, void* ws,
                              void* stream);

/* dX[t,:] = sum_{r in rows(t)} dXp[r,:]  (overwrites dX). */
etr_status etr_dispatch_bwd(const etr_config* cfg, const etr_route* route, const void* dXp,
                            void* dX, void* stream);

/* d delta is non-zero only on selected pairs, where it equals dgate; it is therefore
 * represented by (route, dgate) and this call only checks its arguments. */
etr_status etr_select_bwd(const etr_config* cfg, const etr_route* route, const float* dgate);

/* Router gradient.  With a = ||x_t||, b = ||R_i||, c = sqrt(D)/(a b), over selected pairs:
 *   dX[t,q] += sum_i dgate_ti ( c R_i[q/D]/D - delta_ti x_t[q]/a^2 )      (ADDS to dX)
 *   dR[i,j]  = sum_t dgate_ti ( c z_t[j]     - delta_ti R_i[j]/b^2 )      (overwrites dR)
 * ws: etr_workspace_bytes. */
etr_status etr_affinity_bwd(const etr_config* cfg, const void* X, const float* R,
                            const float* delta, const float* Z, const float* xnorm,
                            const float* rnorm, const etr_route* route, const float* dgate,
                            void* dX, float* dR, void* ws, void* stream);

/* ---- softmax-gate variant and load statistics --------------------------------------------- */

/* Softmax gate (the Softmax example of the gating weight in the general MoE equation): replaces
 * route->gate[r] of every row in use by p_ti = exp(delta_ti - lse[t]) with
 * lse[t] = log sum_j exp(delta_tj) over all E experts, and writes lse [T].  Call after etr_select;
 * rows not in use keep gate 0. */
etr_status etr_gate_softmax(const etr_config* cfg, const float* delta, const etr_route* route,
                            float* lse, void* stream);

/* Its backward (calculus; the paper has none): with g_tj = dgate of the row of pair (t, j) if the
 * pair is selected and 0 otherwise, and s_t = sum_j g_tj p_tj,
 *   ddelta[t][j] = p_tj (g_tj - s_t)   for every expert j;  rows of tokens without a row are 0.
 * ddelta is [T,E] fp32; route->gate must still hold the softmax gates. */
etr_status etr_gate_softmax_bwd(const etr_config* cfg, const float* delta, const float* lse,
                                const etr_route* route, const float* dgate, float* ddelta,
                                void* stream);

/* etr_affinity_bwd for a dense d delta [T,E] (what etr_gate_softmax_bwd produces): same outputs,
 * dX accumulated into, dR overwritten; `route` is read only to skip tokens without rows.
 * ws: etr_workspace_bytes of a config whose gate_mode is ETR_GATE_SOFTMAX. */
etr_status etr_affinity_bwd_dense(const etr_config* cfg, const void* X, const float* R,
                                  const float* delta, const float* Z, const float* xnorm,
                                  const float* rnorm, const etr_route* route, const float* ddelta,
                                  void* dX, float* dR, void* ws, void* stream);

/* Load statistics, the inputs of the auxiliary and locality losses ("Locality Loss"), which are
 * not part of the layer: load[i] = counts[i] / T, the share of the batch's tokens expert i
 * processes, and gate_mean[i] = (sum of the gates of expert i's rows) / T.  Both [E] fp32. */
etr_status etr_load_stats(const etr_config* cfg, const etr_route* route, float* load,
                          float* gate_mean, void* stream);

/* ---- whole layer ---------------------------------------------------------------------- */

/* Zeroes stats, then affinity, select, (gate_softmax,) dispatch, expert_ffn, combine, in that
 * order. */
etr_status etr_layer_forward(const etr_config* cfg, const void* X, const float* R,
                             const void* W1g, const void* W1u, const void* W2,
                             const etr_buffers* buf, void* Y, void* stream);

/* combine_bwd, expert_ffn_bwd, dispatch_bwd, affinity_bwd, in that order, on the buffers
 * a preceding etr_layer_forward filled.  The last two run as one fused kernel (dX is written
 * once, with the row sum kept in fp32 until the router term has been added). */
etr_status etr_layer_backward(const etr_config* cfg, const void* X, const float* R,
                              const void* W1g, const void* W1u, const void* W2,
                              const void* dY, const etr_buffers* buf,
                              void* dX, float* dR, void* dW1g, void* dW1u, void* dW2,
                              void* stream);

/* One training step from HOST activations: copies X_host and dY_host (host, ideally pinned)
 * to buf->X_dev / dY_dev, runs forward and backward, copies Y and dX back to Y_host and
 * dX_host (host), and synchronises the stream.  Parameters and their gradients stay on
 * the device.  buf must have been bound with host staging.  The copy of dY overlaps the
 * forward pass and the copy of Y overlaps the backward pass, on two side streams the
 * library creates once per device (host-side objects; still no device allocation). */
etr_status etr_layer_step_host(const etr_config* cfg, const void* X_host, const void* dY_host,
                               const float* R, const void* W1g, const void* W1u, const void* W2,
                               const etr_buffers* buf, void* Y_host, void* dX_host,
                               float* dR, void* dW1g, void* dW1u, void* dW2, void* stream);

/* Device staging of one host step in flight: four caller-owned device buffers of T*d elements of
 * `dtype` each (16-byte aligned). */
typedef struct etr_host_slot { void* X_dev; void* dY_dev; void* Y_dev; void* dX_dev; } etr_host_slot;
#define ETR_HOST_SLOTS 4

/* Pipelined form of etr_layer_step_host for a loop of steps: enqueues the same work and returns
 * without waiting, so the next step's host-to-device copies run under this step's kernels and this
 * step's device-to-host copies under the next step's.  Steps in flight at the same time use
 * different `slot`s (index 0 .. ETR_HOST_SLOTS-1, each with its own staging); two slots already keep
 * both copy directions busy.  The layer's internal buffers `buf` are shared: the kernels of
 * successive steps run in call order on `stream`, only the copies overlap them.  Re-using a slot
 * index orders the new step after the previous use of that slot on the device; the HOST buffers of
 * a step (all four) belong to the library until etr_layer_step_host_wait(slot) has returned.
 * dR and the weight gradients are those of the most recent step once `stream` is idle. */
etr_status etr_layer_step_host_begin(const etr_config* cfg, const void* X_host, const void* dY_host,
                                     const float* R, const void* W1g, const void* W1u, const void* W2,
                                     const etr_buffers* buf, const etr_host_slot* staging, int32_t slot,
                                     void* Y_host, void* dX_host, float* dR,
                                     void* dW1g, void* dW1u, void* dW2, void* stream);

/* Blocks the calling thread until the last step begun on `slot` has delivered Y_host and dX_host
 * (ETR_OK at once if nothing was begun on it). */
etr_status etr_layer_step_host_wait(int32_t slot);

/* Copies the device stats to the host and synchronises the stream.  Returns
 * ETR_ERR_TIMEOUT if a kernel recorded an expired wait. */
etr_status etr_read_stats(const etr_stats* stats_dev, etr_stats* stats_host, void* stream);
/* The same call under the name the status word suggests. */
etr_status etr_read_status(const etr_stats* stats_dev, etr_stats* stats_host, void* stream);

/* Self-test of the bounded device-side wait (the failure path of the GEMM pipeline, which a healthy
 * run never takes): launches one warp that waits, with the pipeline's own wait routine, on a
 * barrier nothing will ever arrive on.  After limit_cycles SM clock cycles (1 .. 4e9; 1e5 is about
 * 50 microseconds) the wait gives up, the kernel writes a code to stats->error_word and returns
 * normally; etr_read_stats then reports ETR_ERR_TIMEOUT and the stream and context stay usable.
 * Nothing else is in flight in that kernel: no copy, no tensor memory.  The caller clears
 * error_word (etr_layer_forward does) before the next ordinary use of `stats`. */
etr_status etr_selftest_bounded_wait(etr_stats* stats, int64_t limit_cycles, void* stream);

/* Number of kernels launched by this library in the calling process so far. */
int64_t etr_launch_count(void);

/* Per-kernel timing for benchmarks.  While enabled, every kernel the library launches is
 * bracketed by a CUDA event pair recorded on the launch stream (host-side objects; no
 * device memory).  etr_timing_enable clears earlier records.  etr_timing_collect waits for
 * the recorded events, writes up to max_records kernel names into `names` (host, one per
 * line, NUL-terminated) and their durations in milliseconds into `ms` (host; -1 where the
 * time could not be read), clears the records and returns how many it wrote. */
etr_status etr_timing_enable(int on);
int64_t etr_timing_collect(char* names, size_t names_bytes, float* ms, int64_t max_records);

#ifdef __cplusplus
}
#endif
#endif /* ETR_H_ */
