/*
 * unipool.h - C ABI of the B200 (sm_100a) UniPool MoE-layer library.
 *
 * One globally shared pool of M SwiGLU expert FFNs is reached by every one of
 * the L transformer layers through that layer's own NormRouter (paper Sec. 4).
 * The calls below are the steps of one layer's forward and backward pass plus
 * the pool-level balance loss.  The layer-private layout of Eq. 1 runs through
 * the same calls with a pool view (expert_base, n_experts) per layer.
 *
 * Conventions (all calls)
 *   - Return value: 0 on success, a negative UNIPOOL_ERR_* code otherwise.
 *     Arguments are checked on the host before anything is launched; a CUDA
 *     or driver error met later in a call that issues several kernels leaves
 *     the earlier ones queued.  unipool_last_error() gives the message of the
 *     calling thread's last failure.
 *   - Every tensor pointer is a DEVICE pointer owned by the caller; the library
 *     never allocates or frees device memory.  Scratch lives in the workspace
 *     the caller hands to unipool_create().
 *   - Activations and pool weights have the element type of the context:
 *     float (UNIPOOL_FP32) or bf16 (UNIPOOL_BF16, fp32 accumulation).  Gates,
 *     logits, statistics, router weights and all weight gradients are float.
 *   - Tensors are dense row-major; shapes are written [rows, cols].
 *   - Calls are asynchronous on `stream` and never synchronise the host: group
 *     sizes stay on the device.  Calls of one context must be issued on one
 *     stream at a time (they share the workspace).
 *   - Arguments marked "+=" accumulate into what the buffer holds.
 *
 * Permuted ("expert-contiguous") row space
 *   A layer's T*k (token, slot) assignments are sorted by expert, token-major
 *   inside an expert.  Group e starts at offsets[e], a multiple of
 *   UNIPOOL_ROW_ALIGN rows; rows between the end of a group and the next start
 *   are pad rows and hold zeros in every permuted buffer.  Buffers in this
 *   space have unipool_row_capacity() rows; rows >= offsets[n_experts] are
 *   never touched.
 */
#ifndef UNIPOOL_H_
#define UNIPOOL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define UNIPOOL_OK                    0
#define UNIPOOL_ERR_INVALID_ARG      -1
#define UNIPOOL_ERR_UNSUPPORTED      -2   /* shape outside the supported set          */
#define UNIPOOL_ERR_WORKSPACE        -3   /* workspace missing or too small           */
#define UNIPOOL_ERR_CUDA             -4   /* a CUDA runtime/driver call failed        */
#define UNIPOOL_ERR_TIMEOUT          -5   /* a bounded device-side wait ran out       */
#define UNIPOOL_ERR_DEVICE_CHECK     -6   /* a device-side consistency check failed   */

#define UNIPOOL_FP32 0
#define UNIPOOL_BF16 1

/* router_mode of a context */
#define UNIPOOL_ROUTER_NORM    0      /* NormRouter, Eq. 7                          */
#define UNIPOOL_ROUTER_SOFTMAX 1      /* softmax over the router's experts: the     */
                                      /* conventional router of the baselines in    */
                                      /* Sec. 5.1 and of the ablation of Sec. 5.3   */

#define UNIPOOL_ROW_ALIGN 128         /* group starts in the permuted row space    */
#define UNIPOOL_MAX_EXPERTS 512
#define UNIPOOL_MAX_TOPK 8

/* expert_bwd flags */
#define UNIPOOL_BWD_DEFAULT     0
#define UNIPOOL_BWD_SKIP_WGRAD  1     /* leave dW to a later unipool_pool_wgrad     */
#define UNIPOOL_WGRAD_OVERWRITE 2     /* dW of the experts in the view is written,  */
                                      /* not added to: the first contribution of a  */
                                      /* step needs no zeroed buffer and no read    */

typedef struct unipool_ctx unipool_ctx;
typedef void* unipool_stream;         /* a cudaStream_t                            */

/* Shape of one stack of MoE layers.  Supported: d_model % 64 == 0,
 * d_ff % 64 == 0, 1 <= top_k <= 8, top_k <= experts seen by a router,
 * pool_size <= 512, max_tokens * top_k < 2^30. */
typedef struct {
  int32_t d_model;      /* d                                                     */
  int32_t d_ff;         /* f, width of one SwiGLU expert                         */
  int32_t pool_size;    /* M, experts in the shared pool                         */
  int32_t top_k;        /* k                                                     */
  int32_t n_layers;     /* L, layers that route into the pool                    */
  int32_t max_tokens;   /* largest T of any call                                 */
  int32_t dtype;        /* UNIPOOL_FP32 or UNIPOOL_BF16                          */
  float   eps;          /* epsilon of Eq. 7                                      */
  float   c;            /* calibration constant c of Eq. 7 (Alg. 1)              */
  int32_t router_mode;  /* UNIPOOL_ROUTER_NORM or UNIPOOL_ROUTER_SOFTMAX         */
} unipool_config;

/* Rows a permuted buffer must have: max_tokens*top_k + pool_size*(ROW_ALIGN-1),
 * rounded up to ROW_ALIGN.  Host function; returns 0 on a NULL config. */
int64_t unipool_row_capacity(const unipool_config* cfg);

/* Bytes of device scratch unipool_create() needs for this config (host function). */
size_t unipool_workspace_bytes(const unipool_config* cfg);

/* Validates cfg, records the workspace (device memory, 256-byte aligned, at
 * least unipool_workspace_bytes(cfg), owned by the caller and alive until
 * unipool_destroy) and clears it on `stream`.  *out receives a host object. */
int unipool_create(unipool_ctx** out, const unipool_config* cfg, void* workspace,
                   size_t workspace_bytes, unipool_stream stream);
int unipool_destroy(unipool_ctx* ctx);

/* Message of the calling thread's last failed call ("" if none). */
const char* unipool_last_error(void);

/* Reads the context's device status word (the one call that synchronises
 * `stream`).  Returns UNIPOOL_OK, UNIPOOL_ERR_TIMEOUT or
 * UNIPOOL_ERR_DEVICE_CHECK and clears the word.
 * Debug mode: when the environment holds UNIPOOL_DEBUG=1 at the first call
 * into the library, every region of the workspace is followed by a 256-byte
 * guard band (unipool_workspace_bytes() grows by 256 per region) filled by
 * unipool_create(); this call first compares the bands with their fill (one
 * small launch on `stream`) and reports an altered one as
 * UNIPOOL_ERR_DEVICE_CHECK, unipool_last_error() naming the region.  The
 * paper has no counterpart: a development aid. */
int unipool_check_status(unipool_ctx* ctx, unipool_stream stream);

/* NormRouter scoring and top-k of one layer (Eq. 7; Sec. 4.3 "Top-k selection").
 *   z = x W_r^T (+ bias);  n_t = ||z_t||_2 over all n_experts logits;
 *   s = sigma * c * max(0, z / (n + eps));  idx = k highest s, descending,
 *   ties to the lowest expert index;  gate = s[idx] (not renormalised).
 * in : x [T,d] (ctx dtype); W_r [n_experts,d] float; sigma; bias [n_experts]
 *      float or NULL; n_experts = experts this router scores (M for the shared
 *      pool, the private count for the layout of Eq. 1).
 * out: idx [T,k] int32; gate [T,k] float; counts [n_experts] int32 (assignments
 *      per expert); score_sum [n_experts] float (sum over tokens of s, the
 *      numerator of P_i in Eq. 3); znorm [T] float; z_saved [T,n_experts] float
 *      (logits, kept for unipool_route_bwd).  All outputs are overwritten.
 * A context of router_mode UNIPOOL_ROUTER_SOFTMAX scores with
 *   s = exp(z - max z) / sum_j exp(z_j - max z)
 * instead (sigma, c and eps play no part) and stores log sum_j exp(z_j) in
 * znorm; selection, gates and statistics are taken from s in the same way. */
int unipool_route(unipool_ctx* ctx, const void* x, int32_t T, const float* W_r, float sigma,
                  const float* bias, int32_t n_experts, int32_t* idx, float* gate,
                  int32_t* counts, float* score_sum, float* znorm, float* z_saved,
                  unipool_stream stream);

/* Optional set-up of the routers of a bf16 context, once per parameter update.  unipool_route and
 * unipool_route_bwd compute the fp32 logits of Eq. 7 on the tensor cores from three bf16 terms of the
 * fp32 router weights (W = W0 + W1 + W2, every product exact in fp32).  Without this call each of them
 * splits the W_r it is given on every call.  With it the terms of all n_layers routers
 * (W_r [n_layers, n_experts, d], contiguous) are formed by one kernel and kept in the workspace: a
 * later route / route_bwd call whose W_r points at one of these layers (W_r + l*n_experts*d) uses
 * them.  They are a copy: call again after the weights change; n_layers = 0 forgets them.  A context
 * of dtype UNIPOOL_FP32 ignores the call.  n_layers <= config.n_layers. */
int unipool_router_prepare(unipool_ctx* ctx, const float* W_r, int32_t n_layers, int32_t n_experts,
                           unipool_stream stream);

/* Token permute into expert-contiguous order (the grouped layout behind
 * Table 7's "Grouped GEMM"; Eq. 2 evaluates every selected expert, nothing is
 * dropped).  Stable: rows of one expert keep token-major order.
 * in : x [T,d]; idx [T,k].
 * out: offsets [n_experts+1] int32 (group starts, multiples of ROW_ALIGN;
 *      offsets[n_experts] = rows in use); row_of [T,k] int32 (row of each
 *      assignment); token_of [row_capacity] int32 (token of each row, -1 on pad
 *      rows and beyond); tile_expert [row_capacity/ROW_ALIGN] int32 (expert of
 *      each ROW_ALIGN-row tile, -1 beyond); Xp [row_capacity,d] (ctx dtype; rows
 *      below offsets[n_experts] written, pad rows zero). */
int unipool_dispatch(unipool_ctx* ctx, const void* x, int32_t T, const int32_t* idx,
                     int32_t n_experts, int32_t* offsets, int32_t* row_of, int32_t* token_of,
                     int32_t* tile_expert, void* Xp, unipool_stream stream);

/* unipool_dispatch for callers that cannot hand over a workspace (the paper has no counterpart).
 * Some embedders of this library run where device allocation is off limits: inside a
 * memory-planned runtime whose arena is fixed before the first step, or in a plugin that only
 * receives the tensors of one call.  They cannot size and allocate the context's workspace, so
 * this call needs none and no unipool_ctx: the per-chunk histograms the permutation kernels use as
 * scratch live in a 2 MiB array inside the library's own device image (each GPU that loads the
 * library holds it until the process exits).  The call itself never allocates or frees memory.
 * Same inputs, outputs and results as unipool_dispatch, for d_model/dtype/top_k given here and
 * row_capacity = rows of the permuted buffers (a multiple of UNIPOOL_ROW_ALIGN, at least
 * T*top_k + n_experts*(UNIPOOL_ROW_ALIGN-1) rounded up).
 *   - Limit: ceil(T/256) * n_experts <= 524224 (e.g. 261888 tokens at 512 experts); beyond it the
 *     call fails with UNIPOOL_ERR_WORKSPACE and launches nothing.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents; the kernels
 *     rewrite every entry they read, so nothing needs clearing.  Two calls that overlap on the
 *     GPU (different streams) race on it: serialise them.
 *   - An expert index outside [0, n_experts) is dropped (its row_of entry is -1); without a
 *     context there is no status word to report it through.
 *   - Host threads may call concurrently (the per-device look-up is published atomically), but each
 *     call must be made with the device current whose memory the pointers and `stream` belong to:
 *     the array's address is looked up for the CURRENT device. */
int unipool_dispatch_static(const void* x, int32_t T, int32_t d_model, int32_t dtype, int32_t top_k,
                            const int32_t* idx, int32_t n_experts, int64_t row_capacity,
                            int32_t* offsets, int32_t* row_of, int32_t* token_of,
                            int32_t* tile_expert, void* Xp, unipool_stream stream);

/* Grouped SwiGLU expert FFN over the permuted rows (Eq. 2's e_i; App. B):
 *   GU = Xp [W_gate; W_up]^T,  A = silu(G) * U,  Yp = A W_down^T   per group,
 * group e using pool expert expert_base + e.
 * in : Xp [cap,d]; offsets; tile_expert; W_gu [M,2f,d] (rows 0..f-1 of an expert
 *      are W_gate, rows f..2f-1 W_up); W_down [M,d,f]  (ctx dtype).
 * out: GU [cap,2f] (G in columns 0..f-1, U in f..2f-1), A [cap,f], Yp [cap,d]
 *      (ctx dtype; Yp is NOT scaled by the gate).  Kept by the caller for backward. */
int unipool_expert_fwd(unipool_ctx* ctx, const void* Xp, const int32_t* offsets,
                       const int32_t* tile_expert, const void* W_gu, const void* W_down,
                       int32_t expert_base, int32_t n_experts, void* GU, void* A, void* Yp,
                       unipool_stream stream);

/* Gate-weighted combine (Eq. 2): y_t = sum_j gate[t,j] * Yp[row_of[t,j]], summed in
 * fp32 and rounded once; with residual != NULL the output is residual + y (the
 * residual block x_{l+1} = x_l + FFN_l(x_l)).
 * in : Yp [cap,d]; row_of [T,k]; gate [T,k]; residual [T,d] or NULL.  out: y [T,d]. */
int unipool_combine(unipool_ctx* ctx, const void* Yp, const int32_t* row_of, const float* gate,
                    int32_t T, const void* residual, void* y, unipool_stream stream);

/* Backward of combine + expert FFN + permute (derivative of Eq. 2).  With
 * dYp[row(t,j)] = gate[t,j] * dy_t:
 *   dgate[t,j] = <dy_t, Yp[row(t,j)]>
 *   dA = dYp W_down,  dG = dA * U * silu'(G),  dU = dA * silu(G),
 *   dXp = [dG dU] [W_gate; W_up],  dx_t = sum_j dXp[row(t,j)] (+ dx_residual_t)
 *   dW_down[e] += dYp_e^T A_e,   dW_gu[e] += [dG dU]_e^T Xp_e
 * The weight-gradient buffers are the SAME for every layer of a shared pool:
 * each shared expert accumulates the gradient of all L layers (Sec. 3).
 * in : dy [T,d]; row_of, gate, token_of, offsets, tile_expert of the forward
 *      pass; Xp, GU, A, Yp saved by the forward pass; W_gu, W_down;
 *      dx_residual [T,d] or NULL.
 * scratch/out: dYp [cap,d], dGU [cap,2f] (ctx dtype; caller-owned, overwritten;
 *      they are the operands a deferred unipool_pool_wgrad needs).
 * out: dx [T,d] (ctx dtype, overwritten); dgate [T,k] float (overwritten);
 *      dW_gu [M,2f,d] float +=; dW_down [M,d,f] float += (skipped when flags has
 *      UNIPOOL_BWD_SKIP_WGRAD, the pointers may then be NULL; with
 *      UNIPOOL_WGRAD_OVERWRITE the slices of experts expert_base ..
 *      expert_base+n_experts-1 are overwritten, zeros for an expert without rows). */
int unipool_expert_bwd(unipool_ctx* ctx, const void* dy, int32_t T, const int32_t* row_of,
                       const float* gate, const int32_t* token_of, const int32_t* offsets,
                       const int32_t* tile_expert, const void* Xp, const void* GU, const void* A,
                       const void* Yp, const void* W_gu, const void* W_down, int32_t expert_base,
                       int32_t n_experts, const void* dx_residual, void* dYp, void* dGU, void* dx,
                       float* dgate, float* dW_gu, float* dW_down, int32_t flags,
                       unipool_stream stream);

/* Weight gradients of n_layers layers in one pass: for every pool expert the
 * rows of all the given layers are contracted together, so the fp32 pool
 * gradient is read and written once instead of once per layer (same result as
 * the per-layer accumulation of unipool_expert_bwd up to summation order).
 * The per-layer operands are slices of stacked buffers: layer l's Xp is
 * Xp + l*layer_stride_rows*d elements, likewise A, dYp, dGU; offsets is
 * [n_layers, n_experts+1].  flags: 0 (dW +=) or UNIPOOL_WGRAD_OVERWRITE (dW =).
 * One of dW_gu, dW_down may be NULL: only the other product is then computed
 * (its operands alone are read), e.g. to start exchanging dW_down between
 * data-parallel replicas while dW_gu is still being computed. */
int unipool_pool_wgrad(unipool_ctx* ctx, int32_t n_layers, int64_t layer_stride_rows,
                       const int32_t* offsets, const void* Xp, const void* A, const void* dYp,
                       const void* dGU, int32_t expert_base, int32_t n_experts, float* dW_gu,
                       float* dW_down, int32_t flags, unipool_stream stream);

/* Pool-level balance loss (Eqs. 4-5; Eq. 3 when L = 1):
 *   f^(l) = counts^(l) / (T k),  P^(l) = score_sum^(l) / T,  fbar, Pbar = means over l,
 *   loss = alpha * n_experts * sum_i fbar_i Pbar_i.
 * fbar_prev != NULL replaces fbar in the loss (one-step-behind scheme, App. G).
 * in : counts [L,n_experts] int32; score_sum [L,n_experts] float.
 * out: loss (device float); dscore_coef [n_experts] float = alpha*n_experts*fbar_i/(L*T),
 *      the derivative of the loss w.r.t. every score s^(l)_{t,i} (only P carries
 *      gradient); fbar_out [n_experts] float (this batch's fbar). */
int unipool_pool_aux_loss(unipool_ctx* ctx, const int32_t* counts, const float* score_sum,
                          int32_t L, int32_t n_experts, int32_t T, float alpha,
                          const float* fbar_prev, float* loss, float* dscore_coef,
                          float* fbar_out, unipool_stream stream);

/* Backward of the NormRouter (derivative of Eq. 7 and of z = W_r x).  With
 * ds[t,i] = dscore_coef[i] + sum_{j: idx[t,j]=i} dgate[t,j], u = max(z,0),
 * q_t = sum_i ds u:
 *   dz[t,m] = sigma c ( 1{z_m>0} ds_m/(n+eps) - z_m q_t / (n (n+eps)^2) )   (0 if n = 0)
 *   dsigma += c sum ds u/(n+eps);  dW_r += dz^T x;  dx += dz W_r.
 * in : x [T,d]; W_r; sigma; znorm, z_saved, idx from unipool_route; dgate [T,k];
 *      dscore_coef [n_experts] or NULL.
 * out: dx [T,d] (ctx dtype) +=; dW_r [n_experts,d] float +=; dsigma (device float) +=.
 * With router_mode UNIPOOL_ROUTER_SOFTMAX: s = exp(z - znorm) (znorm holds the
 * log-sum-exp), q_t = sum_i ds s, dz[t,m] = s_m (ds_m - q_t); dsigma is left as it is. */
int unipool_route_bwd(unipool_ctx* ctx, const void* x, int32_t T, const float* W_r, float sigma,
                      int32_t n_experts, const float* znorm, const float* z_saved,
                      const int32_t* idx, const float* dgate, const float* dscore_coef,
                      void* dx, float* dW_r, float* dsigma, unipool_stream stream);

/* Distinct-expert accounting (App. E): U(x) = |{ e_l(x) : l = 1..L }|, the number of different pool
 * experts a token selects over all layers (the paper states it for top-1; with top-k every selected
 * expert of every layer counts).  With the shared pool 1 <= U <= min(M, L k); with private experts
 * (expert_base[l] = first pool expert of layer l) U = L k.
 * in : idx [L,T,k] int32 (the routers' indices of all layers, stacked); expert_base [L] int32 or NULL
 *      (= 0 for every layer).  Ids outside the pool are ignored.
 * out: unique [T] int32; total (device uint64) = sum over tokens of U(x) (mean = total / T). */
int unipool_unique_experts(unipool_ctx* ctx, const int32_t* idx, const int32_t* expert_base, int32_t L,
                           int32_t T, int32_t* unique, uint64_t* total, unipool_stream stream);

/* Monte-Carlo estimate of the NormRouter constant c (Alg. 1):
 *   c = E[ 1 / ||top-k(ReLU(x/||x||_2))||_2 ],  x ~ N(0, I_E),
 * over n_samples draws of a counter-based generator seeded by `seed`; draws
 * with no positive component are skipped.  Runs on the device, synchronises
 * `stream`, writes the estimate to the HOST float *c_out. */
int unipool_calibrate_c(unipool_ctx* ctx, int32_t n_experts, int32_t top_k, int32_t n_samples,
                        uint64_t seed, float* c_out, unipool_stream stream);

/* Self-test of the bounded device-side waits (a diagnostic; the paper has no counterpart).  Every
 * pipeline of the library waits on its barriers for a bounded time and reports an expired wait through
 * the status word instead of hanging.  This call launches one thread that waits, for at most
 * limit_cycles SM cycles (0 .. 2e9), on a barrier nobody arrives on: the wait gives up, the kernel
 * returns normally, and the next unipool_check_status returns UNIPOOL_ERR_TIMEOUT and clears the word.
 * The context stays usable. */
int unipool_selftest_wait(unipool_ctx* ctx, int64_t limit_cycles, unipool_stream stream);

/* Per-phase device timing (a measurement aid; the paper has no counterpart).
 * While enabled, every call brackets each of its kernel phases with CUDA events
 * on the call's stream.  unipool_profile_read synchronises those events, adds the
 * elapsed milliseconds and kernel-launch counts per phase into ms[] / launches[]
 * (host arrays of UNIPOOL_N_PHASES entries, overwritten) and forgets them. */
enum {
  UNIPOOL_PH_ROUTE_LOGITS = 0, UNIPOOL_PH_ROUTE_SELECT, UNIPOOL_PH_DISPATCH_MAPS,
  UNIPOOL_PH_DISPATCH_GATHER, UNIPOOL_PH_EXPERT_FWD_GU, UNIPOOL_PH_EXPERT_FWD_DOWN,
  UNIPOOL_PH_COMBINE, UNIPOOL_PH_POOL_AUX, UNIPOOL_PH_BWD_SCALE_GATHER, UNIPOOL_PH_BWD_DGATE,
  UNIPOOL_PH_DGRAD_DOWN, UNIPOOL_PH_DGRAD_GU, UNIPOOL_PH_WGRAD_DOWN, UNIPOOL_PH_WGRAD_GU,
  UNIPOOL_PH_UNPERMUTE_SUM, UNIPOOL_PH_ROUTE_BWD_DZ, UNIPOOL_PH_ROUTE_BWD_DX,
  UNIPOOL_PH_ROUTE_BWD_DW, UNIPOOL_N_PHASES
};
int unipool_profile_enable(unipool_ctx* ctx, int32_t on);
int unipool_profile_read(unipool_ctx* ctx, double* ms, int64_t* launches);

#ifdef __cplusplus
}
#endif
#endif  /* UNIPOOL_H_ */
