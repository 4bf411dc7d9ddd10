// C-ABI entry points: argument validation, context, workspace, error strings.
// Every compute step is a CUDA kernel in one of the other translation units.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "common.cuh"

namespace unipool {

static thread_local char g_error[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_error, sizeof(g_error), fmt, ap);
  va_end(ap);
}

static bool use_tensor_cores(const unipool_ctx* ctx) { return ctx->cfg.dtype == UNIPOOL_BF16; }

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// UNIPOOL_DEBUG=1 in the environment (read once per process): guard bands behind the workspace regions
static bool debug_enabled() {
  static const bool on = [] {
    const char* v = getenv("UNIPOOL_DEBUG");
    return v != nullptr && v[0] == '1' && v[1] == '\0';
  }();
  return on;
}

static int64_t row_capacity_of(const unipool_config& c) {
  int64_t rows = (int64_t)c.max_tokens * c.top_k + (int64_t)c.pool_size * (UNIPOOL_ROW_ALIGN - 1);
  return (rows + UNIPOOL_ROW_ALIGN - 1) / UNIPOOL_ROW_ALIGN * UNIPOOL_ROW_ALIGN;
}

Workspace carve_workspace(const unipool_config& cfg, void* base) {
  Workspace w{};
  size_t off = 0;
  char* p = static_cast<char*>(base);
  const bool guarded = debug_enabled();
  auto take = [&](size_t bytes) {
    char* q = p ? p + off : nullptr;
    off += align_up(bytes, 256);
    if (guarded && w.n_guards < 16) {
      w.guards[w.n_guards++] = p ? p + off : nullptr;
      off += kGuardBytes;
    }
    return q;
  };
  const size_t eb = cfg.dtype == UNIPOOL_BF16 ? 2 : 4;
  const int64_t cap = row_capacity_of(cfg);
  const int64_t blocks = ((int64_t)cfg.max_tokens + kDispatchMinChunkTokens - 1) / kDispatchMinChunkTokens;
  w.status = reinterpret_cast<int32_t*>(take(4 * sizeof(int32_t)));
  w.route_counts = reinterpret_cast<int32_t*>(take(UNIPOOL_MAX_EXPERTS * sizeof(int32_t)));
  w.route_sums = reinterpret_cast<double*>(take(UNIPOOL_MAX_EXPERTS * sizeof(double)));
  w.tickets = reinterpret_cast<uint32_t*>(take(8 * sizeof(uint32_t)));
  w.dsigma_acc = reinterpret_cast<double*>(take(2 * sizeof(double)));
  w.split_any = reinterpret_cast<int32_t*>(take((size_t)(cfg.n_layers + 1) * 4 * sizeof(int32_t)));
  w.block_hist = reinterpret_cast<int32_t*>(take((size_t)blocks * UNIPOOL_MAX_EXPERTS * sizeof(int32_t)));
  {
    const size_t mp = ((size_t)cfg.pool_size + 63) / 64 * 64;
    const size_t per_token = cfg.dtype == UNIPOOL_BF16 ? mp * 2 : (size_t)cfg.pool_size * sizeof(float);
    w.dz = reinterpret_cast<float*>(take((size_t)cfg.max_tokens * per_token));
  }
  w.w_split = cfg.dtype == UNIPOOL_BF16
                  ? take((size_t)(cfg.n_layers + 1) * 3 * cfg.pool_size * cfg.d_model * 2) : nullptr;
  {
    const size_t tiles = 2 * (((size_t)cfg.max_tokens + 255) / 256);   // CTAs of the router: whole pairs
    w.part_counts = reinterpret_cast<int32_t*>(take(tiles * cfg.pool_size * sizeof(int32_t)));
    w.part_sums = reinterpret_cast<float*>(take(tiles * cfg.pool_size * sizeof(float)));
    w.part_dsigma = reinterpret_cast<float*>(take((((size_t)cfg.max_tokens + 63) / 64) * sizeof(float)));
  }
  w.dXp = take((size_t)cap * cfg.d_model * eb);
  w.bytes = off;
  return w;
}

static int validate_config(const unipool_config* c) {
  UP_REQUIRE(c != nullptr, UNIPOOL_ERR_INVALID_ARG, "config is NULL");
  UP_REQUIRE(c->dtype == UNIPOOL_FP32 || c->dtype == UNIPOOL_BF16, UNIPOOL_ERR_INVALID_ARG,
             "dtype must be UNIPOOL_FP32 or UNIPOOL_BF16, got %d", c->dtype);
  UP_REQUIRE(c->d_model > 0 && c->d_model % 64 == 0, UNIPOOL_ERR_UNSUPPORTED,
             "d_model must be a positive multiple of 64, got %d", c->d_model);
  UP_REQUIRE(c->d_ff > 0 && c->d_ff % 64 == 0, UNIPOOL_ERR_UNSUPPORTED,
             "d_ff must be a positive multiple of 64, got %d", c->d_ff);
  UP_REQUIRE(c->pool_size >= 1 && c->pool_size <= UNIPOOL_MAX_EXPERTS, UNIPOOL_ERR_UNSUPPORTED,
             "pool_size must be in [1,%d], got %d", UNIPOOL_MAX_EXPERTS, c->pool_size);
  UP_REQUIRE(c->top_k >= 1 && c->top_k <= UNIPOOL_MAX_TOPK && c->top_k <= c->pool_size,
             UNIPOOL_ERR_UNSUPPORTED, "top_k must be in [1,%d] and <= pool_size, got %d",
             UNIPOOL_MAX_TOPK, c->top_k);
  UP_REQUIRE(c->n_layers >= 1, UNIPOOL_ERR_INVALID_ARG, "n_layers must be >= 1");
  UP_REQUIRE(c->max_tokens >= 1 && (int64_t)c->max_tokens * c->top_k < (1ll << 30),
             UNIPOOL_ERR_UNSUPPORTED, "max_tokens*top_k must be in [1, 2^30)");
  UP_REQUIRE(c->eps >= 0.f && c->c > 0.f, UNIPOOL_ERR_INVALID_ARG, "eps must be >= 0 and c > 0");
  UP_REQUIRE(c->router_mode == UNIPOOL_ROUTER_NORM || c->router_mode == UNIPOOL_ROUTER_SOFTMAX,
             UNIPOOL_ERR_INVALID_ARG, "router_mode must be UNIPOOL_ROUTER_NORM or UNIPOOL_ROUTER_SOFTMAX");
  return UNIPOOL_OK;
}

}  // namespace unipool

using namespace unipool;

#define CHECK_CTX(ctx) UP_REQUIRE((ctx) != nullptr, UNIPOOL_ERR_INVALID_ARG, "ctx is NULL")
#define CHECK_PTR(p) UP_REQUIRE((p) != nullptr, UNIPOOL_ERR_INVALID_ARG, #p " is NULL")
#define CHECK_T(ctx, T)                                                              \
  UP_REQUIRE((T) >= 0 && (T) <= (ctx)->cfg.max_tokens, UNIPOOL_ERR_INVALID_ARG,      \
             "T = %d outside [0, max_tokens = %d]", (int)(T), (ctx)->cfg.max_tokens)
#define CHECK_VIEW(ctx, base, n)                                                              \
  UP_REQUIRE((n) >= 1 && (base) >= 0 && (base) + (n) <= (ctx)->cfg.pool_size,                 \
             UNIPOOL_ERR_INVALID_ARG, "pool view [%d, %d) outside the pool of %d experts",    \
             (int)(base), (int)((base) + (n)), (ctx)->cfg.pool_size)
#define CHECK_ROUTER_WIDTH(ctx, n)                                                            \
  UP_REQUIRE((n) >= (ctx)->cfg.top_k && (n) <= (ctx)->cfg.pool_size, UNIPOOL_ERR_INVALID_ARG, \
             "n_experts = %d must be in [top_k = %d, pool_size = %d]", (int)(n),              \
             (ctx)->cfg.top_k, (ctx)->cfg.pool_size)

extern "C" {

const char* unipool_last_error(void) { return g_error; }

int64_t unipool_row_capacity(const unipool_config* cfg) {
  if (!cfg) return 0;
  return row_capacity_of(*cfg);
}

size_t unipool_workspace_bytes(const unipool_config* cfg) {
  if (!cfg || validate_config(cfg) != UNIPOOL_OK) return 0;
  return carve_workspace(*cfg, nullptr).bytes;
}

int unipool_create(unipool_ctx** out, const unipool_config* cfg, void* workspace,
                   size_t workspace_bytes, unipool_stream stream) {
  CHECK_PTR(out);
  *out = nullptr;
  int rc = validate_config(cfg);
  if (rc != UNIPOOL_OK) return rc;
  UP_REQUIRE(workspace != nullptr && (reinterpret_cast<uintptr_t>(workspace) & 255) == 0,
             UNIPOOL_ERR_WORKSPACE, "workspace must be a 256-byte aligned device pointer");
  Workspace w = carve_workspace(*cfg, workspace);
  UP_REQUIRE(workspace_bytes >= w.bytes, UNIPOOL_ERR_WORKSPACE,
             "workspace has %zu bytes, %zu needed", workspace_bytes, w.bytes);
  unipool_ctx* ctx = new (std::nothrow) unipool_ctx();
  UP_REQUIRE(ctx != nullptr, UNIPOOL_ERR_INVALID_ARG, "out of host memory");
  ctx->cfg = *cfg;
  ctx->ws = w;
  ctx->row_capacity = row_capacity_of(*cfg);
  ctx->elem_bytes = cfg->dtype == UNIPOOL_BF16 ? 2 : 4;
  ctx->tmap_cache = nullptr;
  ctx->prepared_base = nullptr;
  ctx->prepared_layers = ctx->prepared_experts = 0;
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device);
  // the self-cleaning accumulators and the status word start at zero
  size_t head = reinterpret_cast<char*>(w.block_hist) - reinterpret_cast<char*>(workspace);
  if (e == cudaSuccess) e = cudaMemsetAsync(workspace, 0, head, static_cast<cudaStream_t>(stream));
  for (int i = 0; i < w.n_guards && e == cudaSuccess; ++i)
    e = cudaMemsetAsync(w.guards[i], (int)(kGuardWord & 0xff), kGuardBytes, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) {
    set_error("context set-up failed: %s", cudaGetErrorString(e));
    delete ctx;
    return UNIPOOL_ERR_CUDA;
  }
  if (cfg->dtype == UNIPOOL_BF16) {
    rc = tc_module_init(ctx);
    if (rc != UNIPOOL_OK) {
      delete ctx;
      return rc;
    }
  }
  *out = ctx;
  return UNIPOOL_OK;
}

int unipool_destroy(unipool_ctx* ctx) {
  if (!ctx) return UNIPOOL_OK;
  if (ctx->cfg.dtype == UNIPOOL_BF16) tc_module_destroy(ctx);
  for (const ProfRecord& r : ctx->prof.records) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
  for (cudaEvent_t e : ctx->prof.free_events) cudaEventDestroy(e);
  delete ctx;
  return UNIPOOL_OK;
}

int unipool_profile_enable(unipool_ctx* ctx, int32_t on) {
  CHECK_CTX(ctx);
  ctx->prof.enabled = on != 0;
  return UNIPOOL_OK;
}

int unipool_profile_read(unipool_ctx* ctx, double* ms, int64_t* launches) {
  CHECK_CTX(ctx); CHECK_PTR(ms); CHECK_PTR(launches);
  for (int i = 0; i < UNIPOOL_N_PHASES; ++i) { ms[i] = 0.0; launches[i] = 0; }
  for (const ProfRecord& r : ctx->prof.records) {
    UP_CUDA(cudaEventSynchronize(r.stop));
    float t = 0.f;
    UP_CUDA(cudaEventElapsedTime(&t, r.start, r.stop));
    ms[r.phase] += t;
    launches[r.phase] += r.launches;
    ctx->prof.free_events.push_back(r.start);
    ctx->prof.free_events.push_back(r.stop);
  }
  ctx->prof.records.clear();
  return UNIPOOL_OK;
}

int unipool_check_status(unipool_ctx* ctx, unipool_stream stream) {
  CHECK_CTX(ctx);
  int32_t host[4] = {0, 0, 0, 0};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (ctx->ws.n_guards > 0) {
    int rc = guard_check_launch(ctx, s);
    if (rc != UNIPOOL_OK) return rc;
  }
  UP_CUDA(cudaMemcpyAsync(host, ctx->ws.status, sizeof(host), cudaMemcpyDeviceToHost, s));
  UP_CUDA(cudaStreamSynchronize(s));
  if (host[0] == 0) return UNIPOOL_OK;
  UP_CUDA(cudaMemsetAsync(ctx->ws.status, 0, sizeof(host), s));
  UP_CUDA(cudaStreamSynchronize(s));
  if (host[0] == kStatusTimeout) {
    set_error("a bounded device-side wait ran out (site %d, detail %d)", host[1], host[2]);
    return UNIPOOL_ERR_TIMEOUT;
  }
  if (host[1] >= kGuardSite && host[1] < kGuardSite + 16)
    set_error("the guard band behind workspace region %d was overwritten (byte %d of it)", host[1] - kGuardSite, host[2]);
  else
    set_error("device-side consistency check failed (site %d, detail %d)", host[1], host[2]);
  return UNIPOOL_ERR_DEVICE_CHECK;
}

int unipool_route(unipool_ctx* ctx, const void* x, int32_t T, const float* W_r, float sigma,
                  const float* bias, int32_t n_experts, int32_t* idx, float* gate,
                  int32_t* counts, float* score_sum, float* znorm, float* z_saved,
                  unipool_stream stream) {
  CHECK_CTX(ctx); CHECK_T(ctx, T); CHECK_ROUTER_WIDTH(ctx, n_experts);
  CHECK_PTR(x); CHECK_PTR(W_r); CHECK_PTR(idx); CHECK_PTR(gate); CHECK_PTR(counts);
  CHECK_PTR(score_sum); CHECK_PTR(znorm); CHECK_PTR(z_saved);
  return route_launch(ctx, x, T, W_r, sigma, bias, n_experts, idx, gate, counts, score_sum,
                      znorm, z_saved, static_cast<cudaStream_t>(stream));
}

int unipool_router_prepare(unipool_ctx* ctx, const float* W_r, int32_t n_layers, int32_t n_experts,
                           unipool_stream stream) {
  CHECK_CTX(ctx);
  UP_REQUIRE(n_layers >= 0 && n_layers <= ctx->cfg.n_layers, UNIPOOL_ERR_INVALID_ARG,
             "n_layers = %d outside [0, %d]", n_layers, ctx->cfg.n_layers);
  if (n_layers > 0) { CHECK_PTR(W_r); CHECK_ROUTER_WIDTH(ctx, n_experts); }
  if (!use_tensor_cores(ctx)) return UNIPOOL_OK;            // the fp32 path reads W_r itself
  return router_prepare_launch(ctx, W_r, n_layers, n_experts, static_cast<cudaStream_t>(stream));
}

int unipool_dispatch(unipool_ctx* ctx, const void* x, int32_t T, const int32_t* idx,
                     int32_t n_experts, int32_t* offsets, int32_t* row_of, int32_t* token_of,
                     int32_t* tile_expert, void* Xp, unipool_stream stream) {
  CHECK_CTX(ctx); CHECK_T(ctx, T); CHECK_ROUTER_WIDTH(ctx, n_experts);
  CHECK_PTR(x); CHECK_PTR(idx); CHECK_PTR(offsets); CHECK_PTR(row_of); CHECK_PTR(token_of);
  CHECK_PTR(tile_expert); CHECK_PTR(Xp);
  return dispatch_launch(ctx, x, T, idx, n_experts, offsets, row_of, token_of, tile_expert, Xp,
                         static_cast<cudaStream_t>(stream));
}

int unipool_expert_fwd(unipool_ctx* ctx, const void* Xp, const int32_t* offsets,
                       const int32_t* tile_expert, const void* W_gu, const void* W_down,
                       int32_t expert_base, int32_t n_experts, void* GU, void* A, void* Yp,
                       unipool_stream stream) {
  CHECK_CTX(ctx); CHECK_VIEW(ctx, expert_base, n_experts);
  CHECK_PTR(Xp); CHECK_PTR(offsets); CHECK_PTR(tile_expert); CHECK_PTR(W_gu); CHECK_PTR(W_down);
  CHECK_PTR(GU); CHECK_PTR(A); CHECK_PTR(Yp);
  ExpertFwdArgs a{Xp, offsets, tile_expert, W_gu, W_down, expert_base, n_experts, GU, A, Yp};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  return use_tensor_cores(ctx) ? expert_fwd_tc(ctx, a, s) : expert_fwd_simt(ctx, a, s);
}

int unipool_combine(unipool_ctx* ctx, const void* Yp, const int32_t* row_of, const float* gate,
                    int32_t T, const void* residual, void* y, unipool_stream stream) {
  CHECK_CTX(ctx); CHECK_T(ctx, T);
  CHECK_PTR(Yp); CHECK_PTR(row_of); CHECK_PTR(gate); CHECK_PTR(y);
  return combine_launch(ctx, Yp, row_of, gate, T, residual, y, static_cast<cudaStream_t>(stream));
}

int unipool_expert_bwd(unipool_ctx* ctx, const void* dy, int32_t T, const int32_t* row_of,
                       const float* gate, const int32_t* token_of, const int32_t* offsets,
                       const int32_t* tile_expert, const void* Xp, const void* GU, const void* A,
                       const void* Yp, const void* W_gu, const void* W_down, int32_t expert_base,
                       int32_t n_experts, const void* dx_residual, void* dYp, void* dGU, void* dx,
                       float* dgate, float* dW_gu, float* dW_down, int32_t flags,
                       unipool_stream stream) {
  CHECK_CTX(ctx); CHECK_T(ctx, T); CHECK_VIEW(ctx, expert_base, n_experts);
  CHECK_PTR(dy); CHECK_PTR(row_of); CHECK_PTR(gate); CHECK_PTR(token_of); CHECK_PTR(offsets);
  CHECK_PTR(tile_expert); CHECK_PTR(Xp); CHECK_PTR(GU); CHECK_PTR(A); CHECK_PTR(Yp);
  CHECK_PTR(W_gu); CHECK_PTR(W_down); CHECK_PTR(dYp); CHECK_PTR(dGU); CHECK_PTR(dx); CHECK_PTR(dgate);
  UP_REQUIRE((flags & ~(UNIPOOL_BWD_SKIP_WGRAD | UNIPOOL_WGRAD_OVERWRITE)) == 0, UNIPOOL_ERR_INVALID_ARG,
             "unknown flags 0x%x", flags);
  const bool wgrad = !(flags & UNIPOOL_BWD_SKIP_WGRAD);
  if (wgrad) { CHECK_PTR(dW_gu); CHECK_PTR(dW_down); }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = combine_bwd_launch(ctx, dy, T, row_of, gate, token_of, offsets, n_experts, Yp, dYp, dgate, s);
  if (rc != UNIPOOL_OK) return rc;
  ExpertBwdArgs a{offsets, tile_expert, Xp, GU, A, W_gu, W_down, expert_base, n_experts,
                  dYp, dGU, ctx->ws.dXp, dW_gu, dW_down, wgrad, (flags & UNIPOOL_WGRAD_OVERWRITE) != 0};
  rc = use_tensor_cores(ctx) ? expert_bwd_tc(ctx, a, s) : expert_bwd_simt(ctx, a, s);
  if (rc != UNIPOOL_OK) return rc;
  return unpermute_sum_launch(ctx, ctx->ws.dXp, row_of, T, dx_residual, dx, s);
}

int unipool_pool_wgrad(unipool_ctx* ctx, int32_t n_layers, int64_t layer_stride_rows,
                       const int32_t* offsets, const void* Xp, const void* A, const void* dYp,
                       const void* dGU, int32_t expert_base, int32_t n_experts, float* dW_gu,
                       float* dW_down, int32_t flags, unipool_stream stream) {
  CHECK_CTX(ctx); CHECK_VIEW(ctx, expert_base, n_experts);
  UP_REQUIRE(n_layers >= 1, UNIPOOL_ERR_INVALID_ARG, "n_layers must be >= 1");
  UP_REQUIRE(layer_stride_rows >= 0 && layer_stride_rows % UNIPOOL_ROW_ALIGN == 0,
             UNIPOOL_ERR_INVALID_ARG, "layer_stride_rows must be a multiple of %d", UNIPOOL_ROW_ALIGN);
  UP_REQUIRE((int64_t)n_layers * layer_stride_rows < (1ll << 31) && (n_layers == 1 || layer_stride_rows > 0),
             UNIPOOL_ERR_UNSUPPORTED, "n_layers * layer_stride_rows = %lld must stay below 2^31 rows",
             (long long)n_layers * (long long)layer_stride_rows);
  CHECK_PTR(offsets);
  UP_REQUIRE(dW_gu != nullptr || dW_down != nullptr, UNIPOOL_ERR_INVALID_ARG, "dW_gu and dW_down are both NULL");
  if (dW_gu != nullptr) { CHECK_PTR(Xp); CHECK_PTR(dGU); }
  if (dW_down != nullptr) { CHECK_PTR(A); CHECK_PTR(dYp); }
  UP_REQUIRE((flags & ~UNIPOOL_WGRAD_OVERWRITE) == 0, UNIPOOL_ERR_INVALID_ARG, "unknown flags 0x%x", flags);
  PoolWgradArgs a{n_layers, layer_stride_rows, offsets, Xp, A, dYp, dGU, expert_base, n_experts,
                  dW_gu, dW_down, (flags & UNIPOOL_WGRAD_OVERWRITE) != 0};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  return use_tensor_cores(ctx) ? pool_wgrad_tc(ctx, a, s) : pool_wgrad_simt(ctx, a, s);
}

int unipool_pool_aux_loss(unipool_ctx* ctx, const int32_t* counts, const float* score_sum,
                          int32_t L, int32_t n_experts, int32_t T, float alpha,
                          const float* fbar_prev, float* loss, float* dscore_coef,
                          float* fbar_out, unipool_stream stream) {
  CHECK_CTX(ctx);
  UP_REQUIRE(L >= 1 && T >= 1, UNIPOOL_ERR_INVALID_ARG, "L and T must be >= 1");
  UP_REQUIRE(n_experts >= 1 && n_experts <= UNIPOOL_MAX_EXPERTS, UNIPOOL_ERR_INVALID_ARG,
             "n_experts = %d outside [1, %d]", n_experts, UNIPOOL_MAX_EXPERTS);
  CHECK_PTR(counts); CHECK_PTR(score_sum); CHECK_PTR(loss); CHECK_PTR(dscore_coef); CHECK_PTR(fbar_out);
  return aux_launch(ctx, counts, score_sum, L, n_experts, T, alpha, fbar_prev, loss, dscore_coef,
                    fbar_out, static_cast<cudaStream_t>(stream));
}

int unipool_route_bwd(unipool_ctx* ctx, const void* x, int32_t T, const float* W_r, float sigma,
                      int32_t n_experts, const float* znorm, const float* z_saved,
                      const int32_t* idx, const float* dgate, const float* dscore_coef,
                      void* dx, float* dW_r, float* dsigma, unipool_stream stream) {
  CHECK_CTX(ctx); CHECK_T(ctx, T); CHECK_ROUTER_WIDTH(ctx, n_experts);
  CHECK_PTR(x); CHECK_PTR(W_r); CHECK_PTR(znorm); CHECK_PTR(z_saved); CHECK_PTR(idx);
  CHECK_PTR(dgate); CHECK_PTR(dx); CHECK_PTR(dW_r); CHECK_PTR(dsigma);
  return route_bwd_launch(ctx, x, T, W_r, sigma, n_experts, znorm, z_saved, idx, dgate,
                          dscore_coef, dx, dW_r, dsigma, static_cast<cudaStream_t>(stream));
}

int unipool_unique_experts(unipool_ctx* ctx, const int32_t* idx, const int32_t* expert_base, int32_t L,
                           int32_t T, int32_t* unique, uint64_t* total, unipool_stream stream) {
  CHECK_CTX(ctx); CHECK_T(ctx, T); CHECK_PTR(idx); CHECK_PTR(unique); CHECK_PTR(total);
  UP_REQUIRE(L >= 1, UNIPOOL_ERR_INVALID_ARG, "L must be >= 1");
  return unique_experts_launch(ctx, idx, expert_base, L, T, unique, reinterpret_cast<unsigned long long*>(total),
                               static_cast<cudaStream_t>(stream));
}

int unipool_selftest_wait(unipool_ctx* ctx, int64_t limit_cycles, unipool_stream stream) {
  CHECK_CTX(ctx);
  UP_REQUIRE(limit_cycles >= 0 && limit_cycles <= 2000000000ll, UNIPOOL_ERR_INVALID_ARG,
             "limit_cycles = %lld outside [0, 2e9]", (long long)limit_cycles);
  return wait_selftest_launch(ctx, limit_cycles, static_cast<cudaStream_t>(stream));
}

int unipool_calibrate_c(unipool_ctx* ctx, int32_t n_experts, int32_t top_k, int32_t n_samples,
                        uint64_t seed, float* c_out, unipool_stream stream) {
  CHECK_CTX(ctx); CHECK_PTR(c_out);
  UP_REQUIRE(n_experts >= 1 && n_experts <= UNIPOOL_MAX_EXPERTS && top_k >= 1 &&
                 top_k <= UNIPOOL_MAX_TOPK && top_k <= n_experts && n_samples >= 1,
             UNIPOOL_ERR_INVALID_ARG, "calibrate_c: bad (n_experts, top_k, n_samples)");
  return calibrate_launch(ctx, n_experts, top_k, n_samples, seed, c_out,
                          static_cast<cudaStream_t>(stream));
}

}  // extern "C"
