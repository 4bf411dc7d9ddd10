// Shared host/device declarations of the UniPool library (internal header).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "unipool.h"

namespace unipool {

// ---------------------------------------------------------------- errors
void set_error(const char* fmt, ...);

#define UP_REQUIRE(cond, code, ...)      \
  do {                                   \
    if (!(cond)) {                       \
      unipool::set_error(__VA_ARGS__);   \
      return (code);                     \
    }                                    \
  } while (0)

#define UP_CUDA(call)                                                                  \
  do {                                                                                 \
    cudaError_t e__ = (call);                                                          \
    if (e__ != cudaSuccess) {                                                          \
      unipool::set_error("%s failed: %s (%s:%d)", #call, cudaGetErrorString(e__), __FILE__, \
                         __LINE__);                                                    \
      return UNIPOOL_ERR_CUDA;                                                         \
    }                                                                                  \
  } while (0)

#define UP_LAUNCH_CHECK()                                                              \
  do {                                                                                 \
    cudaError_t e__ = cudaGetLastError();                                              \
    if (e__ != cudaSuccess) {                                                          \
      unipool::set_error("kernel launch failed: %s (%s:%d)", cudaGetErrorString(e__),  \
                         __FILE__, __LINE__);                                          \
      return UNIPOOL_ERR_CUDA;                                                         \
    }                                                                                  \
  } while (0)

// ---------------------------------------------------------------- workspace
// Fixed layout of the caller's workspace; every region is 256-byte aligned.
struct Workspace {
  int32_t* status;        // [4]   device status word (+ spare)
  int32_t* route_counts;  // [MAX_EXPERTS] self-cleaning accumulators of route
  double*  route_sums;    // [MAX_EXPERTS]
  uint32_t* tickets;      // [8]   "last block done" counters, self-cleaning
  double*  dsigma_acc;    // [2]   self-cleaning accumulator of route_bwd / calibrate_c
  int32_t* block_hist;    // [dispatch_blocks, MAX_EXPERTS]
  float*   dz;            // route_bwd scratch: fp32 [max_tokens, pool_size], or bf16 [max_tokens, ceil64(pool_size)]
  int32_t* split_any;     // [n_layers + 1][4] which bf16 terms of a router's split weights are non-zero
  void*    w_split;       // [n_layers + 1][3, pool_size, d] bf16 terms of the router weights (bf16 mode): one slot
                          // per prepared layer, the last one scratch for routers that were not prepared
  int32_t* part_counts;   // [2 ceil(max_tokens/256), pool_size] per-CTA routing counts (bf16 mode)
  float*   part_sums;     // [2 ceil(max_tokens/256), pool_size] per-CTA score sums
  float*   part_dsigma;   // [ceil(max_tokens/64)] per-block dsigma terms
  void*    dXp;           // [row_capacity, d] expert_bwd scratch (ctx dtype)
  size_t   bytes;         // total
  char*    guards[16];    // debug mode: the 256-byte guard band behind each region
  int      n_guards;      // 0 unless UNIPOOL_DEBUG=1
};
constexpr int kGuardBytes = 256;
constexpr unsigned kGuardWord = 0xA5A5A5A5u;
constexpr int kGuardSite = 200;               // status site of guard band i: kGuardSite + i

constexpr int kDispatchChunkTokens = 256;     // most tokens per block of the permute kernels (eight warps of 32)
constexpr int kDispatchMinChunkTokens = 64;   // fewest

Workspace carve_workspace(const unipool_config& cfg, void* base);

}  // namespace unipool

namespace unipool {
struct ProfRecord { int phase; int launches; cudaEvent_t start, stop; };
struct Profiler {
  bool enabled = false;
  std::vector<ProfRecord> records;       // events recorded since the last read
  std::vector<cudaEvent_t> free_events;  // recycled events
  cudaEvent_t get() {
    if (!free_events.empty()) { cudaEvent_t e = free_events.back(); free_events.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
  }
};
}  // namespace unipool

struct unipool_ctx {
  unipool::Profiler prof;
  unipool_config cfg;
  unipool::Workspace ws;
  int device;
  int sm_count;
  int64_t row_capacity;
  size_t elem_bytes;
  void* tmap_cache;   // opaque, owned by the tensor-core GEMM module
  const float* prepared_base;   // router weights last given to unipool_router_prepare (NULL: none)
  int prepared_layers, prepared_experts;
};

namespace unipool {

// Brackets the kernels launched during its lifetime with a pair of events (when profiling is on).
struct PhaseTimer {
  unipool_ctx* ctx; cudaStream_t s; cudaEvent_t stop = nullptr;
  PhaseTimer(unipool_ctx* c, int phase, int launches, cudaStream_t stream) : ctx(c), s(stream) {
    if (!ctx->prof.enabled) return;
    cudaEvent_t start = ctx->prof.get();
    stop = ctx->prof.get();
    if (!start || !stop) { stop = nullptr; return; }
    cudaEventRecord(start, s);
    ctx->prof.records.push_back({phase, launches, start, stop});
  }
  ~PhaseTimer() { if (stop) cudaEventRecord(stop, s); }
};

// ---------------------------------------------------------------- element helpers
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

__device__ __forceinline__ float silu_f(float a) { return a / (1.0f + __expf(-a)); }
__device__ __forceinline__ float silu_grad_f(float a) {
  float sig = 1.0f / (1.0f + __expf(-a));
  return sig * (1.0f + a * (1.0f - sig));
}

// status codes written by kernels into ws.status[0]
constexpr int kStatusTimeout = 1;
constexpr int kStatusCheck = 2;

// ---------------------------------------------------------------- module entry points
int route_launch(unipool_ctx*, const void* x, int T, const float* W_r, float sigma,
                 const float* bias, int n_experts, int32_t* idx, float* gate, int32_t* counts,
                 float* score_sum, float* znorm, float* z_saved, cudaStream_t);
int route_bwd_launch(unipool_ctx*, const void* x, int T, const float* W_r, float sigma,
                     int n_experts, const float* znorm, const float* z_saved, const int32_t* idx,
                     const float* dgate, const float* coef, void* dx, float* dW_r, float* dsigma,
                     cudaStream_t);
int dispatch_launch(unipool_ctx*, const void* x, int T, const int32_t* idx, int n_experts,
                    int32_t* offsets, int32_t* row_of, int32_t* token_of, int32_t* tile_expert,
                    void* Xp, cudaStream_t);
int combine_launch(unipool_ctx*, const void* Yp, const int32_t* row_of, const float* gate, int T,
                   const void* residual, void* y, cudaStream_t);
int combine_bwd_launch(unipool_ctx*, const void* dy, int T, const int32_t* row_of,
                       const float* gate, const int32_t* token_of, const int32_t* offsets,
                       int n_experts, const void* Yp, void* dYp, float* dgate, cudaStream_t);
int unpermute_sum_launch(unipool_ctx*, const void* dXp, const int32_t* row_of, int T,
                         const void* residual, void* dx, cudaStream_t);
int aux_launch(unipool_ctx*, const int32_t* counts, const float* S, int L, int n_experts, int T,
               float alpha, const float* fbar_prev, float* loss, float* coef, float* fbar_out,
               cudaStream_t);
int unique_experts_launch(unipool_ctx*, const int32_t* idx, const int32_t* expert_base, int L, int T,
                          int32_t* unique, unsigned long long* total, cudaStream_t);
int wait_selftest_launch(unipool_ctx*, long long limit_cycles, cudaStream_t);
int guard_check_launch(unipool_ctx*, cudaStream_t);
int calibrate_launch(unipool_ctx*, int n_experts, int top_k, int n_samples, uint64_t seed,
                     float* c_out, cudaStream_t);

// grouped GEMMs: CUDA-core path (fp32 mode) and tcgen05 path (bf16 mode)
struct ExpertFwdArgs {
  const void* Xp; const int32_t* offsets; const int32_t* tile_expert;
  const void* W_gu; const void* W_down; int expert_base; int n_experts;
  void* GU; void* A; void* Yp;
};
struct ExpertBwdArgs {
  const int32_t* offsets; const int32_t* tile_expert;
  const void* Xp; const void* GU; const void* A; const void* W_gu; const void* W_down;
  int expert_base; int n_experts;
  const void* dYp; void* dGU; void* dXp; float* dW_gu; float* dW_down; bool wgrad; bool overwrite;
};
struct PoolWgradArgs {
  int n_layers; int64_t layer_stride_rows; const int32_t* offsets;
  const void* Xp; const void* A; const void* dYp; const void* dGU;
  int expert_base; int n_experts; float* dW_gu; float* dW_down; bool overwrite;
};
int route_tc_launch(unipool_ctx*, const void* x, int T, const float* W_r, float sigma, const float* bias,
                    int n_experts, int32_t* idx, float* gate, int32_t* counts, float* score_sum,
                    float* znorm, float* z_saved, cudaStream_t);
int router_prepare_launch(unipool_ctx*, const float* W_r, int n_layers, int n_experts, cudaStream_t);
int route_bwd_tc_launch(unipool_ctx*, const void* x, int T, const float* W_r, float sigma, int n_experts,
                        const float* znorm, const float* z_saved, const int32_t* idx, const float* dgate,
                        const float* coef, void* dx, float* dW_r, float* dsigma, cudaStream_t);
int tc_operand_map(unipool_ctx*, void* out_tensor_map, const void* base, uint64_t cols, uint64_t rows,
                   uint32_t box_rows);
int tc_f32_chunk_map(unipool_ctx*, void* out_tensor_map, const void* base, uint64_t cols, uint64_t rows);
int router_bwd_gemms_tc(unipool_ctx*, const void* dz16, int Mp, const void* W16, const void* x, int T, int M,
                        void* dx, float* dW_r, cudaStream_t);
int expert_fwd_simt(unipool_ctx*, const ExpertFwdArgs&, cudaStream_t);
int expert_bwd_simt(unipool_ctx*, const ExpertBwdArgs&, cudaStream_t);
int pool_wgrad_simt(unipool_ctx*, const PoolWgradArgs&, cudaStream_t);
int expert_fwd_tc(unipool_ctx*, const ExpertFwdArgs&, cudaStream_t);
int expert_bwd_tc(unipool_ctx*, const ExpertBwdArgs&, cudaStream_t);
int pool_wgrad_tc(unipool_ctx*, const PoolWgradArgs&, cudaStream_t);
int tc_module_init(unipool_ctx*);
void tc_module_destroy(unipool_ctx*);

}  // namespace unipool
