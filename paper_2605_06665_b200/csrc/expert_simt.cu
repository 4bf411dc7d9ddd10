// Grouped SwiGLU expert FFN on CUDA cores with exact fp32 accumulation.
// This is the arithmetic path of the fp32 mode (parity bound 1e-5, which TF32
// tensor-core products cannot meet); it also accepts bf16 storage.
#include "common.cuh"
#include "simt_gemm.cuh"

namespace unipool {

// C[rows, N] = A[rows, K] * B_e(k, n) for every 64-row tile of the permuted row
// space; the tile's expert selects B.  Rows at and beyond offsets[n_experts] are
// skipped (tile_expert < 0).
template <typename TE>
__global__ void __launch_bounds__(kSimtThreads)
grouped_rows_gemm_kernel(const TE* __restrict__ A, int64_t lda, const TE* __restrict__ B,
                         int64_t b_expert_stride, int64_t b_sk, int64_t b_sn,
                         const int32_t* __restrict__ tile_expert, int expert_base,
                         TE* __restrict__ C, int64_t ldc, int N, int K, int n_row_tiles) {
  const int n0 = blockIdx.x * kSimtTile;
  for (int rt = blockIdx.y; rt < n_row_tiles; rt += gridDim.y) {
    const int m0 = rt * kSimtTile;
    const int e = tile_expert[m0 / UNIPOOL_ROW_ALIGN];
    if (e < 0) continue;                     // uniform over the block
    float acc[4][4] = {};
    SimtOperands<TE, TE> op{A, lda, 1, B + (int64_t)(expert_base + e) * b_expert_stride, b_sk, b_sn};
    simt_tile_mainloop(op, m0, n0, m0 + kSimtTile, N, 0, K, acc);
    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int n = n0 + tx * 4 + j;
        if (n < N) C[(int64_t)(m0 + ty * 4 + i) * ldc + n] = from_f32<TE>(acc[i][j]);
      }
  }
}

// dW[e][m, n] += sum over the rows r of group e (of every listed layer) of P[r, m] * Q[r, n].
template <typename TE>
__global__ void __launch_bounds__(kSimtThreads)
grouped_k_gemm_kernel(const TE* __restrict__ P, int64_t ldp, const TE* __restrict__ Q, int64_t ldq,
                      const int32_t* __restrict__ offsets, int n_experts, int expert_base,
                      int n_layers, int64_t layer_stride_rows, float* __restrict__ dW,
                      int64_t w_expert_stride, int Mdim, int Ndim, bool overwrite) {
  const int m0 = blockIdx.x * kSimtTile, n0 = blockIdx.y * kSimtTile;
  const int e = blockIdx.z;
  float acc[4][4] = {};
  for (int l = 0; l < n_layers; ++l) {
    const int32_t* off = offsets + (int64_t)l * (n_experts + 1);
    const int r0 = off[e], r1 = off[e + 1];
    if (r1 <= r0) continue;
    const TE* Pl = P + l * layer_stride_rows * ldp;
    const TE* Ql = Q + l * layer_stride_rows * ldq;
    SimtOperands<TE, TE> op{Pl, 1, ldp, Ql, ldq, 1};
    simt_tile_mainloop(op, m0, n0, Mdim, Ndim, r0, r1, acc);
  }
  float* out = dW + (int64_t)(expert_base + e) * w_expert_stride;
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int m = m0 + ty * 4 + i;
    if (m >= Mdim) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int n = n0 + tx * 4 + j;
      if (n < Ndim) out[(int64_t)m * Ndim + n] = overwrite ? acc[i][j] : out[(int64_t)m * Ndim + n] + acc[i][j];
    }
  }
}

// A[r, j] = silu(G[r, j]) * U[r, j] over rows < offsets_end.
template <typename TE>
__global__ void swiglu_kernel(const TE* __restrict__ GU, TE* __restrict__ A,
                              const int32_t* __restrict__ offsets_end, int f) {
  const int64_t total = (int64_t)(*offsets_end) * f;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t r = i / f;
    int j = (int)(i % f);
    float g = to_f32(GU[r * 2 * f + j]), u = to_f32(GU[r * 2 * f + f + j]);
    A[i] = from_f32<TE>(silu_f(g) * u);
  }
}

// In place on dGU, whose U half holds dA on entry:
//   dG = dA * U * silu'(G) -> dGU[:, :f];   dU = dA * silu(G) -> dGU[:, f:].
template <typename TE>
__global__ void swiglu_bwd_kernel(const TE* __restrict__ GU, TE* __restrict__ dGU,
                                  const int32_t* __restrict__ offsets_end, int f) {
  const int64_t total = (int64_t)(*offsets_end) * f;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t r = i / f;
    int j = (int)(i % f);
    float g = to_f32(GU[r * 2 * f + j]), u = to_f32(GU[r * 2 * f + f + j]);
    float dA = to_f32(dGU[r * 2 * f + f + j]);
    dGU[r * 2 * f + j] = from_f32<TE>(dA * u * silu_grad_f(g));
    dGU[r * 2 * f + f + j] = from_f32<TE>(dA * silu_f(g));
  }
}

template <typename TE>
static int fwd_impl(unipool_ctx* ctx, const ExpertFwdArgs& a, cudaStream_t s) {
  const int d = ctx->cfg.d_model, f = ctx->cfg.d_ff;
  const int n_row_tiles = (int)(ctx->row_capacity / kSimtTile);
  const int gy = n_row_tiles < 4096 ? n_row_tiles : 4096;
  const TE* Xp = static_cast<const TE*>(a.Xp);
  const TE* Wgu = static_cast<const TE*>(a.W_gu);
  const TE* Wd = static_cast<const TE*>(a.W_down);
  TE* GU = static_cast<TE*>(a.GU);
  TE* A = static_cast<TE*>(a.A);
  TE* Yp = static_cast<TE*>(a.Yp);
  // GU = Xp W_gu[e]^T : B(k, n) = W_gu[e][n, k]
  {
  PhaseTimer pt(ctx, UNIPOOL_PH_EXPERT_FWD_GU, 2, s);
  grouped_rows_gemm_kernel<TE><<<dim3(2 * f / kSimtTile, gy), kSimtThreads, 0, s>>>(
      Xp, d, Wgu, (int64_t)2 * f * d, 1, d, a.tile_expert, a.expert_base, GU, 2 * f, 2 * f, d, n_row_tiles);
  UP_LAUNCH_CHECK();
  swiglu_kernel<TE><<<ctx->sm_count * 8, 256, 0, s>>>(GU, A, a.offsets + a.n_experts, f);
  UP_LAUNCH_CHECK();
  }
  PhaseTimer pt(ctx, UNIPOOL_PH_EXPERT_FWD_DOWN, 1, s);
  // Yp = A W_down[e]^T : B(k, n) = W_down[e][n, k]
  grouped_rows_gemm_kernel<TE><<<dim3(d / kSimtTile, gy), kSimtThreads, 0, s>>>(
      A, f, Wd, (int64_t)d * f, 1, f, a.tile_expert, a.expert_base, Yp, d, d, f, n_row_tiles);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

template <typename TE>
static int wgrad_impl(unipool_ctx* ctx, const PoolWgradArgs& a, cudaStream_t s) {
  const int d = ctx->cfg.d_model, f = ctx->cfg.d_ff;
  // dW_down[e][d, f] += dYp_e^T A_e
  if (a.dW_down != nullptr) {
  PhaseTimer pt(ctx, UNIPOOL_PH_WGRAD_DOWN, 1, s);
  grouped_k_gemm_kernel<TE><<<dim3(d / kSimtTile, f / kSimtTile, a.n_experts), kSimtThreads, 0, s>>>(
      static_cast<const TE*>(a.dYp), d, static_cast<const TE*>(a.A), f, a.offsets, a.n_experts,
      a.expert_base, a.n_layers, a.layer_stride_rows, a.dW_down, (int64_t)d * f, d, f, a.overwrite);
  UP_LAUNCH_CHECK();
  }
  if (a.dW_gu == nullptr) return UNIPOOL_OK;
  PhaseTimer pt(ctx, UNIPOOL_PH_WGRAD_GU, 1, s);
  // dW_gu[e][2f, d] += dGU_e^T Xp_e
  grouped_k_gemm_kernel<TE><<<dim3(2 * f / kSimtTile, d / kSimtTile, a.n_experts), kSimtThreads, 0, s>>>(
      static_cast<const TE*>(a.dGU), 2 * f, static_cast<const TE*>(a.Xp), d, a.offsets, a.n_experts,
      a.expert_base, a.n_layers, a.layer_stride_rows, a.dW_gu, (int64_t)2 * f * d, 2 * f, d, a.overwrite);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

template <typename TE>
static int bwd_impl(unipool_ctx* ctx, const ExpertBwdArgs& a, cudaStream_t s) {
  const int d = ctx->cfg.d_model, f = ctx->cfg.d_ff;
  const int n_row_tiles = (int)(ctx->row_capacity / kSimtTile);
  const int gy = n_row_tiles < 4096 ? n_row_tiles : 4096;
  const TE* dYp = static_cast<const TE*>(a.dYp);
  TE* dGU = static_cast<TE*>(a.dGU);
  // dA = dYp W_down[e] : B(k, n) = W_down[e][k, n]; lands in the U half of dGU
  {
  PhaseTimer pt(ctx, UNIPOOL_PH_DGRAD_DOWN, 2, s);
  grouped_rows_gemm_kernel<TE><<<dim3(f / kSimtTile, gy), kSimtThreads, 0, s>>>(
      dYp, d, static_cast<const TE*>(a.W_down), (int64_t)d * f, f, 1, a.tile_expert, a.expert_base,
      dGU + f, 2 * f, f, d, n_row_tiles);
  UP_LAUNCH_CHECK();
  swiglu_bwd_kernel<TE><<<ctx->sm_count * 8, 256, 0, s>>>(static_cast<const TE*>(a.GU), dGU,
                                                          a.offsets + a.n_experts, f);
  UP_LAUNCH_CHECK();
  }
  // dXp = dGU W_gu[e] : B(k, n) = W_gu[e][k, n]
  {
  PhaseTimer pt(ctx, UNIPOOL_PH_DGRAD_GU, 1, s);
  grouped_rows_gemm_kernel<TE><<<dim3(d / kSimtTile, gy), kSimtThreads, 0, s>>>(
      dGU, 2 * f, static_cast<const TE*>(a.W_gu), (int64_t)2 * f * d, d, 1, a.tile_expert,
      a.expert_base, static_cast<TE*>(a.dXp), d, d, 2 * f, n_row_tiles);
  UP_LAUNCH_CHECK();
  }
  if (a.wgrad) {
    PoolWgradArgs w{1, 0, a.offsets, a.Xp, a.A, a.dYp, a.dGU, a.expert_base, a.n_experts, a.dW_gu, a.dW_down,
                    a.overwrite};
    return wgrad_impl<TE>(ctx, w, s);
  }
  return UNIPOOL_OK;
}

int expert_fwd_simt(unipool_ctx* ctx, const ExpertFwdArgs& a, cudaStream_t s) {
  return ctx->cfg.dtype == UNIPOOL_BF16 ? fwd_impl<__nv_bfloat16>(ctx, a, s) : fwd_impl<float>(ctx, a, s);
}
int expert_bwd_simt(unipool_ctx* ctx, const ExpertBwdArgs& a, cudaStream_t s) {
  return ctx->cfg.dtype == UNIPOOL_BF16 ? bwd_impl<__nv_bfloat16>(ctx, a, s) : bwd_impl<float>(ctx, a, s);
}
int pool_wgrad_simt(unipool_ctx* ctx, const PoolWgradArgs& a, cudaStream_t s) {
  return ctx->cfg.dtype == UNIPOOL_BF16 ? wgrad_impl<__nv_bfloat16>(ctx, a, s) : wgrad_impl<float>(ctx, a, s);
}

}  // namespace unipool
