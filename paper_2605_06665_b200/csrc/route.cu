// Router forward (NormRouter, Eq. 7, or softmax; top-k, Sec. 4.3) and backward.
#include <cfloat>

#include "common.cuh"
#include "simt_gemm.cuh"

namespace unipool {

// ---------------------------------------------------------------- logits  z = x W_r^T (+ bias)
template <typename TX>
__global__ void __launch_bounds__(kSimtThreads)
router_logits_kernel(const TX* __restrict__ x, const float* __restrict__ W_r,
                     const float* __restrict__ bias, float* __restrict__ z, int T, int M, int d) {
  const int m0 = blockIdx.x * kSimtTile, n0 = blockIdx.y * kSimtTile;
  float acc[4][4] = {};
  SimtOperands<TX, float> op{x, d, 1, W_r, 1, d};
  simt_tile_mainloop(op, m0, n0, T, M, 0, d, acc);
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int t = m0 + ty * 4 + i;
    if (t >= T) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int e = n0 + tx * 4 + j;
      if (e < M) z[(int64_t)t * M + e] = acc[i][j] + (bias ? bias[e] : 0.f);
    }
  }
}

// ---------------------------------------------------------------- scores, top-k, statistics
// One warp per token.  Lane l holds experts l, l+32, ...  Selection key: score
// descending, expert index ascending.
constexpr int kRouteWarps = 8;
constexpr int kRouteTokensPerWarp = 4;

template <bool SOFTMAX>
__global__ void __launch_bounds__(kRouteWarps * 32)
router_select_kernel(const float* __restrict__ z, int T, int M, int k, float sigma_c, float eps,
                     int32_t* __restrict__ idx, float* __restrict__ gate, float* __restrict__ znorm,
                     int32_t* __restrict__ counts_out, float* __restrict__ sum_out,
                     int32_t* __restrict__ acc_counts, double* __restrict__ acc_sums,
                     uint32_t* __restrict__ ticket) {
  extern __shared__ float smem[];
  float* sc = smem;                                           // [warps][M] scores of the current token
  float* wsum = smem + kRouteWarps * M;                       // [warps][M] per-warp score sums
  int* hist = reinterpret_cast<int*>(wsum + kRouteWarps * M); // [M]
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  for (int i = threadIdx.x; i < M; i += blockDim.x) hist[i] = 0;
  for (int i = lane; i < M; i += 32) wsum[warp * M + i] = 0.f;
  __syncthreads();

  float* my = sc + warp * M;
  const int t_begin = (blockIdx.x * kRouteWarps + warp) * kRouteTokensPerWarp;
  for (int tt = 0; tt < kRouteTokensPerWarp; ++tt) {
    const int t = t_begin + tt;
    if (t >= T) break;
    const float* zr = z + (int64_t)t * M;
    if (SOFTMAX) {
      // s = exp(z - max) / sum exp(z - max); the log-sum-exp goes where the NormRouter keeps ||z||
      float mx = -INFINITY;
      for (int i = lane; i < M; i += 32) {
        float v = zr[i];
        my[i] = v;
        mx = fmaxf(mx, v);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      float tot = 0.f;
      for (int i = lane; i < M; i += 32) {
        float e = expf(my[i] - mx);
        my[i] = e;
        tot += e;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
      for (int i = lane; i < M; i += 32) {
        float s = my[i] / tot;
        my[i] = s;
        wsum[warp * M + i] += s;
      }
      if (lane == 0) znorm[t] = mx + logf(tot);
    } else {
      float ss = 0.f;
      for (int i = lane; i < M; i += 32) {
        float v = zr[i];
        my[i] = v;
        ss = fmaf(v, v, ss);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      const float n = sqrtf(ss);
      const float den = n + eps;
      for (int i = lane; i < M; i += 32) {
        float s = sigma_c * fmaxf(0.f, my[i] / den);
        my[i] = s;
        wsum[warp * M + i] += s;
      }
      if (lane == 0) znorm[t] = n;
    }
    __syncwarp();
    for (int j = 0; j < k; ++j) {
      float bv = -INFINITY;
      int bi = INT_MAX;
      for (int i = lane; i < M; i += 32) {
        float v = my[i];
        if (v != -INFINITY && !(v == v)) v = -FLT_MAX;       // NaN scores sort last but stay selectable
        if (v > bv) { bv = v; bi = i; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      if (lane == 0) {
        idx[(int64_t)t * k + j] = bi;
        gate[(int64_t)t * k + j] = my[bi];
        atomicAdd(&hist[bi], 1);
        my[bi] = -INFINITY;
      }
      __syncwarp();
    }
  }
  __syncthreads();
  // block totals -> global accumulators (integer counts exact; score sums in double)
  for (int i = threadIdx.x; i < M; i += blockDim.x) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kRouteWarps; ++w) s += wsum[w * M + i];
    if (hist[i]) atomicAdd(&acc_counts[i], hist[i]);
    if (s != 0.f) atomicAdd(&acc_sums[i], (double)s);
  }
  __threadfence();
  __shared__ bool last;
  __syncthreads();
  if (threadIdx.x == 0) last = atomicAdd(ticket, 1u) == gridDim.x - 1;
  __syncthreads();
  if (last) {                       // the block that arrives last publishes and resets
    __threadfence();
    for (int i = threadIdx.x; i < M; i += blockDim.x) {
      counts_out[i] = __ldcg(&acc_counts[i]);
      sum_out[i] = (float)__ldcg(&acc_sums[i]);
      acc_counts[i] = 0;
      acc_sums[i] = 0.0;
    }
    if (threadIdx.x == 0) *ticket = 0u;
  }
}

__global__ void zero_stats_kernel(int32_t* counts, float* sums, int M) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < M) { counts[i] = 0; sums[i] = 0.f; }
}

int route_launch(unipool_ctx* ctx, const void* x, int T, const float* W_r, float sigma,
                 const float* bias, int M, int32_t* idx, float* gate, int32_t* counts,
                 float* score_sum, float* znorm, float* z_saved, cudaStream_t s) {
  const int d = ctx->cfg.d_model, k = ctx->cfg.top_k;
  if (T == 0) {
    zero_stats_kernel<<<(M + 127) / 128, 128, 0, s>>>(counts, score_sum, M);
    UP_LAUNCH_CHECK();
    return UNIPOOL_OK;
  }
  if (ctx->cfg.dtype == UNIPOOL_BF16)
    return route_tc_launch(ctx, x, T, W_r, sigma, bias, M, idx, gate, counts, score_sum, znorm, z_saved, s);
  dim3 g1((T + kSimtTile - 1) / kSimtTile, (M + kSimtTile - 1) / kSimtTile);
  {
  PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_LOGITS, 1, s);
  if (ctx->cfg.dtype == UNIPOOL_BF16)
    router_logits_kernel<__nv_bfloat16><<<g1, kSimtThreads, 0, s>>>(
        static_cast<const __nv_bfloat16*>(x), W_r, bias, z_saved, T, M, d);
  else
    router_logits_kernel<float><<<g1, kSimtThreads, 0, s>>>(static_cast<const float*>(x), W_r, bias,
                                                            z_saved, T, M, d);
  UP_LAUNCH_CHECK();
  }
  PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_SELECT, 1, s);
  const int per_block = kRouteWarps * kRouteTokensPerWarp;
  const int blocks = (T + per_block - 1) / per_block;
  const size_t smem = (size_t)(2 * kRouteWarps * M) * sizeof(float) + (size_t)M * sizeof(int);
  auto kern = ctx->cfg.router_mode == UNIPOOL_ROUTER_SOFTMAX ? router_select_kernel<true> : router_select_kernel<false>;
  if (smem > 48 * 1024)
    UP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<blocks, kRouteWarps * 32, smem, s>>>(
      z_saved, T, M, k, sigma * ctx->cfg.c, ctx->cfg.eps, idx, gate, znorm, counts, score_sum,
      ctx->ws.route_counts, ctx->ws.route_sums, ctx->ws.tickets + 0);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

// ---------------------------------------------------------------- backward
// dz from (z, n, idx, dgate, coef); one warp per token.
template <bool SOFTMAX>
__global__ void __launch_bounds__(256)
router_dz_kernel(const float* __restrict__ z, const float* __restrict__ znorm,
                 const int32_t* __restrict__ idx, const float* __restrict__ dgate,
                 const float* __restrict__ coef, int T, int M, int k, float sigma, float c, float eps,
                 float* __restrict__ dz, float* __restrict__ dsigma, double* __restrict__ acc,
                 uint32_t* __restrict__ ticket) {
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int t = blockIdx.x * (blockDim.x / 32) + warp;
  float dsig_part = 0.f;
  if (t < T) {
    const float* zr = z + (int64_t)t * M;
    int my_idx = -1;
    float my_dg = 0.f;
    if (lane < k) { my_idx = idx[(int64_t)t * k + lane]; my_dg = dgate[(int64_t)t * k + lane]; }
    const float n = znorm[t];
    const float ne = n + eps;
    float q = 0.f;
    // pass 1: q = sum_i ds_i * max(z_i, 0)
    for (int i0 = 0; i0 < M; i0 += 32) {
      int i = i0 + lane;
      float ds = (i < M && coef) ? coef[i] : 0.f;
      for (int j = 0; j < k; ++j) {
        int ej = __shfl_sync(0xffffffffu, my_idx, j);
        float dj = __shfl_sync(0xffffffffu, my_dg, j);
        if (ej == i) ds += dj;
      }
      if (i < M) q = fmaf(ds, SOFTMAX ? expf(zr[i] - n) : fmaxf(zr[i], 0.f), q);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    const float scale = sigma * c;
    const float qn = n > 0.f ? q / (n * ne * ne) : 0.f;
    for (int i0 = 0; i0 < M; i0 += 32) {
      int i = i0 + lane;
      float ds = (i < M && coef) ? coef[i] : 0.f;
      for (int j = 0; j < k; ++j) {
        int ej = __shfl_sync(0xffffffffu, my_idx, j);
        float dj = __shfl_sync(0xffffffffu, my_dg, j);
        if (ej == i) ds += dj;
      }
      if (i < M) {
        float zi = zr[i];
        float v = n > 0.f ? scale * ((zi > 0.f ? ds / ne : 0.f) - zi * qn) : 0.f;
        if (SOFTMAX) v = expf(zi - n) * (ds - q);          // n holds log sum exp(z)
        dz[(int64_t)t * M + i] = v;
      }
    }
    dsig_part = SOFTMAX ? 0.f : c * q / ne;
  }
  __shared__ float part[8];
  if (lane == 0) part[warp] = dsig_part;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < (int)(blockDim.x / 32); ++w) s += (double)part[w];
    atomicAdd(acc, s);
    __threadfence();
    if (atomicAdd(ticket, 1u) == gridDim.x - 1) {
      __threadfence();
      *dsigma += (float)__ldcg(acc);
      *acc = 0.0;
      *ticket = 0u;
    }
  }
}

// dx[t,:] += dz[t,:] W_r     (K = M)
template <typename TX>
__global__ void __launch_bounds__(kSimtThreads)
router_dx_kernel(const float* __restrict__ dz, const float* __restrict__ W_r, TX* __restrict__ dx,
                 int T, int M, int d) {
  const int m0 = blockIdx.x * kSimtTile, n0 = blockIdx.y * kSimtTile;
  float acc[4][4] = {};
  SimtOperands<float, float> op{dz, M, 1, W_r, d, 1};
  simt_tile_mainloop(op, m0, n0, T, d, 0, M, acc);
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int t = m0 + ty * 4 + i;
    if (t >= T) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int q = n0 + tx * 4 + j;
      if (q < d) {
        int64_t o = (int64_t)t * d + q;
        dx[o] = from_f32<TX>(to_f32(dx[o]) + acc[i][j]);
      }
    }
  }
}

// dW_r[m,:] += sum_t dz[t,m] x[t,:]   (K = T, split over blockIdx.z, fp32 atomics)
template <typename TX>
__global__ void __launch_bounds__(kSimtThreads)
router_dw_kernel(const float* __restrict__ dz, const TX* __restrict__ x, float* __restrict__ dW_r,
                 int T, int M, int d, int k_len) {
  const int m0 = blockIdx.x * kSimtTile, n0 = blockIdx.y * kSimtTile;
  const int k_begin = blockIdx.z * k_len;
  const int k_end = min(T, k_begin + k_len);
  float acc[4][4] = {};
  SimtOperands<float, TX> op{dz, 1, M, x, d, 1};
  simt_tile_mainloop(op, m0, n0, M, d, k_begin, k_end, acc);
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int q = n0 + tx * 4 + j;
      if (q < d) atomicAdd(&dW_r[(int64_t)m * d + q], acc[i][j]);
    }
  }
}

int route_bwd_launch(unipool_ctx* ctx, const void* x, int T, const float* W_r, float sigma, int M,
                     const float* znorm, const float* z_saved, const int32_t* idx,
                     const float* dgate, const float* coef, void* dx, float* dW_r, float* dsigma,
                     cudaStream_t s) {
  if (T == 0) return UNIPOOL_OK;
  if (ctx->cfg.dtype == UNIPOOL_BF16)
    return route_bwd_tc_launch(ctx, x, T, W_r, sigma, M, znorm, z_saved, idx, dgate, coef, dx, dW_r, dsigma, s);
  const int d = ctx->cfg.d_model, k = ctx->cfg.top_k;
  float* dz = ctx->ws.dz;
  {
  PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_BWD_DZ, 1, s);
  auto kern = ctx->cfg.router_mode == UNIPOOL_ROUTER_SOFTMAX ? router_dz_kernel<true> : router_dz_kernel<false>;
  kern<<<(T + 7) / 8, 256, 0, s>>>(z_saved, znorm, idx, dgate, coef, T, M, k, sigma, ctx->cfg.c,
                                   ctx->cfg.eps, dz, dsigma, ctx->ws.dsigma_acc, ctx->ws.tickets + 1);
  UP_LAUNCH_CHECK();
  }
  dim3 g2((T + kSimtTile - 1) / kSimtTile, d / kSimtTile);
  const int k_len = 1024;
  dim3 g3((M + kSimtTile - 1) / kSimtTile, d / kSimtTile, (T + k_len - 1) / k_len);
  const bool bf16 = ctx->cfg.dtype == UNIPOOL_BF16;
  {
    PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_BWD_DX, 1, s);
    if (bf16)
      router_dx_kernel<__nv_bfloat16><<<g2, kSimtThreads, 0, s>>>(dz, W_r, static_cast<__nv_bfloat16*>(dx), T, M, d);
    else
      router_dx_kernel<float><<<g2, kSimtThreads, 0, s>>>(dz, W_r, static_cast<float*>(dx), T, M, d);
    UP_LAUNCH_CHECK();
  }
  PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_BWD_DW, 1, s);
  if (bf16)
    router_dw_kernel<__nv_bfloat16><<<g3, kSimtThreads, 0, s>>>(dz, static_cast<const __nv_bfloat16*>(x), dW_r, T, M, d, k_len);
  else
    router_dw_kernel<float><<<g3, kSimtThreads, 0, s>>>(dz, static_cast<const float*>(x), dW_r, T, M, d, k_len);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

}  // namespace unipool
