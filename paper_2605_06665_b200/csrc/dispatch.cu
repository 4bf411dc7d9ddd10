// Token permute into expert-contiguous order and its inverse (combine), forward
// and backward.  All data movement is in 16-byte vectors; one warp moves one row.
#include <atomic>

#include "common.cuh"

namespace unipool {

// ---------------------------------------------------------------- maps
// Block b owns tokens [b*CH, (b+1)*CH), warp w of it the tokens [w*CH/8, (w+1)*CH/8) of those: the
// stable (token-major) order is block order, then warp order, then lane order inside a warp.
constexpr int kDispatchWarps = 8;
// A chunk holds `chunk` tokens (a multiple of 8, at most kDispatchChunkTokens), a warp chunk / 8 of them.

// hist[w][e] = assignments to expert e among warp w's tokens (shared memory, [kDispatchWarps][M]).
// `status` (may be NULL) receives a corrupt routing entry; the assignment is dropped either way.
__device__ __forceinline__ void chunk_histograms(const int32_t* __restrict__ idx, int T, int k, int M, int chunk,
                                                 int* hist, int32_t* status, int64_t& a_begin, int64_t& a_end) {
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  for (int i = threadIdx.x; i < kDispatchWarps * M; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  const int64_t total = (int64_t)T * k;
  const int warp_tokens = chunk / kDispatchWarps;
  a_begin = min(total, ((int64_t)blockIdx.x * chunk + (int64_t)warp * warp_tokens) * k);
  a_end = min(total, a_begin + (int64_t)warp_tokens * k);
  for (int64_t a = a_begin + lane; a < a_end; a += 32) {
    const int e = idx[a];
    if (e < 0 || e >= M) {          // corrupt routing table: record it, drop the assignment
      if (status != nullptr && atomicCAS(status, 0, kStatusCheck) == 0) { status[1] = 10; status[2] = e; }
      continue;
    }
    atomicAdd(&hist[warp * M + e], 1);
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kDispatchWarps * 32)
dispatch_hist_kernel(const int32_t* __restrict__ idx, int T, int k, int M, int chunk,
                     int32_t* __restrict__ block_hist, int32_t* __restrict__ status) {
  extern __shared__ int hist[];
  int64_t a_begin, a_end;
  chunk_histograms(idx, T, k, M, chunk, hist, status, a_begin, a_end);
  for (int e = threadIdx.x; e < M; e += blockDim.x) {
    int total = 0;
#pragma unroll
    for (int w = 0; w < kDispatchWarps; ++w) total += hist[w * M + e];
    block_hist[(int64_t)e * gridDim.x + blockIdx.x] = total;      // expert-major: [M][chunks]
  }
}

// Second (and last) kernel of the permute.  Block b owns the tokens of chunk b.  From the per-chunk
// histograms of the first kernel every block derives, for itself, the padded group starts (column sums
// over all chunks, exclusive scan over the experts) and the rows its own chunk starts at (column sums
// over the chunks before it); it then ranks its assignments (block, warp, lane order = token order, so
// the permutation is stable), writes row_of / token_of and moves its tokens: a token's row is read
// once and written to each of its k rows.  Every block also takes a share of the bookkeeping: pad rows
// (token_of = -1, zeros in Xp), the tile -> expert table, the rows behind the last group.
constexpr int kPlaceTokens = 8;          // tokens a warp has in flight while moving rows
constexpr int kVpl = 3;                  // 16-byte vectors per lane and pass of the row movers

__global__ void __launch_bounds__(kDispatchWarps * 32)
dispatch_place_kernel(const int32_t* __restrict__ idx, int T, int k, int M, int chunk,
                      const int32_t* __restrict__ block_hist, int n_blocks, const uint4* __restrict__ x,
                      int row_vecs, int row_capacity, int32_t* __restrict__ offsets,
                      int32_t* __restrict__ row_of, int32_t* __restrict__ token_of,
                      int32_t* __restrict__ tile_expert, uint4* __restrict__ Xp) {
  extern __shared__ int sm[];
  int* hist = sm;                                   // [8][M] per-warp histograms, then per-warp next rows
  int* start = hist + kDispatchWarps * M;           // [M + 1] group starts
  int* total = start + M + 1;                       // [M] assignments per expert, all chunks
  int* before = total + M;                          // [M] assignments per expert in the chunks before this one
  int* rows_s = before + M;                         // [chunk * k] row of each assignment of this chunk
  __shared__ int warp_sum[kDispatchWarps];
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int me = (int)blockIdx.x;

  // (a) sums over the chunks of the (expert-major) chunk histograms: a warp per expert, lanes over chunks
  for (int e = warp; e < M; e += kDispatchWarps) {
    int tot = 0, bef = 0;
    for (int b = lane; b < n_blocks; b += 32) {
      const int v = block_hist[(int64_t)e * n_blocks + b];
      tot += v;
      bef += b < me ? v : 0;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      tot += __shfl_xor_sync(0xffffffffu, tot, o);
      bef += __shfl_xor_sync(0xffffffffu, bef, o);
    }
    if (lane == 0) { total[e] = tot; before[e] = bef; }
  }
  __syncthreads();
  // (b) exclusive scan of the padded totals: a thread takes a run of experts, warps and the block scan the runs
  {
    const int per = (M + (int)blockDim.x - 1) / (int)blockDim.x;
    const int e0 = threadIdx.x * per;
    int mine = 0;
    for (int i = 0; i < per; ++i)
      if (e0 + i < M) mine += (total[e0 + i] + UNIPOOL_ROW_ALIGN - 1) / UNIPOOL_ROW_ALIGN * UNIPOOL_ROW_ALIGN;
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    int base = 0;
    for (int w = 0; w < warp; ++w) base += warp_sum[w];
    int run = base + incl - mine;
    for (int i = 0; i < per; ++i)
      if (e0 + i < M) {
        start[e0 + i] = run;
        run += (total[e0 + i] + UNIPOOL_ROW_ALIGN - 1) / UNIPOOL_ROW_ALIGN * UNIPOOL_ROW_ALIGN;
      }
    if (threadIdx.x == blockDim.x - 1) start[M] = run;   // the last thread's run ends the last group
  }
  __syncthreads();
  // (c) this chunk's per-warp histograms -> first row of every warp per expert
  int64_t a_begin, a_end;
  chunk_histograms(idx, T, k, M, chunk, hist, nullptr, a_begin, a_end);
  for (int e = threadIdx.x; e < M; e += blockDim.x) {
    int run = start[e] + before[e];
#pragma unroll
    for (int w = 0; w < kDispatchWarps; ++w) {
      const int n = hist[w * M + e];
      hist[w * M + e] = run;
      run += n;
    }
  }
  __syncthreads();
  // (d) ranks: every warp walks its assignments in lane order
  const int64_t chunk_a0 = (int64_t)me * chunk * k;
  int* next_row = hist + warp * M;
  for (int64_t a0 = a_begin; a0 < a_end; a0 += 32) {
    const int64_t a = a0 + lane;
    const bool live = a < a_end;
    int e = live ? idx[a] : -1;
    const bool ok = live && e >= 0 && e < M;
    if (!ok) e = -1 - lane;                                  // unique key: matches nobody
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    const int rank = __popc(peers & ((1u << lane) - 1u));
    int row = -1;
    if (ok) row = next_row[e] + rank;
    __syncwarp();
    if (ok && rank == 0) next_row[e] += __popc(peers);       // leader = lowest lane of the peer set
    __syncwarp();
    if (live) { row_of[a] = row; rows_s[a - chunk_a0] = row; }
    if (ok) token_of[row] = (int)(a / k);
  }
  __syncthreads();
  // (e) move the chunk's tokens: a warp keeps kPlaceTokens rows of x in flight
  const int t0 = me * chunk;
  const int n_tok = min(chunk, T - t0);
  for (int v0 = lane; v0 < row_vecs; v0 += 32 * kVpl) {
    for (int tt = warp * kPlaceTokens; tt < n_tok; tt += kDispatchWarps * kPlaceTokens) {
      uint4 buf[kPlaceTokens][kVpl];
#pragma unroll
      for (int q = 0; q < kPlaceTokens; ++q)
#pragma unroll
        for (int i = 0; i < kVpl; ++i) {
          const int v = v0 + 32 * i;
          buf[q][i] = (tt + q < n_tok && v < row_vecs) ? __ldg(x + (int64_t)(t0 + tt + q) * row_vecs + v)
                                                       : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
      for (int q = 0; q < kPlaceTokens; ++q) {
        if (tt + q >= n_tok) break;
        for (int j = 0; j < k; ++j) {
          const int row = rows_s[(tt + q) * k + j];
          if (row < 0) continue;
          uint4* dst = Xp + (int64_t)row * row_vecs;
#pragma unroll
          for (int i = 0; i < kVpl; ++i) {
            const int v = v0 + 32 * i;
            if (v < row_vecs) dst[v] = buf[q][i];
          }
        }
      }
    }
  }
  // (f) bookkeeping, shared out over the blocks
  if (me == 0)
    for (int e = threadIdx.x; e <= M; e += blockDim.x) offsets[e] = start[e];
  for (int e = me; e < M; e += gridDim.x) {
    const int lo = start[e] + total[e], hi = start[e + 1];
    for (int r = lo + warp; r < hi; r += kDispatchWarps) {               // pad rows: no token, zeros
      if (lane == 0) token_of[r] = -1;
      uint4* dst = Xp + (int64_t)r * row_vecs;
      for (int v = lane; v < row_vecs; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
    }
    for (int tl = start[e] / UNIPOOL_ROW_ALIGN + threadIdx.x; tl < hi / UNIPOOL_ROW_ALIGN; tl += blockDim.x)
      tile_expert[tl] = e;
  }
  const int used = start[M];
  const int gid = me * (int)blockDim.x + threadIdx.x, gstride = (int)(gridDim.x * blockDim.x);
  for (int r = used + gid; r < row_capacity; r += gstride) token_of[r] = -1;
  for (int tl = used / UNIPOOL_ROW_ALIGN + gid; tl < row_capacity / UNIPOOL_ROW_ALIGN; tl += gstride) tile_expert[tl] = -1;
}

template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static uint4 pack(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void unpack(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static uint4 pack(const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};

// y[t] = (residual[t]) + sum_j gate[t,j] * Yp[row_of[t,j]]   (gate == NULL: unit weights)
// KT = compile-time bound of k (registers for the rows in flight).
template <typename T, int KT>
__global__ void __launch_bounds__(256)
combine_kernel(const uint4* __restrict__ Yp, const int32_t* __restrict__ row_of,
               const float* __restrict__ gate, const uint4* __restrict__ residual,
               uint4* __restrict__ y, int n_tokens, int k, int row_vecs) {
  constexpr int N = Vec16<T>::N;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  for (int t = blockIdx.x * 8 + warp; t < n_tokens; t += gridDim.x * 8) {
    int rows[KT];
    float g[KT];
#pragma unroll
    for (int j = 0; j < KT; ++j) {
      rows[j] = j < k ? row_of[(int64_t)t * k + j] : -1;
      g[j] = (j < k && gate) ? gate[(int64_t)t * k + j] : 1.f;
    }
    for (int v0 = lane; v0 < row_vecs; v0 += 32 * kVpl) {
      uint4 rv[kVpl], yv[KT][kVpl];
#pragma unroll
      for (int i = 0; i < kVpl; ++i) {
        const int v = v0 + 32 * i;
        rv[i] = (residual && v < row_vecs) ? __ldg(residual + (int64_t)t * row_vecs + v) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int j = 0; j < KT; ++j)
          yv[j][i] = (rows[j] >= 0 && v < row_vecs) ? __ldg(Yp + (int64_t)rows[j] * row_vecs + v)
                                                    : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int i = 0; i < kVpl; ++i) {
        const int v = v0 + 32 * i;
        if (v >= row_vecs) continue;
        float acc[N];
        if (residual) {
          Vec16<T>::unpack(rv[i], acc);
        } else {
#pragma unroll
          for (int q = 0; q < N; ++q) acc[q] = 0.f;
        }
#pragma unroll
        for (int j = 0; j < KT; ++j) {
          if (rows[j] < 0) continue;
          float fv[N];
          Vec16<T>::unpack(yv[j][i], fv);
#pragma unroll
          for (int q = 0; q < N; ++q) acc[q] = fmaf(g[j], fv[q], acc[q]);
        }
        y[(int64_t)t * row_vecs + v] = Vec16<T>::pack(acc);
      }
    }
  }
}

// Backward of the combine, token-major: for token t and slot j with row r = row_of[t,j]
//   dgate[t,j] = <dy[t], Yp[r]>,   dYp[r] = gate[t,j] * dy[t];
// afterwards the pad rows (token_of < 0) below offsets[M] are zeroed.  A warp takes KT slots of one
// token; with k > KT the token's slots are split over ceil(k / KT) warps (each re-reads dy[t], which
// keeps the registers per thread low enough for four resident blocks per SM).
template <typename T, int KT>
__global__ void __launch_bounds__(256, 4)
combine_bwd_kernel(const uint4* __restrict__ dy, const uint4* __restrict__ Yp,
                   const int32_t* __restrict__ row_of, const float* __restrict__ gate,
                   const int32_t* __restrict__ token_of, const int32_t* __restrict__ offsets_end,
                   uint4* __restrict__ dYp, float* __restrict__ dgate, int n_tokens, int k, int row_vecs) {
  constexpr int N = Vec16<T>::N;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int groups = (k + KT - 1) / KT;
  const int n_items = n_tokens * groups;                 // < 2^30: T * k is
  for (int item = blockIdx.x * 8 + warp; item < n_items; item += gridDim.x * 8) {
    const int t = groups == 1 ? item : item / groups, j0 = groups == 1 ? 0 : (item % groups) * KT;
    int rows[KT];
    float g[KT], dot[KT];
#pragma unroll
    for (int j = 0; j < KT; ++j) {
      rows[j] = j0 + j < k ? row_of[(int64_t)t * k + j0 + j] : -1;
      g[j] = j0 + j < k ? gate[(int64_t)t * k + j0 + j] : 0.f;
      dot[j] = 0.f;
    }
    for (int v0 = lane; v0 < row_vecs; v0 += 32 * kVpl) {
      uint4 dv[kVpl], yv[KT][kVpl];
#pragma unroll
      for (int i = 0; i < kVpl; ++i) {
        const int v = v0 + 32 * i;
        dv[i] = v < row_vecs ? __ldg(dy + (int64_t)t * row_vecs + v) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int j = 0; j < KT; ++j)
          yv[j][i] = (rows[j] >= 0 && v < row_vecs) ? __ldg(Yp + (int64_t)rows[j] * row_vecs + v)
                                                    : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int i = 0; i < kVpl; ++i) {
        const int v = v0 + 32 * i;
        if (v >= row_vecs) continue;
        float a[N];
        Vec16<T>::unpack(dv[i], a);
#pragma unroll
        for (int j = 0; j < KT; ++j) {
          if (rows[j] < 0) continue;
          float fv[N], o[N];
          Vec16<T>::unpack(yv[j][i], fv);
#pragma unroll
          for (int q = 0; q < N; ++q) {
            dot[j] = fmaf(a[q], fv[q], dot[j]);
            o[q] = g[j] * a[q];
          }
          dYp[(int64_t)rows[j] * row_vecs + v] = Vec16<T>::pack(o);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < KT; ++j) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) dot[j] += __shfl_xor_sync(0xffffffffu, dot[j], o);
      if (lane == 0 && j0 + j < k) dgate[(int64_t)t * k + j0 + j] = dot[j];
    }
  }
  const int used = *offsets_end;
  for (int r = blockIdx.x * 8 + warp; r < used; r += gridDim.x * 8) {
    if (token_of[r] >= 0) continue;
    uint4* dst = dYp + (int64_t)r * row_vecs;
    for (int v = lane; v < row_vecs; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
  }
}

__global__ void dispatch_empty_kernel(int32_t* offsets, int32_t* token_of, int32_t* tile_expert, int M,
                                      int row_capacity) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i <= M) offsets[i] = 0;
  if (i < row_capacity) token_of[i] = -1;
  if (i < row_capacity / UNIPOOL_ROW_ALIGN) tile_expert[i] = -1;
}

static size_t place_smem_bytes(int M, int k, int chunk) {
  return ((size_t)kDispatchWarps * M + (M + 1) + 2 * (size_t)M + (size_t)chunk * k) * sizeof(int);
}

// Tokens per chunk (= per block of the two permute kernels): the largest of 256, 128, 64 that still
// gives every SM a block - a block moves its own tokens, and an SM alone pulls well under its share of
// the memory bandwidth; but every block reads the histograms of all chunks, so no more chunks than that.
static int dispatch_chunk_tokens(int T, int sm_count) {
  for (int chunk = kDispatchChunkTokens; chunk > kDispatchMinChunkTokens; chunk /= 2)
    if ((T + chunk - 1) / chunk >= sm_count) return chunk;
  return kDispatchMinChunkTokens;
}

static int row_mover_grid(const unipool_ctx* ctx, int64_t rows) {
  int64_t want = (rows + 7) / 8;
  int64_t cap = (int64_t)ctx->sm_count * 8;      // 8 resident 256-thread blocks per SM
  return (int)(want < 1 ? 1 : (want < cap ? want : cap));
}

int dispatch_launch(unipool_ctx* ctx, const void* x, int T, const int32_t* idx, int M,
                    int32_t* offsets, int32_t* row_of, int32_t* token_of, int32_t* tile_expert,
                    void* Xp, cudaStream_t s) {
  const int k = ctx->cfg.top_k, d = ctx->cfg.d_model;
  const int cap = (int)ctx->row_capacity;
  if (T == 0) {
    dispatch_empty_kernel<<<(cap + 255) / 256, 256, 0, s>>>(offsets, token_of, tile_expert, M, cap);
    UP_LAUNCH_CHECK();
    return UNIPOOL_OK;
  }
  const int chunk = dispatch_chunk_tokens(T, ctx->sm_count);
  const int n_blocks = (T + chunk - 1) / chunk;
  int32_t* bh = ctx->ws.block_hist;
  const int row_vecs = (int)((size_t)d * ctx->elem_bytes / 16);
  {
    PhaseTimer pt(ctx, UNIPOOL_PH_DISPATCH_MAPS, 1, s);
    dispatch_hist_kernel<<<n_blocks, kDispatchWarps * 32, kDispatchWarps * M * sizeof(int), s>>>(idx, T, k, M, chunk, bh,
                                                                                                ctx->ws.status);
    UP_LAUNCH_CHECK();
  }
  PhaseTimer pt(ctx, UNIPOOL_PH_DISPATCH_GATHER, 1, s);
  dispatch_place_kernel<<<n_blocks, kDispatchWarps * 32, place_smem_bytes(M, k, chunk), s>>>(
      idx, T, k, M, chunk, bh, n_blocks, static_cast<const uint4*>(x), row_vecs, cap, offsets, row_of, token_of, tile_expert,
      static_cast<uint4*>(Xp));
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

template <typename T>
static void combine_dispatch_k(int grid, cudaStream_t s, int k, const void* Yp, const int32_t* row_of,
                               const float* gate, const void* residual, void* y, int n_tokens, int row_vecs) {
  auto Y = static_cast<const uint4*>(Yp);
  auto R = static_cast<const uint4*>(residual);
  auto O = static_cast<uint4*>(y);
  if (k <= 1) combine_kernel<T, 1><<<grid, 256, 0, s>>>(Y, row_of, gate, R, O, n_tokens, k, row_vecs);
  else if (k <= 2) combine_kernel<T, 2><<<grid, 256, 0, s>>>(Y, row_of, gate, R, O, n_tokens, k, row_vecs);
  else if (k <= 4) combine_kernel<T, 4><<<grid, 256, 0, s>>>(Y, row_of, gate, R, O, n_tokens, k, row_vecs);
  else combine_kernel<T, 8><<<grid, 256, 0, s>>>(Y, row_of, gate, R, O, n_tokens, k, row_vecs);
}

static int combine_phase(unipool_ctx* ctx, int phase, const void* Yp, const int32_t* row_of,
                         const float* gate, int T, const void* residual, void* y, cudaStream_t s) {
  if (T == 0) return UNIPOOL_OK;
  PhaseTimer pt(ctx, phase, 1, s);
  const int k = ctx->cfg.top_k;
  const int row_vecs = (int)((size_t)ctx->cfg.d_model * ctx->elem_bytes / 16);
  const int grid = row_mover_grid(ctx, T);
  if (ctx->cfg.dtype == UNIPOOL_BF16)
    combine_dispatch_k<__nv_bfloat16>(grid, s, k, Yp, row_of, gate, residual, y, T, row_vecs);
  else
    combine_dispatch_k<float>(grid, s, k, Yp, row_of, gate, residual, y, T, row_vecs);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

int combine_launch(unipool_ctx* ctx, const void* Yp, const int32_t* row_of, const float* gate, int T,
                   const void* residual, void* y, cudaStream_t s) {
  return combine_phase(ctx, UNIPOOL_PH_COMBINE, Yp, row_of, gate, T, residual, y, s);
}

template <typename T>
static void combine_bwd_dispatch_k(int grid, cudaStream_t s, int k, const void* dy, const void* Yp,
                                   const int32_t* row_of, const float* gate, const int32_t* token_of,
                                   const int32_t* offsets_end, void* dYp, float* dgate, int n_tokens, int row_vecs) {
  auto D = static_cast<const uint4*>(dy);
  auto Y = static_cast<const uint4*>(Yp);
  auto O = static_cast<uint4*>(dYp);
  if (k <= 1) combine_bwd_kernel<T, 1><<<grid, 256, 0, s>>>(D, Y, row_of, gate, token_of, offsets_end, O, dgate, n_tokens, k, row_vecs);
  else combine_bwd_kernel<T, 2><<<grid, 256, 0, s>>>(D, Y, row_of, gate, token_of, offsets_end, O, dgate, n_tokens, k, row_vecs);
}

int combine_bwd_launch(unipool_ctx* ctx, const void* dy, int T, const int32_t* row_of,
                       const float* gate, const int32_t* token_of, const int32_t* offsets, int M,
                       const void* Yp, void* dYp, float* dgate, cudaStream_t s) {
  if (T == 0) return UNIPOOL_OK;
  const int k = ctx->cfg.top_k;
  const int row_vecs = (int)((size_t)ctx->cfg.d_model * ctx->elem_bytes / 16);
  const int grid = row_mover_grid(ctx, (int64_t)T * ((k + 1) / 2));     // one warp per token and pair of slots
  PhaseTimer pt(ctx, UNIPOOL_PH_BWD_SCALE_GATHER, 1, s);
  if (ctx->cfg.dtype == UNIPOOL_BF16)
    combine_bwd_dispatch_k<__nv_bfloat16>(grid, s, k, dy, Yp, row_of, gate, token_of, offsets + M, dYp, dgate, T, row_vecs);
  else
    combine_bwd_dispatch_k<float>(grid, s, k, dy, Yp, row_of, gate, token_of, offsets + M, dYp, dgate, T, row_vecs);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

int unpermute_sum_launch(unipool_ctx* ctx, const void* dXp, const int32_t* row_of, int T,
                         const void* residual, void* dx, cudaStream_t s) {
  // dx_t = residual_t + sum_j dXp[row_of[t,j]]: the combine kernel with unit weights
  return combine_phase(ctx, UNIPOOL_PH_UNPERMUTE_SUM, dXp, row_of, nullptr, T, residual, dx, s);
}

}  // namespace unipool

// ---------------------------------------------------------------- dispatch without a workspace
// Scratch of unipool_dispatch_static: the per-chunk histograms of the map kernels plus a status
// word, held in the library's own device image.  Every GPU that loads the library carries these
// 2 MiB until the process exits.  All calls share them.
namespace {
constexpr int64_t kStaticHistInts = 1024 * 512 - 64;      // chunks x experts that fit
static __device__ __align__(256) int32_t g_dispatch_scratch[1024 * 512];
constexpr int kMaxDevices = 64;
// per device: the array's address there, looked up by the first call on that device.
// Host threads may race on the first call: the entry is complete before its address becomes visible.
struct ScratchInfo { int32_t* addr; };
std::atomic<const ScratchInfo*> g_scratch[kMaxDevices];
ScratchInfo g_scratch_slots[kMaxDevices][2];
std::atomic<int> g_scratch_next[kMaxDevices];
}  // namespace

extern "C" int unipool_dispatch_static(const void* x, int32_t T, int32_t d_model, int32_t dtype, int32_t top_k,
                                       const int32_t* idx, int32_t n_experts, int64_t row_capacity,
                                       int32_t* offsets, int32_t* row_of, int32_t* token_of,
                                       int32_t* tile_expert, void* Xp, unipool_stream stream) {
  using namespace unipool;
  UP_REQUIRE(x && idx && offsets && row_of && token_of && tile_expert && Xp, UNIPOOL_ERR_INVALID_ARG,
             "dispatch_static: a tensor pointer is NULL");
  UP_REQUIRE(dtype == UNIPOOL_FP32 || dtype == UNIPOOL_BF16, UNIPOOL_ERR_INVALID_ARG, "dispatch_static: bad dtype %d", dtype);
  const size_t eb = dtype == UNIPOOL_BF16 ? 2 : 4;
  UP_REQUIRE(d_model > 0 && ((size_t)d_model * eb) % 16 == 0, UNIPOOL_ERR_UNSUPPORTED,
             "dispatch_static: a row of %d elements is not a whole number of 16-byte vectors", d_model);
  UP_REQUIRE(n_experts >= 1 && n_experts <= UNIPOOL_MAX_EXPERTS && top_k >= 1 && top_k <= UNIPOOL_MAX_TOPK &&
                 top_k <= n_experts, UNIPOOL_ERR_UNSUPPORTED, "dispatch_static: bad (n_experts, top_k) = (%d, %d)",
             n_experts, top_k);
  UP_REQUIRE(T >= 0 && (int64_t)T * top_k < (1ll << 30), UNIPOOL_ERR_UNSUPPORTED, "dispatch_static: bad T = %d", T);
  const int64_t need_rows = ((int64_t)T * top_k + (int64_t)n_experts * (UNIPOOL_ROW_ALIGN - 1) + UNIPOOL_ROW_ALIGN - 1) /
                            UNIPOOL_ROW_ALIGN * UNIPOOL_ROW_ALIGN;
  UP_REQUIRE(row_capacity % UNIPOOL_ROW_ALIGN == 0 && row_capacity >= need_rows && row_capacity < (1ll << 31),
             UNIPOOL_ERR_INVALID_ARG, "dispatch_static: row_capacity %lld, need a multiple of %d >= %lld",
             (long long)row_capacity, UNIPOOL_ROW_ALIGN, (long long)need_rows);
  const int n_blocks = (T + kDispatchChunkTokens - 1) / kDispatchChunkTokens;
  UP_REQUIRE((int64_t)n_blocks * n_experts <= kStaticHistInts, UNIPOOL_ERR_WORKSPACE,
             "dispatch_static: ceil(T/%d) * n_experts = %lld exceeds the built-in scratch of %lld entries "
             "(use unipool_dispatch with a workspace)", kDispatchChunkTokens, (long long)n_blocks * n_experts,
             (long long)kStaticHistInts);
  int dev = 0;
  UP_CUDA(cudaGetDevice(&dev));
  UP_REQUIRE(dev >= 0 && dev < kMaxDevices, UNIPOOL_ERR_UNSUPPORTED, "dispatch_static: device ordinal %d", dev);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const ScratchInfo* info = g_scratch[dev].load(std::memory_order_acquire);
  if (info == nullptr) {
    // Once per device, with that device current: in host code the array's name is only a handle,
    // the kernels need the address it has on THIS device.  Two threads that both get here look up the
    // same values; each fills a slot of its own and publishes it.
    int32_t* ptr = nullptr;
    UP_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_dispatch_scratch));
    UP_REQUIRE(ptr != nullptr, UNIPOOL_ERR_CUDA, "dispatch_static: no address for the built-in scratch");
    const int slot = g_scratch_next[dev].fetch_add(1) & 1;
    g_scratch_slots[dev][slot] = ScratchInfo{ptr};
    g_scratch[dev].store(&g_scratch_slots[dev][slot], std::memory_order_release);
    info = &g_scratch_slots[dev][slot];
  }
  int32_t* status = info->addr;                            // [0, 64): status word (+ spare)
  int32_t* bh = info->addr + 64;                           // per-chunk histograms / bases
  const int cap = (int)row_capacity;
  if (T == 0) {
    dispatch_empty_kernel<<<(cap + 255) / 256, 256, 0, s>>>(offsets, token_of, tile_expert, n_experts, cap);
    UP_LAUNCH_CHECK();
    return UNIPOOL_OK;
  }
  // the histograms are fully rewritten by the first kernel for the chunks of this call; nothing
  // else in the array has to start at zero
  dispatch_hist_kernel<<<n_blocks, kDispatchWarps * 32, kDispatchWarps * n_experts * sizeof(int), s>>>(
      idx, T, top_k, n_experts, kDispatchChunkTokens, bh, status);
  UP_LAUNCH_CHECK();
  const int row_vecs = (int)((size_t)d_model * eb / 16);
  dispatch_place_kernel<<<n_blocks, kDispatchWarps * 32, place_smem_bytes(n_experts, top_k, kDispatchChunkTokens), s>>>(
      idx, T, top_k, n_experts, kDispatchChunkTokens, bh, n_blocks, static_cast<const uint4*>(x), row_vecs, cap, offsets, row_of, token_of,
      tile_expert, static_cast<uint4*>(Xp));
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}
