// CUDA-core tiled GEMM building block (fp32 accumulation, arbitrary strides).
// Used where exact fp32 arithmetic is required (the fp32 mode of the library,
// whose 1e-5 parity bound rules out TF32) and for the small router GEMMs.
#pragma once

#include "common.cuh"

namespace unipool {

constexpr int kSimtTile = 64;     // output tile is 64 x 64
constexpr int kSimtKC = 16;       // k-chunk staged in shared memory
constexpr int kSimtThreads = 256; // 16 x 16 threads, 4 x 4 outputs each

// Element (m,k) of A is A[m*a_sm + k*a_sk]; element (k,n) of B is B[k*b_sk + n*b_sn].
template <typename TA, typename TB>
struct SimtOperands {
  const TA* A; int64_t a_sm, a_sk;
  const TB* B; int64_t b_sk, b_sn;
};

// Accumulates the 64x64 tile with origin (m0, n0) over k in [k_begin, k_end) into
// acc[4][4]; thread (ty, tx) owns rows m0 + ty*4 + i and columns n0 + tx*4 + j.
// Rows >= m_end and columns >= n_end read as zero.
template <typename TA, typename TB>
__device__ __forceinline__ void simt_tile_mainloop(const SimtOperands<TA, TB>& op, int m0, int n0,
                                                   int m_end, int n_end, int k_begin, int k_end,
                                                   float (&acc)[4][4]) {
  __shared__ float As[kSimtKC][kSimtTile + 4];
  __shared__ float Bs[kSimtKC][kSimtTile + 4];
  const int tid = threadIdx.x;
  const int ty = tid / 16, tx = tid % 16;
  // loader mapping: pick the fast index along the operand's contiguous dimension
  const bool a_k_fast = op.a_sk == 1;
  const bool b_n_fast = op.b_sn == 1;
  for (int k0 = k_begin; k0 < k_end; k0 += kSimtKC) {
#pragma unroll
    for (int it = 0; it < (kSimtTile * kSimtKC) / kSimtThreads; ++it) {
      int e = tid + it * kSimtThreads;
      int mm, kk;
      if (a_k_fast) { kk = e % kSimtKC; mm = e / kSimtKC; } else { mm = e % kSimtTile; kk = e / kSimtTile; }
      int m = m0 + mm, k = k0 + kk;
      float v = 0.f;
      if (m < m_end && k < k_end) v = to_f32(op.A[(int64_t)m * op.a_sm + (int64_t)k * op.a_sk]);
      As[kk][mm] = v;
      int nn, kb;
      if (b_n_fast) { nn = e % kSimtTile; kb = e / kSimtTile; } else { kb = e % kSimtKC; nn = e / kSimtKC; }
      int n = n0 + nn;
      k = k0 + kb;
      v = 0.f;
      if (n < n_end && k < k_end) v = to_f32(op.B[(int64_t)k * op.b_sk + (int64_t)n * op.b_sn]);
      Bs[kb][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kSimtKC; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
}

}  // namespace unipool
