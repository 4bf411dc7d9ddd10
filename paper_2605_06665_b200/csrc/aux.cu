// Pool-level balance loss (Eqs. 4-5) and the Monte-Carlo constant c (Alg. 1).
#include "common.cuh"
#include "tc_ptx.cuh"

namespace unipool {

// One block.  counts [L,M] int32, S [L,M] float.
__global__ void __launch_bounds__(512)
pool_aux_kernel(const int32_t* __restrict__ counts, const float* __restrict__ S, int L, int M, int T,
                int k, float alpha, const float* __restrict__ fbar_prev, float* __restrict__ loss,
                float* __restrict__ coef, float* __restrict__ fbar_out) {
  __shared__ double red[512];
  double term = 0.0;
  for (int i = threadIdx.x; i < M; i += blockDim.x) {
    double fsum = 0.0, psum = 0.0;
    for (int l = 0; l < L; ++l) {
      fsum += (double)counts[(int64_t)l * M + i];
      psum += (double)S[(int64_t)l * M + i];
    }
    const double fbar = fsum / ((double)T * k) / L;       // mean over layers of counts/(T k)
    const double pbar = psum / (double)T / L;             // mean over layers of S/T
    const double f_used = fbar_prev ? (double)fbar_prev[i] : fbar;
    fbar_out[i] = (float)fbar;
    coef[i] = (float)((double)alpha * M * f_used / ((double)L * T));
    term += f_used * pbar;
  }
  red[threadIdx.x] = term;
  __syncthreads();
  for (int o = blockDim.x / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *loss = (float)((double)alpha * M * red[0]);
}

int aux_launch(unipool_ctx* ctx, const int32_t* counts, const float* S, int L, int M, int T,
               float alpha, const float* fbar_prev, float* loss, float* coef, float* fbar_out,
               cudaStream_t s) {
  PhaseTimer pt(ctx, UNIPOOL_PH_POOL_AUX, 1, s);
  pool_aux_kernel<<<1, 512, 0, s>>>(counts, S, L, M, T, ctx->cfg.top_k, alpha, fbar_prev, loss, coef,
                                    fbar_out);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

// ---------------------------------------------------------------- distinct-expert accounting (App. E)
// U(x) = |{ pool experts token x selects in any layer }|; one thread per token keeps a bit set of
// the M <= 512 pool experts.  idx is [L, T, k] (router-local ids), expert_base[l] maps layer l's ids
// into the pool (0 everywhere for the shared pool).
__global__ void __launch_bounds__(256)
unique_experts_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ expert_base, int L, int T,
                      int k, int M, int32_t* __restrict__ unique, unsigned long long* __restrict__ total) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  int u = 0;
  if (t < T) {
    uint32_t bits[UNIPOOL_MAX_EXPERTS / 32];
#pragma unroll
    for (int w = 0; w < UNIPOOL_MAX_EXPERTS / 32; ++w) bits[w] = 0u;
    for (int l = 0; l < L; ++l) {
      const int base = expert_base ? expert_base[l] : 0;
      for (int j = 0; j < k; ++j) {
        const int e = base + idx[((int64_t)l * T + t) * k + j];
        if (e < 0 || e >= M) continue;               // dropped assignment
#pragma unroll
        for (int w = 0; w < UNIPOOL_MAX_EXPERTS / 32; ++w)
          if (w == (e >> 5)) bits[w] |= 1u << (e & 31);
      }
    }
#pragma unroll
    for (int w = 0; w < UNIPOOL_MAX_EXPERTS / 32; ++w) u += __popc(bits[w]);
    unique[t] = u;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) u += __shfl_xor_sync(0xffffffffu, u, o);
  if ((threadIdx.x & 31) == 0 && u) atomicAdd(total, (unsigned long long)u);
}

int unique_experts_launch(unipool_ctx* ctx, const int32_t* idx, const int32_t* expert_base, int L, int T,
                          int32_t* unique, unsigned long long* total, cudaStream_t s) {
  UP_CUDA(cudaMemsetAsync(total, 0, sizeof(unsigned long long), s));
  if (T == 0) return UNIPOOL_OK;
  unique_experts_kernel<<<(T + 255) / 256, 256, 0, s>>>(idx, expert_base, L, T, ctx->cfg.top_k, ctx->cfg.pool_size,
                                                       unique, total);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

// ---------------------------------------------------------------- Alg. 1
// Counter-based generator: a 64-bit mix of (seed, sample, element) gives two
// uniform 32-bit words, turned into one normal draw by Box-Muller.
__device__ __forceinline__ uint64_t mix64(uint64_t v) {
  v += 0x9E3779B97F4A7C15ull;
  v = (v ^ (v >> 30)) * 0xBF58476D1CE4E5B9ull;
  v = (v ^ (v >> 27)) * 0x94D049BB133111EBull;
  return v ^ (v >> 31);
}

__device__ __forceinline__ float normal_draw(uint64_t seed, uint64_t sample, uint32_t elem) {
  uint64_t h = mix64(mix64(seed ^ (sample * 0xD1342543DE82EF95ull)) + elem);
  float u1 = ((uint32_t)(h >> 32) + 1.0f) * (1.0f / 4294967808.0f);   // (0,1)
  float u2 = (uint32_t)h * (1.0f / 4294967296.0f);
  return sqrtf(-2.0f * __logf(u1)) * __cosf(6.283185307179586f * u2);
}

// One thread per sample: keeps the k largest positive components of x, then
// 1/||top-k(relu(x/||x||))|| = ||x|| / ||top-k(relu(x))||.
__global__ void __launch_bounds__(256)
calibrate_kernel(int E, int k, int n_samples, uint64_t seed, double* __restrict__ acc) {
  const int sidx = blockIdx.x * blockDim.x + threadIdx.x;
  double inv = 0.0, used = 0.0;
  if (sidx < n_samples) {
    float top[UNIPOOL_MAX_TOPK];
#pragma unroll
    for (int j = 0; j < UNIPOOL_MAX_TOPK; ++j) top[j] = 0.f;
    float ss = 0.f;
    for (int e = 0; e < E; ++e) {
      float v = normal_draw(seed, (uint64_t)sidx, (uint32_t)e);
      ss = fmaf(v, v, ss);
      float r = fmaxf(v, 0.f);
      // insertion into the descending list top[0..k)
#pragma unroll
      for (int j = 0; j < UNIPOOL_MAX_TOPK; ++j) {
        if (j < k && r > top[j]) { float tmp = top[j]; top[j] = r; r = tmp; }
      }
    }
    float ts = 0.f;
#pragma unroll
    for (int j = 0; j < UNIPOOL_MAX_TOPK; ++j) if (j < k) ts = fmaf(top[j], top[j], ts);
    if (ts > 0.f) { inv = (double)(sqrtf(ss) / sqrtf(ts)); used = 1.0; }
  }
  __shared__ double r0[256], r1[256];
  r0[threadIdx.x] = inv;
  r1[threadIdx.x] = used;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) { r0[threadIdx.x] += r0[threadIdx.x + o]; r1[threadIdx.x] += r1[threadIdx.x + o]; }
    __syncthreads();
  }
  if (threadIdx.x == 0) { atomicAdd(&acc[0], r0[0]); atomicAdd(&acc[1], r1[0]); }
}

int calibrate_launch(unipool_ctx* ctx, int E, int k, int n_samples, uint64_t seed, float* c_out,
                     cudaStream_t s) {
  double* acc = ctx->ws.dsigma_acc;     // two doubles, zero between calls
  calibrate_kernel<<<(n_samples + 255) / 256, 256, 0, s>>>(E, k, n_samples, seed, acc);
  UP_LAUNCH_CHECK();
  double host[2];
  UP_CUDA(cudaMemcpyAsync(host, acc, sizeof(host), cudaMemcpyDeviceToHost, s));
  UP_CUDA(cudaMemsetAsync(acc, 0, sizeof(host), s));
  UP_CUDA(cudaStreamSynchronize(s));
  UP_REQUIRE(host[1] > 0.0, UNIPOOL_ERR_DEVICE_CHECK, "calibrate_c: no usable sample");
  *c_out = (float)(host[0] / host[1]);
  return UNIPOOL_OK;
}

// Exercises the bounded wait every pipeline of the library is built on: one thread waits, for at most
// limit_cycles SM cycles, on an mbarrier that nobody arrives on.  The wait gives up, the kernel records
// the time-out in the status word the way the GEMM and router kernels do, and returns normally.
__global__ void wait_selftest_kernel(long long limit_cycles, int32_t* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    tc::mbar_init(&bar, 1);
    tc::fence_barrier_init();
    if (!tc::mbar_wait(&bar, 0, &abort_flag, limit_cycles)) {
      abort_flag = 1;
      if (atomicCAS(status, 0, kStatusTimeout) == 0) {
        status[1] = 99;                                   // site code of this self-test
        status[2] = 0;
      }
    }
  }
}

// Debug mode: one block per guard band, a thread per word; the first band found altered is reported in
// the status word (site kGuardSite + band, detail = byte offset inside the band).
struct GuardList { const unsigned* band[16]; };
__global__ void guard_check_kernel(GuardList gl, int32_t* status) {
  if (gl.band[blockIdx.x][threadIdx.x] != kGuardWord && atomicCAS(status, 0, kStatusCheck) == 0) {
    status[1] = kGuardSite + (int)blockIdx.x;
    status[2] = (int)threadIdx.x * 4;
  }
}

int guard_check_launch(unipool_ctx* ctx, cudaStream_t s) {
  GuardList gl{};
  for (int i = 0; i < ctx->ws.n_guards; ++i) gl.band[i] = reinterpret_cast<const unsigned*>(ctx->ws.guards[i]);
  guard_check_kernel<<<ctx->ws.n_guards, kGuardBytes / 4, 0, s>>>(gl, ctx->ws.status);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

int wait_selftest_launch(unipool_ctx* ctx, long long limit_cycles, cudaStream_t s) {
  wait_selftest_kernel<<<1, 32, 0, s>>>(limit_cycles, ctx->ws.status);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

}  // namespace unipool
