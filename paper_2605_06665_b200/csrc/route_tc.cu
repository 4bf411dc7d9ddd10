// NormRouter forward on the tensor cores (bf16 activations): one kernel computes the fp32
// logits z = x W_r^T (+ bias) of a 128-token tile into TMEM, then each epilogue thread owns
// one token and derives from its TMEM row the norm, the scores of Eq. 7, the top-k experts
// (ties to the lowest index), the gates and this tile's share of the per-expert statistics.
//
// The router weights are fp32.  They are split once per call into three bf16 terms
// W = W0 + W1 + W2 (each the bf16 rounding of what the previous terms left over), so that
// every product x * W_s is exact in fp32 and the tensor-core accumulation reproduces the fp32
// logits; terms that are zero everywhere (weights that are bf16 numbers already) are skipped.
#include <cfloat>
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace unipool {

namespace {

constexpr int kTile = 128;             // tokens per CTA = TMEM lanes
constexpr int kBK = 64;                // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int kMaxStages = 6;
constexpr uint32_t kXBytes = kTile * kBK * 2;
constexpr int kThreads = 192;          // warps 0-3 epilogue, warp 4 TMA producer, warp 5 MMA issuer

struct RouteParams {
  const float* bias;
  int T, M, d, k;
  float sigma_c, eps;
  int32_t* idx; float* gate; float* znorm; float* z_saved;
  int32_t* counts_out; float* sum_out;
  int32_t* part_counts; float* part_sums; uint32_t* ticket;   // per-tile statistics [tiles][M]
  const int32_t* split_any;            // [3] does split s hold a non-zero anywhere
  int stages;                          // operand stages that fit into shared memory
  uint32_t w_bytes;                    // bytes of one W k-block: ceil(M / 128) boxes of 128 rows
  uint32_t tmem_cols;                  // power of two >= max(32, ceil16(M))
  int32_t* status;
};

// W_r fp32 [M, d] -> three bf16 terms [3][M][d]; any[s] != 0 iff term s has a non-zero element.
__global__ void __launch_bounds__(256)
router_split_kernel(const float* __restrict__ W, int64_t n, __nv_bfloat16* __restrict__ out,
                    int32_t* __restrict__ any) {
  int flags = 0;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const float w = W[i];
    const __nv_bfloat16 h0 = __float2bfloat16_rn(w);
    const float r1 = w - __bfloat162float(h0);
    const __nv_bfloat16 h1 = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(h1);
    const __nv_bfloat16 h2 = __float2bfloat16_rn(r2);
    out[i] = h0;
    out[n + i] = h1;
    out[2 * n + i] = h2;
    if (__bfloat162float(h1) != 0.f) flags |= 2;
    if (__bfloat162float(h2) != 0.f) flags |= 4;
  }
  flags = __reduce_or_sync(0xffffffffu, flags);
  if ((threadIdx.x & 31) == 0) {
    if (flags & 2) atomicOr(&any[1], 1);
    if (flags & 4) atomicOr(&any[2], 1);
  }
}

__device__ __forceinline__ void route_timeout(const RouteParams& p, volatile int* abort, int site) {
  *abort = 1;
  if (atomicCAS(p.status, 0, kStatusTimeout) == 0) {
    p.status[1] = site;
    p.status[2] = (int)blockIdx.x;
  }
}

template <int KMAX, bool SOFTMAX>
__global__ void __launch_bounds__(kThreads, 1)
route_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                const __grid_constant__ CUtensorMap tmZ, const RouteParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t stage_bytes = kXBytes + p.w_bytes;
  uint8_t* zstage = smem + (size_t)p.stages * stage_bytes;        // [4 warps][2] 32 x 32 fp32 tiles of z
  uint8_t* tail = zstage + 4 * 2 * 4096;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(tail);
  uint64_t* empty_bar = full_bar + kMaxStages;
  uint64_t* tmem_full = empty_bar + kMaxStages;
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(tmem_full + 1);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_ptr + 1);
  int* last_flag = const_cast<int*>(abort) + 1;
  int* hist = reinterpret_cast<int*>(tail + 128);                  // [M]
  float* wsum = reinterpret_cast<float*>(hist + UNIPOOL_MAX_EXPERTS);   // [4][M] per-warp score sums
  float* sbias = wsum + 4 * p.M;                                         // [ceil32(M)] logit bias (zeros without one)

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int M = p.M;
  const int n_cols = (M + 15) / 16 * 16;                           // MMA N (all chunks together)
  const int kblocks = p.d / kBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { tc::mbar_init(&full_bar[s], 1); tc::mbar_init(&empty_bar[s], 1); }
    tc::mbar_init(tmem_full, 1);
    *abort = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmX);
    tc::tma_prefetch_desc(&tmW);
  }
  for (int i = threadIdx.x; i < M; i += blockDim.x) hist[i] = 0;
  for (int i = threadIdx.x; i < (M + 31) / 32 * 32; i += blockDim.x) sbias[i] = (p.bias && i < M) ? p.bias[i] : 0.f;
  if (warp == 5) {
    tc::tmem_alloc(tmem_ptr, p.tmem_cols);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;

  if (warp == 4) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int s = 0; s < 3 && ok; ++s) {
        if (s > 0 && p.split_any[s] == 0) continue;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!tc::mbar_wait(&empty_bar[stage], phase ^ 1u, abort)) { route_timeout(p, abort, 11); ok = false; break; }
          uint8_t* sX = smem + (size_t)stage * stage_bytes;
          uint8_t* sW = sX + kXBytes;
          tc::mbar_expect_tx(&full_bar[stage], stage_bytes);
          tc::tma_load_2d(sX, &tmX, &full_bar[stage], kb * kBK, blockIdx.x * kTile);
          for (uint32_t b = 0; b * 16384u < p.w_bytes; ++b)
            tc::tma_load_2d(sW + b * 16384u, &tmW, &full_bar[stage], kb * kBK, s * M + 128 * (int)b);
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok)
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const int n1 = n_cols < 256 ? n_cols : 256, n2 = n_cols - n1;
      const uint32_t idesc1 = tc::instr_desc_bf16(n1, false, false);
      const uint32_t idesc2 = tc::instr_desc_bf16(n2 > 0 ? n2 : 16, false, false);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      uint32_t accumulate = 0;
      for (int s = 0; s < 3 && ok; ++s) {
        if (s > 0 && p.split_any[s] == 0) continue;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!tc::mbar_wait(&full_bar[stage], phase, abort)) { route_timeout(p, abort, 12); ok = false; break; }
          tc::tc_fence_after_sync();
          const uint32_t xaddr = tc::smem_u32(smem + (size_t)stage * stage_bytes);
          const uint64_t xdesc = tc::smem_desc_sw128(xaddr, 16, 1024);
          const uint64_t wdesc = tc::smem_desc_sw128(xaddr + kXBytes, 16, 1024);
          const uint64_t wdesc2 = tc::smem_desc_sw128(xaddr + kXBytes + 256 * 128, 16, 1024);
#pragma unroll
          for (int j = 0; j < kBK / 16; ++j) {
            tc::umma_bf16(tmem_base, xdesc + 2 * j, wdesc + 2 * j, idesc1, accumulate);
            if (n2 > 0) tc::umma_bf16(tmem_base + 256, xdesc + 2 * j, wdesc2 + 2 * j, idesc2, accumulate);
            accumulate = 1;
          }
          tc::umma_commit(&empty_bar[stage]);
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (ok) tc::umma_commit(tmem_full);
    }
  } else {
    // ------------------------------------------------------------ epilogue: thread = token
    const int t = blockIdx.x * kTile + threadIdx.x;
    const bool live = t < p.T;
    float* my_wsum = wsum + warp * M;
    for (int i = lane; i < M; i += 32) my_wsum[i] = 0.f;
    bool ok = tc::mbar_wait(tmem_full, 0, abort);
    if (!ok && lane == 0) route_timeout(p, abort, 13);
    tc::tc_fence_after_sync();
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
    if (ok) {
      // pass 1: logits (+ bias) -> z_saved, squared norm (softmax: running maximum and the sum of
      // exponentials relative to it).  With a 16-byte row pitch (M % 4 == 0) the
      // 32 x 32 chunk is staged in shared memory (128-byte swizzle, conflict-free) and leaves by a
      // TMA store, which clips it at M columns and T rows.
      float ss = 0.f, mx = -INFINITY;
      float* zrow = p.z_saved + (int64_t)t * M;
      const bool vec = (M & 3) == 0;
      uint8_t* my_stage = zstage + warp * 2 * 4096;
      int nstore = 0;
      for (int c0 = 0; c0 < M; c0 += 32) {
        uint32_t rr[32];
        tc::tmem_ld_32x32(t_row + c0, rr);
        tc::tmem_ld_wait();
        float z[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          z[i] = c0 + i < M ? __uint_as_float(rr[i]) + sbias[c0 + i] : (SOFTMAX ? -INFINITY : 0.f);
          if (!SOFTMAX) ss = fmaf(z[i], z[i], ss);
        }
        if (SOFTMAX) {
          float cm = z[0];
#pragma unroll
          for (int i = 1; i < 32; ++i) cm = fmaxf(cm, z[i]);
          cm = fmaxf(cm, mx);
          float part = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) part += expf(z[i] - cm);
          ss = ss * expf(mx - cm) + part;                 // the first chunk rescales an empty sum
          mx = cm;
        }
        if (vec) {
          uint8_t* buf = my_stage + (nstore++ & 1) * 4096;
          if (lane == 0) tc::bulk_wait_read<1>();       // the store issued two chunks ago has drained `buf`
          __syncwarp();
#pragma unroll
          for (int q = 0; q < 8; ++q)
            *reinterpret_cast<float4*>(buf + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                make_float4(z[4 * q], z[4 * q + 1], z[4 * q + 2], z[4 * q + 3]);
          tc::fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            tc::tma_store_2d(&tmZ, buf, c0, blockIdx.x * kTile + warp * 32);
            tc::bulk_commit();
          }
        } else if (live) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (c0 + i < M) zrow[c0 + i] = z[i];
        }
      }
      const float n = SOFTMAX ? mx + logf(ss) : sqrtf(ss);           // softmax keeps log sum exp(z) here
      // NormRouter: a zero logit vector scores zero.  Softmax: 1 / sum of exponentials.
      const float scale = SOFTMAX ? 1.f / ss : (ss > 0.f ? p.sigma_c / (n + p.eps) : 0.f);
      if (live) p.znorm[t] = n;
      // pass 2: scores, top-k (score descending, expert index ascending), per-expert score sums
      float tv[KMAX];
      int ti[KMAX];
#pragma unroll
      for (int j = 0; j < KMAX; ++j) { tv[j] = -INFINITY; ti[j] = -1; }
      for (int c0 = 0; c0 < M; c0 += 32) {
        uint32_t rr[32];
        tc::tmem_ld_32x32(t_row + c0, rr);
        tc::tmem_ld_wait();
        float sv[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int e = c0 + i;
          const float z = __uint_as_float(rr[i]) + sbias[e < M ? e : 0];
          const float s = e < M ? scale * (SOFTMAX ? expf(z - mx) : fmaxf(z, 0.f)) : 0.f;
          float key = s == s ? s : -FLT_MAX;              // NaN scores sort last but stay selectable
          if (e >= M) key = -INFINITY;                    // never selected
          // Insert behind every entry that is >= key (equal keys keep the lower index in front) and
          // shift the displaced entries down by one.  For short lists this is a fixed sequence of
          // selects; long lists test the last entry first, since most scores do not enter.
          if (KMAX <= 2 || key > tv[KMAX - 1]) {
            float cv = key;
            int ci = e;
            bool moved = false;
#pragma unroll
            for (int j = 0; j < KMAX; ++j) {
              const bool sw = moved || cv > tv[j];
              const float fv = tv[j];
              const int fi = ti[j];
              tv[j] = sw ? cv : fv;
              ti[j] = sw ? ci : fi;
              cv = sw ? fv : cv;
              ci = sw ? fi : ci;
              moved = sw;
            }
          }
          sv[i] = live ? s : 0.f;
        }
        // column sums over the warp's 32 tokens: recursive halving, lane l ends with column c0 + l
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
          const bool upper = (lane & o) != 0;
#pragma unroll
          for (int j = 0; j < o; ++j) {
            const float send = upper ? sv[j] : sv[j + o];
            const float keep = upper ? sv[j + o] : sv[j];
            sv[j] = keep + __shfl_xor_sync(0xffffffffu, send, o);
          }
        }
        if (c0 + lane < M) my_wsum[c0 + lane] += sv[0];
      }
      if (live) {
        for (int j = 0; j < p.k; ++j) {
          int e = -1;
          float g = 0.f;
#pragma unroll
          for (int q = 0; q < KMAX; ++q)
            if (q == j) { e = ti[q]; g = tv[q]; }
          p.idx[(int64_t)t * p.k + j] = e;
          // the gate is the score itself (a NaN score was only re-keyed for the ordering)
          p.gate[(int64_t)t * p.k + j] = g == -FLT_MAX ? __int_as_float(0x7fc00000) : g;
          if (e >= 0) atomicAdd(&hist[e], 1);
        }
      }
    }
    if (lane == 0) tc::bulk_wait<0>();                   // the z tiles have left shared memory
    tc::tc_fence_before_sync();
    // the four epilogue warps publish the tile's statistics (named barrier 1: 128 threads)
    asm volatile("bar.sync 1, 128;" ::: "memory");
    for (int i = threadIdx.x; i < M; i += kTile) {
      p.part_counts[(int64_t)blockIdx.x * M + i] = hist[i];
      p.part_sums[(int64_t)blockIdx.x * M + i] = (wsum[i] + wsum[M + i]) + (wsum[2 * M + i] + wsum[3 * M + i]);
    }
    __threadfence();
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (threadIdx.x == 0) *last_flag = atomicAdd(p.ticket, 1u) == gridDim.x - 1 ? 1 : 0;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (*last_flag) {                     // the CTA that arrives last adds the tiles up
      // warp w sums the tiles b = w, w + 4, ... (independent loads), then the four partial sums of an
      // expert are added in warp order: the result does not depend on which CTA came last
      __threadfence();
      double* dsum = reinterpret_cast<double*>(zstage);  // [4][M] in the z staging tiles (they have drained)
      int* csum = reinterpret_cast<int*>(zstage + 4 * UNIPOOL_MAX_EXPERTS * sizeof(double));   // [4][M]
      if ((M & 3) == 0) {                  // 16-byte rows: a lane takes four neighbouring experts per load
        for (int i = 4 * lane; i < M; i += 128) {
          int4 cnt = make_int4(0, 0, 0, 0);
          double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
#pragma unroll 8
          for (int b = warp; b < (int)gridDim.x; b += 4) {
            const int4 c = __ldcg(reinterpret_cast<const int4*>(p.part_counts + (int64_t)b * M + i));
            const float4 v = __ldcg(reinterpret_cast<const float4*>(p.part_sums + (int64_t)b * M + i));
            cnt.x += c.x; cnt.y += c.y; cnt.z += c.z; cnt.w += c.w;
            s0 += (double)v.x; s1 += (double)v.y; s2 += (double)v.z; s3 += (double)v.w;
          }
          csum[warp * M + i] = cnt.x; csum[warp * M + i + 1] = cnt.y;
          csum[warp * M + i + 2] = cnt.z; csum[warp * M + i + 3] = cnt.w;
          dsum[warp * M + i] = s0; dsum[warp * M + i + 1] = s1;
          dsum[warp * M + i + 2] = s2; dsum[warp * M + i + 3] = s3;
        }
      } else {
        for (int i = lane; i < M; i += 32) {
          int cnt = 0;
          double sum = 0.0;
#pragma unroll 8
          for (int b = warp; b < (int)gridDim.x; b += 4) {
            cnt += __ldcg(&p.part_counts[(int64_t)b * M + i]);
            sum += (double)__ldcg(&p.part_sums[(int64_t)b * M + i]);
          }
          csum[warp * M + i] = cnt;
          dsum[warp * M + i] = sum;
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      for (int i = threadIdx.x; i < M; i += kTile) {
        p.counts_out[i] = (csum[i] + csum[M + i]) + (csum[2 * M + i] + csum[3 * M + i]);
        p.sum_out[i] = (float)((dsum[i] + dsum[M + i]) + (dsum[2 * M + i] + dsum[3 * M + i]));
      }
      if (threadIdx.x == 0) *p.ticket = 0u;
    }
  }

  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 5) {
    tc::tc_fence_after_sync();
    tc::tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

// dz of the router's derivative as bf16 [T, Mp] (columns >= M are zero); four lanes per token, each
// taking four neighbouring experts per step when the rows are 16-byte aligned (M % 4 == 0).
template <bool SOFTMAX, int KT>
__global__ void __launch_bounds__(256)
router_dz16_kernel(const float* __restrict__ z, const float* __restrict__ znorm, const int32_t* __restrict__ idx,
                   const float* __restrict__ dgate, const float* __restrict__ coef, int T, int M, int Mp, int k,
                   float sigma, float c, float eps, __nv_bfloat16* __restrict__ dz16, float* __restrict__ dsigma,
                   double* __restrict__ acc, uint32_t* __restrict__ ticket) {
  const int gid = blockIdx.x * blockDim.x + threadIdx.x;
  const int sub = gid & 3;
  const bool live = (gid >> 2) < T;
  const int t = live ? gid >> 2 : T - 1;
  const float* zr = z + (int64_t)t * M;
  int e_sel[KT];
  float dg_sel[KT];
#pragma unroll
  for (int j = 0; j < KT; ++j) {
    e_sel[j] = j < k ? idx[(int64_t)t * k + j] : -1;
    dg_sel[j] = j < k ? dgate[(int64_t)t * k + j] : 0.f;
  }
  auto ds_of = [&](int i) {
    float ds = coef ? __ldg(coef + i) : 0.f;
#pragma unroll
    for (int j = 0; j < KT; ++j)
      if (e_sel[j] == i) ds += dg_sel[j];
    return ds;
  };
  const float n = znorm[t];                       // ||z||; softmax: log sum exp(z)
  const bool vec = (M & 3) == 0;
  float q = 0.f;
  if (vec) {
    for (int i = 4 * sub; i < M; i += 16) {
      const float4 zv = *reinterpret_cast<const float4*>(zr + i);
      const float zz[4] = {zv.x, zv.y, zv.z, zv.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) q = fmaf(ds_of(i + u), SOFTMAX ? expf(zz[u] - n) : fmaxf(zz[u], 0.f), q);
    }
  } else {
    for (int i = sub; i < M; i += 4) q = fmaf(ds_of(i), SOFTMAX ? expf(zr[i] - n) : fmaxf(zr[i], 0.f), q);
  }
  q += __shfl_xor_sync(0xffffffffu, q, 1);
  q += __shfl_xor_sync(0xffffffffu, q, 2);
  const float ne = n + eps;
  const float scale = sigma * c;
  const float qn = n > 0.f ? q / (n * ne * ne) : 0.f;
  auto dz_of = [&](int i, float zi) {
    if (SOFTMAX) return expf(zi - n) * (ds_of(i) - q);
    return n > 0.f ? scale * ((zi > 0.f ? ds_of(i) / ne : 0.f) - zi * qn) : 0.f;
  };
  if (live) {
    __nv_bfloat16* out = dz16 + (int64_t)t * Mp;
    if (vec) {                                     // Mp is a multiple of 64: rows of dz16 are 8-byte aligned
      for (int i = 4 * sub; i < Mp; i += 16) {
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (i < M) {
          const float4 zv = *reinterpret_cast<const float4*>(zr + i);
          v[0] = dz_of(i, zv.x); v[1] = dz_of(i + 1, zv.y); v[2] = dz_of(i + 2, zv.z); v[3] = dz_of(i + 3, zv.w);
        }
        const __nv_bfloat162 lo = __floats2bfloat162_rn(v[0], v[1]), hi = __floats2bfloat162_rn(v[2], v[3]);
        uint2 w;
        w.x = *reinterpret_cast<const uint32_t*>(&lo);
        w.y = *reinterpret_cast<const uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(out + i) = w;
      }
    } else {
      for (int i = sub; i < Mp; i += 4) out[i] = __float2bfloat16_rn(i < M ? dz_of(i, zr[i]) : 0.f);
    }
  }
  float part = (live && sub == 0 && !SOFTMAX) ? c * q / ne : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
  __shared__ float wpart[8];
  if ((threadIdx.x & 31) == 0) wpart[threadIdx.x / 32] = part;
  __syncthreads();
  if (threadIdx.x == 0) {
    double sum = 0.0;
    for (int w = 0; w < (int)(blockDim.x / 32); ++w) sum += (double)wpart[w];
    atomicAdd(acc, sum);
    __threadfence();
    if (atomicAdd(ticket, 1u) == gridDim.x - 1) {
      __threadfence();
      *dsigma += (float)__ldcg(acc);
      *acc = 0.0;
      *ticket = 0u;
    }
  }
}

}  // namespace

// Splits W_r into ws.w_split (three bf16 terms) and sets ws.split_any.
int router_split_launch(unipool_ctx* ctx, const float* W_r, int M, cudaStream_t s) {
  const int64_t n = (int64_t)M * ctx->cfg.d_model;
  UP_CUDA(cudaMemsetAsync(ctx->ws.split_any, 0, 4 * sizeof(int32_t), s));
  const int blocks = (int)((n + 255) / 256 < 592 ? (n + 255) / 256 : 592);
  router_split_kernel<<<blocks, 256, 0, s>>>(W_r, n, static_cast<__nv_bfloat16*>(ctx->ws.w_split), ctx->ws.split_any);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

int route_tc_launch(unipool_ctx* ctx, const void* x, int T, const float* W_r, float sigma, const float* bias,
                    int M, int32_t* idx, float* gate, int32_t* counts, float* score_sum, float* znorm,
                    float* z_saved, cudaStream_t s) {
  const int d = ctx->cfg.d_model, k = ctx->cfg.top_k;
  RouteParams p{};
  p.bias = bias; p.T = T; p.M = M; p.d = d; p.k = k;
  p.sigma_c = sigma * ctx->cfg.c; p.eps = ctx->cfg.eps;
  p.idx = idx; p.gate = gate; p.znorm = znorm; p.z_saved = z_saved;
  p.counts_out = counts; p.sum_out = score_sum;
  p.part_counts = ctx->ws.part_counts; p.part_sums = ctx->ws.part_sums; p.ticket = ctx->ws.tickets + 0;
  p.split_any = ctx->ws.split_any;
  p.status = ctx->ws.status;
  p.w_bytes = (uint32_t)((M + 127) / 128) * 16384u;
  const uint32_t stage_bytes = kXBytes + p.w_bytes;
  const uint32_t tail_bytes = 4 * 2 * 4096 + 128 + UNIPOOL_MAX_EXPERTS * 4 + 4 * M * 4 + (M + 31) / 32 * 32 * 4;
  const uint32_t budget = 227 * 1024 - 1024 - tail_bytes;
  p.stages = (int)(budget / stage_bytes);
  if (p.stages > kMaxStages) p.stages = kMaxStages;
  UP_REQUIRE(p.stages >= 2, UNIPOOL_ERR_UNSUPPORTED, "router of %d experts does not fit the logits kernel", M);
  const int n_cols = (M + 15) / 16 * 16;
  p.tmem_cols = 32;
  while ((int)p.tmem_cols < n_cols) p.tmem_cols *= 2;
  int rc;
  {
    PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_LOGITS, 1, s);
    if ((rc = router_split_launch(ctx, W_r, M, s)) != UNIPOOL_OK) return rc;
  }
  CUtensorMap tmX, tmW, tmZ;
  if ((M & 3) == 0) {
    if ((rc = tc_f32_chunk_map(ctx, &tmZ, z_saved, M, T)) != UNIPOOL_OK) return rc;
  } else {
    tmZ = CUtensorMap{};                 // not used: rows of z are not 16-byte aligned, plain stores instead
  }
  if ((rc = tc_operand_map(ctx, &tmX, x, d, T, kTile)) != UNIPOOL_OK) return rc;
  if ((rc = tc_operand_map(ctx, &tmW, ctx->ws.w_split, d, (uint64_t)3 * M, 128)) != UNIPOOL_OK) return rc;
  PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_SELECT, 1, s);
  const size_t smem = (size_t)p.stages * stage_bytes + tail_bytes + 1024;
  const int grid = (T + kTile - 1) / kTile;
  const bool softmax = ctx->cfg.router_mode == UNIPOOL_ROUTER_SOFTMAX;
  auto kern = k <= 2 ? (softmax ? route_tc_kernel<2, true> : route_tc_kernel<2, false>)
                     : (softmax ? route_tc_kernel<UNIPOOL_MAX_TOPK, true> : route_tc_kernel<UNIPOOL_MAX_TOPK, false>);
  UP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<grid, kThreads, smem, s>>>(tmX, tmW, tmZ, p);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

int route_bwd_tc_launch(unipool_ctx* ctx, const void* x, int T, const float* W_r, float sigma, int M,
                        const float* znorm, const float* z_saved, const int32_t* idx, const float* dgate,
                        const float* coef, void* dx, float* dW_r, float* dsigma, cudaStream_t s) {
  const int k = ctx->cfg.top_k;
  const int Mp = (M + 63) / 64 * 64;
  __nv_bfloat16* dz16 = reinterpret_cast<__nv_bfloat16*>(ctx->ws.dz);
  int rc;
  {
    PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_BWD_DZ, 2, s);
    if ((rc = router_split_launch(ctx, W_r, M, s)) != UNIPOOL_OK) return rc;   // term 0 = bf16(W_r)
    const int64_t threads = (int64_t)T * 4;
    const bool softmax = ctx->cfg.router_mode == UNIPOOL_ROUTER_SOFTMAX;
    auto kern = k <= 2 ? (softmax ? router_dz16_kernel<true, 2> : router_dz16_kernel<false, 2>)
                       : (softmax ? router_dz16_kernel<true, UNIPOOL_MAX_TOPK> : router_dz16_kernel<false, UNIPOOL_MAX_TOPK>);
    kern<<<(int)((threads + 255) / 256), 256, 0, s>>>(
        z_saved, znorm, idx, dgate, coef, T, M, Mp, k, sigma, ctx->cfg.c, ctx->cfg.eps, dz16, dsigma,
        ctx->ws.dsigma_acc, ctx->ws.tickets + 1);
    UP_LAUNCH_CHECK();
  }
  return router_bwd_gemms_tc(ctx, dz16, Mp, ctx->ws.w_split, x, T, M, dx, dW_r, s);
}

}  // namespace unipool
