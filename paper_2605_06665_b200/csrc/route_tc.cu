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

constexpr int kTile = 128;             // tokens per CTA tile = TMEM lanes
constexpr int kBK = 64;                // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int kMaxStages = 8;
constexpr uint32_t kXBytes = kTile * kBK * 2;
constexpr int kEpiWarps = 8;           // two per TMEM lane quarter: they take alternate 32-expert chunks
constexpr int kThreads = 64 + 32 * kEpiWarps;   // warp 0 TMA producer, warp 1 MMA issuer, warps 2-9 epilogue
constexpr uint32_t kZStage = 4096;     // one 32 x 32 fp32 chunk of z per epilogue warp

struct RouteParams {
  const float* bias;
  int T, M, d, k;
  float sigma_c, eps;
  int32_t* idx; float* gate; float* znorm; float* z_saved;
  int32_t* counts_out; float* sum_out;
  int32_t* acc_counts; long long* acc_sums; uint32_t* ticket;   // [M] accumulators of all CTAs (start at zero,
                                                                // left at zero), [0] CTAs done, [1] non-finite sum
  const int32_t* split_any;            // [3] does split s hold a non-zero anywhere
  int stages;                          // operand stages that fit into shared memory
  int n1, n2;                          // MMA N of the first (<= 256) and second instruction; n1 + n2 = ceil16(M)
  uint32_t stage_bytes;
  int32_t* status;
};

// W_r fp32 [n_layers][M*d] -> three bf16 terms per layer [n_layers][3][M*d]; any[4 l + s] != 0 iff term
// s of layer l has a non-zero element.
__global__ void __launch_bounds__(256)
router_split_kernel(const float* __restrict__ W, int64_t n, int n_layers, __nv_bfloat16* __restrict__ out,
                    int32_t* __restrict__ any) {
  const int64_t total = n * n_layers;
  for (int64_t base = (int64_t)blockIdx.x * blockDim.x; base < total; base += (int64_t)gridDim.x * blockDim.x) {
    const int64_t g = base + threadIdx.x;
    int flags = 0;
    const int64_t l = (g < total ? g : total - 1) / n;
    if (g < total) {
      const int64_t i = g - l * n;
      const float w = W[g];
      const __nv_bfloat16 h0 = __float2bfloat16_rn(w);
      const float r1 = w - __bfloat162float(h0);
      const __nv_bfloat16 h1 = __float2bfloat16_rn(r1);
      const float r2 = r1 - __bfloat162float(h1);
      const __nv_bfloat16 h2 = __float2bfloat16_rn(r2);
      __nv_bfloat16* o = out + l * 3 * n;
      o[i] = h0;
      o[n + i] = h1;
      o[2 * n + i] = h2;
      if (__bfloat162float(h1) != 0.f) flags |= 2;
      if (__bfloat162float(h2) != 0.f) flags |= 4;
    }
    // a warp may straddle two layers: every lane reports for its own
    if (flags & 2) atomicOr(&any[4 * l + 1], 1);
    if (flags & 4) atomicOr(&any[4 * l + 2], 1);
  }
}

__device__ __forceinline__ void route_timeout(const RouteParams& p, volatile int* abort, int site) {
  *abort = 1;
  if (atomicCAS(p.status, 0, kStatusTimeout) == 0) {
    p.status[1] = site;
    p.status[2] = (int)blockIdx.x;
  }
}

// Inserts (key, e) into the descending list (tv, ti): in front of every entry with a smaller key or an
// equal key and a larger expert index, so that equal scores keep the lower index in front.
template <int KMAX>
__device__ __forceinline__ void topk_insert(float (&tv)[KMAX], int (&ti)[KMAX], float key, int e) {
  float cv = key;
  int ci = e;
  bool moved = false;
#pragma unroll
  for (int j = 0; j < KMAX; ++j) {
    const bool sw = moved || cv > tv[j] || (cv == tv[j] && ci < ti[j] && ti[j] >= 0) || (ti[j] < 0 && cv >= tv[j]);
    const float fv = tv[j];
    const int fi = ti[j];
    tv[j] = sw ? cv : fv;
    ti[j] = sw ? ci : fi;
    cv = sw ? fv : cv;
    ci = sw ? fi : ci;
    moved = sw;
  }
}

// One CTA pair (cta_group::2, M = 256) scores 256 tokens per tile: each CTA holds 128 tokens in its own
// TMEM lanes and loads its own x rows plus HALF of the router weights' rows of a k-block.  The pairs are
// persistent; with at most 256 logit columns the accumulator is double-buffered, so the per-token
// epilogue of one tile overlaps the loads and MMAs of the next.  Eight epilogue warps: the two warps
// of a TMEM lane quarter share its 32 tokens and take alternate 32-expert chunks; they combine their
// partial norms and top-k lists through shared memory.  The per-expert statistics of all CTAs are
// added up with integer atomics (the score sums in fixed point), so they do not depend on timing.
template <int KMAX, bool SOFTMAX>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
route_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW1,
                const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmZ,
                const RouteParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int M = p.M;
  uint8_t* zstage = smem + (size_t)p.stages * p.stage_bytes;      // [8 warps] 32 x 32 fp32 tiles of z
  uint8_t* tail = zstage + kEpiWarps * kZStage;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(tail);
  uint64_t* empty_bar = full_bar + kMaxStages;
  uint64_t* tmem_full = empty_bar + kMaxStages;                     // [2]
  uint64_t* tmem_empty = tmem_full + 2;                             // [2]
  uint64_t* xbar = tmem_empty + 2;                                  // [4 quarters][2 sync points]
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(xbar + 8);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_ptr + 1);
  int* last_flag = const_cast<int*>(abort) + 1;
  float* xnorm = reinterpret_cast<float*>(tail + 256);              // [2 halves][128 tokens][2] partial norm terms
  float* xtopv = xnorm + 2 * kTile * 2;                             // [128 tokens][KMAX] keys of the second warp
  int* xtopi = reinterpret_cast<int*>(xtopv + kTile * UNIPOOL_MAX_TOPK);
  int* hist = xtopi + kTile * UNIPOOL_MAX_TOPK;                     // [M]
  float* wsum = reinterpret_cast<float*>(hist + UNIPOOL_MAX_EXPERTS);   // [8 warps][M] score sums
  float* sbias = wsum + kEpiWarps * M;                              // [ceil32(M)] logit bias (zeros without one)

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int rank = (int)tc::cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_cols = p.n1 + p.n2;
  const int kblocks = p.d / kBK;
  const int n_tp = (p.T + 2 * kTile - 1) / (2 * kTile);             // tile pairs
  const bool two_acc = n_cols <= 256;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { tc::mbar_init(&full_bar[s], 1); tc::mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { tc::mbar_init(&tmem_full[a], 1); tc::mbar_init(&tmem_empty[a], 2 * kEpiWarps); }
    for (int i = 0; i < 8; ++i) tc::mbar_init(&xbar[i], 2);
    *abort = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmX);
    tc::tma_prefetch_desc(&tmW1);
  }
  for (int i = threadIdx.x; i < M; i += blockDim.x) hist[i] = 0;
  for (int i = threadIdx.x; i < kEpiWarps * M; i += blockDim.x) wsum[i] = 0.f;
  for (int i = threadIdx.x; i < (M + 31) / 32 * 32; i += blockDim.x) sbias[i] = (p.bias && i < M) ? p.bias[i] : 0.f;
  if (warp == 1) {
    tc::tmem_alloc_pair(tmem_ptr, 512);
    tc::tmem_relinquish_pair();
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync();                                               // both CTAs' barriers exist before any remote use
  tc::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;
  const uint32_t w1_bytes = (uint32_t)(p.n1 / 2) * (kBK * 2), w2_bytes = (uint32_t)(p.n2 / 2) * (kBK * 2);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (one in each CTA)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tp = pair; tp < n_tp && ok; tp += n_pairs) {
        const int t0 = tp * 2 * kTile + rank * kTile;
        for (int s = 0; s < 3 && ok; ++s) {
          if (s > 0 && p.split_any[s] == 0) continue;
          for (int kb = 0; kb < kblocks; ++kb) {
            if (!tc::mbar_wait(&empty_bar[stage], phase ^ 1u, abort)) { route_timeout(p, abort, 11); ok = false; break; }
            uint8_t* sX = smem + (size_t)stage * p.stage_bytes;
            uint8_t* sW = sX + kXBytes;
            if (rank == 0) tc::mbar_expect_tx(&full_bar[stage], 2 * (kXBytes + w1_bytes + w2_bytes));
            tc::tma_load_2d_pair(sX, &tmX, &full_bar[stage], kb * kBK, t0);
            tc::tma_load_2d_pair(sW, &tmW1, &full_bar[stage], kb * kBK, s * M + rank * (p.n1 / 2));
            if (p.n2 > 0)
              tc::tma_load_2d_pair(sW + w1_bytes, &tmW2, &full_bar[stage], kb * kBK, s * M + p.n1 + rank * (p.n2 / 2));
            if (++stage == p.stages) { stage = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok)
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc1 = tc::instr_desc_bf16(p.n1, false, false, 256);
      const uint32_t idesc2 = tc::instr_desc_bf16(p.n2 > 0 ? p.n2 : 16, false, false, 256);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int local = 0;
      for (int tp = pair; tp < n_tp && ok; tp += n_pairs) {
        const int acc = two_acc ? (local & 1) : 0;
        const uint32_t acc_phase = two_acc ? ((local >> 1) & 1) : (local & 1);
        ++local;
        if (!tc::mbar_wait(&tmem_empty[acc], acc_phase ^ 1u, abort)) { route_timeout(p, abort, 14); break; }
        tc::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * 256;
        uint32_t accumulate = 0;
        for (int s = 0; s < 3 && ok; ++s) {
          if (s > 0 && p.split_any[s] == 0) continue;
          for (int kb = 0; kb < kblocks; ++kb) {
            if (!tc::mbar_wait(&full_bar[stage], phase, abort)) { route_timeout(p, abort, 12); ok = false; break; }
            tc::tc_fence_after_sync();
            const uint32_t xaddr = tc::smem_u32(smem + (size_t)stage * p.stage_bytes);
            const uint64_t xdesc = tc::smem_desc_sw128(xaddr, 16, 1024);
            const uint64_t wdesc = tc::smem_desc_sw128(xaddr + kXBytes, 16, 1024);
            const uint64_t wdesc2 = tc::smem_desc_sw128(xaddr + kXBytes + w1_bytes, 16, 1024);
#pragma unroll
            for (int j = 0; j < kBK / 16; ++j) {
              tc::umma_bf16_pair(d_tmem, xdesc + 2 * j, wdesc + 2 * j, idesc1, accumulate);
              if (p.n2 > 0) tc::umma_bf16_pair(d_tmem + 256, xdesc + 2 * j, wdesc2 + 2 * j, idesc2, accumulate);
              accumulate = 1;
            }
            tc::umma_commit_pair(&empty_bar[stage], 3);
            if (++stage == p.stages) { stage = 0; phase ^= 1u; }
          }
        }
        if (ok) tc::umma_commit_pair(&tmem_full[acc], 3);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue: thread = token, two warps per quarter
    const int quarter = warp & 3;
    const int half = (warp - 2) >> 2;                               // 0 takes chunks 0, 2, ..; 1 takes 1, 3, ..
    const int tok_in_tile = quarter * 32 + lane;
    float* my_wsum = wsum + (warp - 2) * M;
    uint8_t* my_stage = zstage + (warp - 2) * kZStage;
    uint64_t* qbar = xbar + 2 * quarter;
    const bool vec = (M & 3) == 0;
    const int n_chunks = (M + 31) / 32;
    bool ok = true;
    int local = 0;
    for (int tp = pair; tp < n_tp && ok; tp += n_pairs) {
      const int acc = two_acc ? (local & 1) : 0;
      const uint32_t acc_phase = two_acc ? ((local >> 1) & 1) : (local & 1);
      const uint32_t xphase = local & 1;
      ++local;
      const int t = tp * 2 * kTile + rank * kTile + tok_in_tile;
      const bool live = t < p.T;
      if (!tc::mbar_wait(&tmem_full[acc], acc_phase, abort)) {
        if (lane == 0) route_timeout(p, abort, 13);
        break;
      }
      tc::tc_fence_after_sync();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * 256;
      // pass 1 over this warp's chunks: logits (+ bias) -> z_saved, squared norm (softmax: running maximum
      // and the sum of exponentials relative to it), and the selection - the order of the scores is the
      // order of max(z, 0) (of z for the softmax), so the top-k list needs no scale yet.
      float ss = 0.f, mx = -INFINITY;
      float tv[KMAX];
      int ti[KMAX];
#pragma unroll
      for (int j = 0; j < KMAX; ++j) { tv[j] = -INFINITY; ti[j] = -1; }
      float* zrow = p.z_saved + (int64_t)t * M;
      for (int c = half; c < n_chunks; c += 2) {
        const int c0 = 32 * c;
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
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int e = c0 + i;
          const float u = SOFTMAX ? z[i] : fmaxf(z[i], 0.f);
          float key = u == u ? u : -FLT_MAX;              // NaN logits sort last but stay selectable
          if (e >= M) key = -INFINITY;                    // never selected
          // a later equal key stays behind (experts are visited in ascending order)
          if (KMAX <= 2) {                                // two selects per entry, no branch
            const bool g0 = key > tv[0], g1 = key > tv[KMAX - 1];
            tv[KMAX - 1] = g0 ? tv[0] : (g1 ? key : tv[KMAX - 1]);
            ti[KMAX - 1] = g0 ? ti[0] : (g1 ? e : ti[KMAX - 1]);
            tv[0] = g0 ? key : tv[0];
            ti[0] = g0 ? e : ti[0];
          } else if (key > tv[KMAX - 1]) {                // most keys do not enter: test the last entry first
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
        }
        if (vec) {
          // the 32 x 32 chunk is staged in shared memory (128-byte swizzle, conflict-free) and leaves by a
          // TMA store, which clips it at M columns and T rows
          if (lane == 0) tc::bulk_wait_read<0>();         // the previous chunk's store has drained the tile
          __syncwarp();
#pragma unroll
          for (int q = 0; q < 8; ++q)
            *reinterpret_cast<float4*>(my_stage + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                make_float4(z[4 * q], z[4 * q + 1], z[4 * q + 2], z[4 * q + 3]);
          tc::fence_proxy_async();
          __syncwarp();
          const int zrow0 = tp * 2 * kTile + rank * kTile + quarter * 32;
          if (lane == 0 && zrow0 < p.T) {                 // a store never starts outside the tensor
            tc::tma_store_2d(&tmZ, my_stage, c0, zrow0);
            tc::bulk_commit();
          }
        } else if (live) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (c0 + i < M) zrow[c0 + i] = z[i];
        }
      }
      // the two warps of the quarter exchange their partial norms
      xnorm[(half * kTile + tok_in_tile) * 2] = ss;
      xnorm[(half * kTile + tok_in_tile) * 2 + 1] = mx;
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&qbar[0]);
      if (!tc::mbar_wait(&qbar[0], xphase, abort)) {
        if (lane == 0) route_timeout(p, abort, 15);
        break;
      }
      {
        const float oss = xnorm[((half ^ 1) * kTile + tok_in_tile) * 2];
        const float omx = xnorm[((half ^ 1) * kTile + tok_in_tile) * 2 + 1];
        if (SOFTMAX) {
          const float cm = fmaxf(mx, omx);
          // a warp without chunks contributes an empty sum at -inf
          ss = (mx == -INFINITY ? 0.f : ss * expf(mx - cm)) + (omx == -INFINITY ? 0.f : oss * expf(omx - cm));
          mx = cm;
        } else {
          ss = half == 0 ? ss + oss : oss + ss;           // the same order in both warps
        }
      }
      const float n = SOFTMAX ? mx + logf(ss) : sqrtf(ss);           // softmax keeps log sum exp(z) here
      // NormRouter: a zero logit vector scores zero.  Softmax: 1 / sum of exponentials.
      const float scale = SOFTMAX ? 1.f / ss : (ss > 0.f ? p.sigma_c / (n + p.eps) : 0.f);
      if (live && half == 0) p.znorm[t] = n;
      // pass 2: scores and their per-expert sums over the warp's 32 tokens.  The chunks are dealt the
      // other way round, so that with an odd number of chunks each warp takes the extra one once.
      for (int c = half ^ (n_chunks & 1); c < n_chunks; c += 2) {
        const int c0 = 32 * c;
        uint32_t rr[32];
        tc::tmem_ld_32x32(t_row + c0, rr);
        tc::tmem_ld_wait();
        float sv[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int e = c0 + i;
          const float z = __uint_as_float(rr[i]) + sbias[e < M ? e : 0];
          const float s = e < M ? scale * (SOFTMAX ? expf(z - mx) : fmaxf(z, 0.f)) : 0.f;
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
      // the accumulator has been read twice by this warp: the next tile may overwrite it
      tc::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        if (rank == 0) tc::mbar_arrive(&tmem_empty[acc]);
        else tc::mbar_arrive_leader(&tmem_empty[acc]);
      }
      // the second warp hands its top-k list to the first, which merges and writes the token's routing
      if (half == 1) {
#pragma unroll
        for (int j = 0; j < KMAX; ++j) { xtopv[tok_in_tile * KMAX + j] = tv[j]; xtopi[tok_in_tile * KMAX + j] = ti[j]; }
      }
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&qbar[1]);
      if (!tc::mbar_wait(&qbar[1], xphase, abort)) {
        if (lane == 0) route_timeout(p, abort, 16);
        break;
      }
      if (half == 0) {
#pragma unroll
        for (int j = 0; j < KMAX; ++j) {
          const float ov = xtopv[tok_in_tile * KMAX + j];
          const int oi = xtopi[tok_in_tile * KMAX + j];
          if (oi >= 0) topk_insert<KMAX>(tv, ti, ov, oi);
        }
        if (live) {
          for (int j = 0; j < p.k; ++j) {
            int e = -1;
            float key = 0.f;
#pragma unroll
            for (int q = 0; q < KMAX; ++q)
              if (q == j) { e = ti[q]; key = tv[q]; }
            p.idx[(int64_t)t * p.k + j] = e;
            // the gate is the score itself (a NaN logit was only re-keyed for the ordering)
            const float g = SOFTMAX ? scale * expf(key - mx) : scale * key;
            p.gate[(int64_t)t * p.k + j] = key == -FLT_MAX ? __int_as_float(0x7fc00000) : g;
            if (e >= 0) atomicAdd(&hist[e], 1);
          }
        }
      }
      // the first warp must be done with xtop before the second overwrites it for the next tile: the
      // next tile's first exchange (qbar[0]) orders that
    }
    if (lane == 0) tc::bulk_wait<0>();                   // the z tiles have left shared memory
    tc::tc_fence_before_sync();
    // the eight epilogue warps publish the CTA's statistics (named barrier 1: 256 threads)
    asm volatile("bar.sync 1, 256;" ::: "memory");
    // Counts are integers; a CTA's score sums are rounded to multiples of 2^-28 and added as 64-bit
    // integers too, so the totals do not depend on the order in which the CTAs arrive (|sum| < 2^35).
    const int et = threadIdx.x - 64;
    constexpr float kFix = 268435456.f;                   // 2^28
    for (int i = et; i < M; i += 32 * kEpiWarps) {
      float sum = 0.f;
#pragma unroll
      for (int w = 0; w < kEpiWarps; ++w) sum += wsum[w * M + i];
      if (hist[i] != 0) atomicAdd(&p.acc_counts[i], hist[i]);
      if (!(fabsf(sum) < 3.0e10f)) atomicOr(p.ticket + 1, 1u);          // NaN or out of range
      else if (sum != 0.f)
        atomicAdd(reinterpret_cast<unsigned long long*>(&p.acc_sums[i]), (unsigned long long)__float2ll_rn(sum * kFix));
    }
    __threadfence();
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (et == 0) *last_flag = atomicAdd(p.ticket, 1u) == gridDim.x - 1 ? 1 : 0;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (*last_flag) {                     // the CTA that arrives last publishes the totals and clears the accumulators
      __threadfence();
      const bool bad = __ldcg(p.ticket + 1) != 0u;
      for (int i = et; i < M; i += 32 * kEpiWarps) {
        p.counts_out[i] = __ldcg(&p.acc_counts[i]);
        const long long fixed = __ldcg(&p.acc_sums[i]);
        p.sum_out[i] = bad ? __int_as_float(0x7fc00000) : (float)((double)fixed * (1.0 / 268435456.0));
        p.acc_counts[i] = 0;
        p.acc_sums[i] = 0;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (et == 0) { p.ticket[0] = 0u; p.ticket[1] = 0u; }
    }
  }

  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync();                                        // neither CTA leaves while the other may still signal it
  if (warp == 1) {
    tc::tc_fence_after_sync();
    tc::tmem_dealloc_pair(tmem_base, 512);
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

// Workspace layout of the split router weights: the prepared layers [l][3][M][d] packed from the start
// (M = experts of the prepared routers), and one scratch set [3][M'][d] for a router that was not
// prepared, behind the space n_layers routers of the whole pool would take.
static __nv_bfloat16* scratch_terms(unipool_ctx* ctx) {
  return static_cast<__nv_bfloat16*>(ctx->ws.w_split) +
         (int64_t)ctx->cfg.n_layers * 3 * ctx->cfg.pool_size * ctx->cfg.d_model;
}

// Splits the fp32 router weights of n_layers layers ([n_layers][M][d], contiguous) into three bf16 terms
// per layer; flags[4 l + s] tells whether term s of layer l has a non-zero element.
static int router_split_launch(unipool_ctx* ctx, const float* W_r, int n_layers, int M, __nv_bfloat16* out,
                               int32_t* flags, cudaStream_t s) {
  const int64_t n = (int64_t)M * ctx->cfg.d_model;
  UP_CUDA(cudaMemsetAsync(flags, 0, (size_t)n_layers * 4 * sizeof(int32_t), s));
  const int64_t total = n * n_layers;
  const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
  router_split_kernel<<<blocks, 256, 0, s>>>(W_r, n, n_layers, out, flags);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

int router_prepare_launch(unipool_ctx* ctx, const float* W_r, int n_layers, int M, cudaStream_t s) {
  ctx->prepared_base = nullptr;
  if (n_layers == 0) return UNIPOOL_OK;
  PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_LOGITS, 1, s);
  const int rc = router_split_launch(ctx, W_r, n_layers, M, static_cast<__nv_bfloat16*>(ctx->ws.w_split),
                                     ctx->ws.split_any, s);
  if (rc != UNIPOOL_OK) return rc;
  ctx->prepared_base = W_r;
  ctx->prepared_layers = n_layers;
  ctx->prepared_experts = M;
  return UNIPOOL_OK;
}

// The bf16 terms of W_r and their flags: the prepared ones if W_r is a layer of the array last given to
// unipool_router_prepare, otherwise the scratch set, filled now.
static int router_terms(unipool_ctx* ctx, const float* W_r, int M, int phase, const __nv_bfloat16** terms,
                        const int32_t** flags, cudaStream_t s) {
  const int64_t n = (int64_t)M * ctx->cfg.d_model;
  if (ctx->prepared_base != nullptr && M == ctx->prepared_experts && W_r >= ctx->prepared_base) {
    const int64_t off = W_r - ctx->prepared_base;
    if (off % n == 0 && off / n < ctx->prepared_layers) {
      *terms = static_cast<const __nv_bfloat16*>(ctx->ws.w_split) + (off / n) * 3 * n;
      *flags = ctx->ws.split_any + 4 * (off / n);
      return UNIPOOL_OK;
    }
  }
  *terms = scratch_terms(ctx);
  *flags = ctx->ws.split_any + 4 * ctx->cfg.n_layers;
  PhaseTimer pt(ctx, phase, 1, s);
  return router_split_launch(ctx, W_r, 1, M, scratch_terms(ctx), ctx->ws.split_any + 4 * ctx->cfg.n_layers, s);
}

int route_tc_launch(unipool_ctx* ctx, const void* x, int T, const float* W_r, float sigma, const float* bias,
                    int M, int32_t* idx, float* gate, int32_t* counts, float* score_sum, float* znorm,
                    float* z_saved, cudaStream_t s) {
  const int d = ctx->cfg.d_model, k = ctx->cfg.top_k;
  int rc;
  const __nv_bfloat16* terms;
  const int32_t* flags;
  if ((rc = router_terms(ctx, W_r, M, UNIPOOL_PH_ROUTE_LOGITS, &terms, &flags, s)) != UNIPOOL_OK) return rc;
  RouteParams p{};
  p.bias = bias; p.T = T; p.M = M; p.d = d; p.k = k;
  p.sigma_c = sigma * ctx->cfg.c; p.eps = ctx->cfg.eps;
  p.idx = idx; p.gate = gate; p.znorm = znorm; p.z_saved = z_saved;
  p.counts_out = counts; p.sum_out = score_sum;
  p.acc_counts = ctx->ws.route_counts; p.acc_sums = reinterpret_cast<long long*>(ctx->ws.route_sums);
  p.ticket = ctx->ws.tickets + 2;                        // [2] CTAs done, [3] a non-finite score sum was seen
  p.split_any = flags;
  p.status = ctx->ws.status;
  const int n_cols = (M + 15) / 16 * 16;
  p.n1 = n_cols < 256 ? n_cols : 256;
  p.n2 = n_cols - p.n1;
  p.stage_bytes = kXBytes + (uint32_t)(n_cols / 2) * (kBK * 2);
  const uint32_t tail_bytes = 256 + 2 * kTile * 2 * 4 + 2 * kTile * UNIPOOL_MAX_TOPK * 4 + UNIPOOL_MAX_EXPERTS * 4 +
                              kEpiWarps * M * 4 + (M + 31) / 32 * 32 * 4;
  const uint32_t budget = 227 * 1024 - 1024 - tail_bytes - kEpiWarps * kZStage;
  p.stages = (int)(budget / p.stage_bytes);
  if (p.stages > kMaxStages) p.stages = kMaxStages;
  UP_REQUIRE(p.stages >= 2 && ctx->sm_count >= 2, UNIPOOL_ERR_UNSUPPORTED,
             "router of %d experts does not fit the logits kernel", M);
  CUtensorMap tmX, tmW1, tmW2, tmZ;
  if ((M & 3) == 0) {
    if ((rc = tc_f32_chunk_map(ctx, &tmZ, z_saved, M, T)) != UNIPOOL_OK) return rc;
  } else {
    tmZ = CUtensorMap{};                 // not used: rows of z are not 16-byte aligned, plain stores instead
  }
  if ((rc = tc_operand_map(ctx, &tmX, x, d, T, kTile)) != UNIPOOL_OK) return rc;
  if ((rc = tc_operand_map(ctx, &tmW1, terms, d, (uint64_t)3 * M, p.n1 / 2)) != UNIPOOL_OK) return rc;
  if (p.n2 > 0) {
    if ((rc = tc_operand_map(ctx, &tmW2, terms, d, (uint64_t)3 * M, p.n2 / 2)) != UNIPOOL_OK) return rc;
  } else {
    tmW2 = tmW1;
  }
  PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_SELECT, 1, s);
  const size_t smem = (size_t)p.stages * p.stage_bytes + kEpiWarps * kZStage + tail_bytes + 1024;
  const int n_tp = (T + 2 * kTile - 1) / (2 * kTile);
  const int max_pairs = ctx->sm_count / 2;
  const int grid = 2 * (n_tp < max_pairs ? n_tp : max_pairs);
  const bool softmax = ctx->cfg.router_mode == UNIPOOL_ROUTER_SOFTMAX;
  auto kern = k <= 2 ? (softmax ? route_tc_kernel<2, true> : route_tc_kernel<2, false>)
                     : (softmax ? route_tc_kernel<UNIPOOL_MAX_TOPK, true> : route_tc_kernel<UNIPOOL_MAX_TOPK, false>);
  UP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<grid, kThreads, smem, s>>>(tmX, tmW1, tmW2, tmZ, p);
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
  const __nv_bfloat16* terms;                                  // term 0 = bf16(W_r)
  const int32_t* flags;
  if ((rc = router_terms(ctx, W_r, M, UNIPOOL_PH_ROUTE_BWD_DZ, &terms, &flags, s)) != UNIPOOL_OK) return rc;
  {
    PhaseTimer pt(ctx, UNIPOOL_PH_ROUTE_BWD_DZ, 1, s);
    const int64_t threads = (int64_t)T * 4;
    const bool softmax = ctx->cfg.router_mode == UNIPOOL_ROUTER_SOFTMAX;
    auto kern = k <= 2 ? (softmax ? router_dz16_kernel<true, 2> : router_dz16_kernel<false, 2>)
                       : (softmax ? router_dz16_kernel<true, UNIPOOL_MAX_TOPK> : router_dz16_kernel<false, UNIPOOL_MAX_TOPK>);
    kern<<<(int)((threads + 255) / 256), 256, 0, s>>>(
        z_saved, znorm, idx, dgate, coef, T, M, Mp, k, sigma, ctx->cfg.c, ctx->cfg.eps, dz16, dsigma,
        ctx->ws.dsigma_acc, ctx->ws.tickets + 1);
    UP_LAUNCH_CHECK();
  }
  return router_bwd_gemms_tc(ctx, dz16, Mp, terms, x, T, M, dx, dW_r, s);
}

}  // namespace unipool
