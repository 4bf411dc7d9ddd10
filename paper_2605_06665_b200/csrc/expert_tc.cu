// Grouped SwiGLU expert GEMMs on the 5th-generation tensor cores (tcgen05) for
// bf16 storage with fp32 accumulation: forward (Eq. 2's e_i), dgrad and wgrad.
//
// Persistent, warp-specialised kernels, one CTA per SM:
//   warp 0      TMA producer   (one lane issues cp.async.bulk.tensor loads)
//   warp 1      MMA issuer     (one lane issues tcgen05.mma; owns the TMEM allocation)
//   warps 2-5   epilogue       (tcgen05.ld from TMEM, fused element-wise math, results staged in
//                               shared memory and written by TMA stores / add-reduces)
// Operand tiles are staged in shared memory with the 128-byte swizzle, accumulators
// are double-buffered in TMEM so the epilogue of one tile overlaps the main loop of
// the next.  The tile schedule is read from device memory (group offsets), so no call
// synchronises the host.  Every mbarrier wait is bounded: on expiry the kernel records
// UNIPOOL_ERR_TIMEOUT in the status word, all roles leave, TMEM is released.
//   grouped_gemm_tc_kernel<MODE>  one CTA per 128 x 256 tile (cta_group::1), all six GEMMs
//   wgrad_pair_kernel             the weight gradient on CTA pairs (cta_group::2, M = 256)
//   row_pair_kernel<MODE>         the four row-tile GEMMs on CTA pairs (M = 256, and M = 128 for a
//                                 group's odd last tile)
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace unipool {

namespace {

constexpr int BM = 128;          // rows of an output tile (TMEM lanes)
constexpr int BN = 256;          // columns of an output tile (one tcgen05.mma of N = 256)
constexpr int BK = 64;           // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int kThreads = 192;           // producer warp, MMA warp, four epilogue warps
constexpr int kThreadsIo = 448;         // dgrad1: eight epilogue warps plus four warps that move their operands
constexpr int kEpiWarps = 4;
constexpr uint32_t kABytes = BM * BK * 2;
constexpr uint32_t kBBytes = BN * BK * 2;
constexpr uint32_t kStageBytes = kABytes + kBBytes;
constexpr uint32_t kMnBlockBytes = 64 * BK * 2;   // one 64(MN) x 64(K) box
constexpr uint32_t kBarOffset = 229376;           // operand stages + epilogue staging fill this much
constexpr uint32_t kTableBytes = (UNIPOOL_MAX_EXPERTS + 8) * sizeof(uint16_t);   // one 16-bit count per expert
constexpr uint32_t kSmemTotal = kBarOffset + 512 + kTableBytes + 1024;   // + barriers + table + alignment slack
static_assert(kSmemTotal <= 227 * 1024, "shared-memory budget");
constexpr int kChunk = 32;       // output columns one epilogue step moves (a 32 x 32 box per warp)
constexpr uint32_t kBf16ChunkBytes = 32 * kChunk * 2;      // 2 KiB, 64-byte rows, 64-byte swizzle
constexpr uint32_t kF32ChunkBytes = 32 * kChunk * 4;       // 4 KiB, 128-byte rows, 128-byte swizzle

enum Mode : int {
  kFwd1 = 0,    // GU = Xp W_gu^T, A = silu(G)*U        A K-major, B K-major (3-D map), row tiles
  kFwd2 = 1,    // Yp = A W_down^T                      A K-major, B K-major,           row tiles
  kDgrad1 = 2,  // dGU = swiglu'(dYp W_down, GU)        A K-major, B MN-major,          row tiles
  kDgrad2 = 3,  // dXp = dGU W_gu                       A K-major, B MN-major,          row tiles
  kWgrad = 4,   // dW[e] (+)= P_e^T Q_e                 A MN-major, B MN-major,         ragged K
};

struct GemmParams {
  const int32_t* offsets;       // row tiles: &offsets[n_experts]; wgrad: [n_layers][n_experts+1]
  const int32_t* tile_expert;   // row tiles only
  const int32_t* group_offsets; // row tiles on CTA pairs: [n_experts + 1] starts of the groups
  int n_experts, expert_base;
  int n_layers;                 // wgrad
  int layer_stride_rows;        // wgrad
  int Mdim, Ndim, Kdim;         // wgrad: dW is [Mdim, Ndim]; row tiles: output columns, contraction
  int f;                        // expert width (fwd1 / dgrad1 addressing)
  int overwrite;                // 1 = the output is written, 0 = it is added to (wgrad, dgrad2)
  int uniform_rows;             // wgrad without offsets: group e = rows [e*Kdim, (e+1)*Kdim) of this many
  int32_t* status;
};

// Shared memory: kStages operand stages, then one staging region per epilogue warp.
// The SwiGLU-derivative epilogue also reads G and U, so it trades one operand stage
// for a ring of five (G, U) chunk buffers per warp that are fetched three chunks ahead.
template <int MODE> struct Traits {
  static constexpr int kThreads = MODE == 2 ? kThreadsIo : unipool::kThreads;
  static constexpr int kStages = MODE == 2 ? 3 : 4;
  static constexpr uint32_t kStagingOffset = kStages * kStageBytes;
  static constexpr uint32_t kStagingPerWarp = MODE == 2 ? 20480 : 8192;
  static_assert(kStagingOffset + kEpiWarps * kStagingPerWarp == kBarOffset, "shared-memory budget");
  static constexpr bool kAMn = MODE == kWgrad;
  static constexpr bool kBMn = MODE == kDgrad1 || MODE == kDgrad2 || MODE == kWgrad;
  static constexpr bool kRowTiles = MODE != kWgrad;
};

struct TileCoord { int e, mt, nt, kblocks; bool valid; int col0, ncols; };   // output columns [col0, col0 + ncols)

template <int MODE>
__device__ __forceinline__ int tiles_total(const GemmParams& p, int& n_nt, int& n_mt) {
  if constexpr (Traits<MODE>::kRowTiles) {
    n_mt = p.offsets ? *p.offsets / BM : p.Mdim;     // no offsets: one group of Mdim row tiles
    const int ncols = MODE == kFwd1 ? BN / 2 : BN;
    n_nt = (p.Ndim + ncols - 1) / ncols;
    return n_mt * n_nt;
  } else {
    n_mt = (p.Mdim + BM - 1) / BM;
    n_nt = (p.Ndim + BN - 1) / BN;
    return p.n_experts * n_mt * n_nt;
  }
}

template <int MODE>
__device__ __forceinline__ TileCoord tile_coord(const GemmParams& p, int tile, int n_nt, int n_mt) {
  TileCoord c;
  if constexpr (Traits<MODE>::kRowTiles) {
    // A kernel that consumes what the previous launch produced in ascending row order (the down
    // projection reads A, the second dgrad reads dGU) walks the rows downwards: the rows written
    // last are the ones still in L2.
    constexpr bool kDescending = MODE == kFwd2 || MODE == kDgrad2;
    c.mt = kDescending ? n_mt - 1 - tile / n_nt : tile / n_nt;
    c.nt = tile % n_nt;
    c.e = p.tile_expert ? p.tile_expert[c.mt] : 0;
    c.kblocks = p.Kdim / BK;
    c.valid = c.e >= 0 && c.e < p.n_experts;
    c.col0 = c.nt * BN;
    c.ncols = BN;
  } else {
    const int per_e = n_mt * n_nt;
    c.e = tile / per_e;
    const int rem = tile % per_e;
    c.mt = rem / n_nt;
    c.nt = rem % n_nt;
    int kb = 0;
    if (p.offsets == nullptr) {
      const int left = p.uniform_rows - c.e * p.Kdim;
      kb = (left < p.Kdim ? left : p.Kdim) / BK;
    } else {
      for (int l = 0; l < p.n_layers; ++l) {
        const int32_t* off = p.offsets + (int64_t)l * (p.n_experts + 1);
        kb += (off[c.e + 1] - off[c.e]) / BK;
      }
    }
    c.kblocks = kb;
    c.valid = kb > 0;
    c.col0 = c.nt * BN;
    c.ncols = BN;
  }
  return c;
}

// The tiles of a launch are dealt round-robin to the CTAs; the last, partial round would keep a few
// CTAs busy for a whole tile while the rest wait.  For the plain row-tile GEMMs (down projection,
// second dgrad) the tiles of that round are cut into 2 or 4 column slices (MMA N = 128 or 64) so that
// they spread over (nearly) all CTAs.  Work units: [0, full) whole tiles, then slices.
struct TailSplit { int full, slices, units; };
template <int MODE>
__device__ __forceinline__ TailSplit tail_split(const GemmParams& p, int total) {
  TailSplit t{total, 1, total};
  if constexpr (MODE == kFwd2 || MODE == kDgrad2) {
    const int grid = (int)gridDim.x;
    const int rest = total % grid;
    if (rest > 0 && 2 * rest <= grid) {
      t.full = total - rest;
      t.slices = 4 * rest <= grid ? 4 : 2;
      t.units = t.full + rest * t.slices;
    }
  }
  return t;
}
template <int MODE>
__device__ __forceinline__ TileCoord unit_coord(const GemmParams& p, const TailSplit& ts, int unit, int n_nt, int n_mt) {
  if (unit < ts.full) return tile_coord<MODE>(p, unit, n_nt, n_mt);
  const int u = unit - ts.full;
  TileCoord c = tile_coord<MODE>(p, ts.full + u / ts.slices, n_nt, n_mt);
  c.ncols = BN / ts.slices;
  c.col0 += (u % ts.slices) * c.ncols;
  return c;
}

__device__ __forceinline__ void report_timeout(const GemmParams& p, volatile int* abort, int site) {
  *abort = 1;
  if (atomicCAS(p.status, 0, kStatusTimeout) == 0) {
    p.status[1] = site;
    p.status[2] = (int)blockIdx.x;
  }
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// logistic function through one special-function op: sig(a) = 0.5 + 0.5 tanh(a/2)
__device__ __forceinline__ float sigmoid_fast(float a) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * a));
  return fmaf(0.5f, t, 0.5f);
}

// Staging tiles are 32 rows (one per lane) of kChunk columns in the layout the TMA
// swizzle modes expect, so that a warp's 16-byte accesses never collide on a bank:
//   bf16: 64-byte rows, 16-byte piece q of row r sits at piece q ^ ((r >> 1) & 3)
//   fp32: 128-byte rows, piece q of row r sits at piece q ^ (r & 7)
__device__ __forceinline__ uint4* bf16_piece(uint8_t* tile, int r, int q) {
  return reinterpret_cast<uint4*>(tile + r * 64 + ((q ^ ((r >> 1) & 3)) << 4));
}
__device__ __forceinline__ uint4* f32_piece(uint8_t* tile, int r, int q) {
  return reinterpret_cast<uint4*>(tile + r * 128 + ((q ^ (r & 7)) << 4));
}
__device__ __forceinline__ void stage_row_bf16(uint8_t* tile, int r, const float (&v)[32]) {
#pragma unroll
  for (int q = 0; q < 4; ++q)
    *bf16_piece(tile, r, q) =
        make_uint4(pack_bf16(v[8 * q + 0], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                   pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
}
__device__ __forceinline__ void unstage_row_bf16(uint8_t* tile, int r, float (&v)[32]) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint4 w = *bf16_piece(tile, r, q);
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[8 * q + 2 * i] = __uint_as_float(ww[i] << 16);
      v[8 * q + 2 * i + 1] = __uint_as_float(ww[i] & 0xffff0000u);
    }
  }
}

// dgrad1: the (G, U) chunks of one epilogue warp's rows, over all tiles of this CTA, in the
// order the epilogue consumes them.  Chunk number n of the stream uses ring slot n % kRing.
constexpr int kRing = 5, kAhead = 3;                   // ring slots per warp, prefetch distance
template <int MODE>
struct ChunkCursor {
  int tile, ch, nch, nt, row0;
  __device__ void seek(const GemmParams& p, int total, int n_nt, int n_mt, int quarter) {
    while (tile < total) {                              // next tile that has chunks
      const TileCoord c = tile_coord<MODE>(p, tile, n_nt, n_mt);
      if (c.valid) {
        nt = c.nt;
        row0 = c.mt * BM + quarter * 32;
        nch = min(BN / kChunk, (p.f - c.nt * BN) / kChunk);
        ch = 0;
        if (nch > 0) return;
      }
      tile += gridDim.x;
    }
  }
  __device__ void start(const GemmParams& p, int total, int n_nt, int n_mt, int quarter) {
    tile = blockIdx.x; ch = 0; nch = 0; nt = 0; row0 = 0;
    seek(p, total, n_nt, n_mt, quarter);
  }
  __device__ void next(const GemmParams& p, int total, int n_nt, int n_mt, int quarter) {
    if (++ch == nch) { tile += gridDim.x; seek(p, total, n_nt, n_mt, quarter); }
  }
  __device__ int col() const { return nt * BN + ch * kChunk; }
};

// Epilogue of the gate/up projection for one warp's 32 rows: G and U leave TMEM, A = silu(G) * U is
// formed, and the three bf16 chunks are staged and stored (GU through tmC0, A through tmC1).
// t_g / t_u: TMEM addresses of this warp's lanes at the first G and the first U column; the chunks are
// nch steps of 32 features from feat0.  Warps that share a TMEM lane quarter split the chunks: this
// warp takes ch0, ch0 + step, ...
__device__ __forceinline__ void epilogue_swiglu(const CUtensorMap* tmC0, const CUtensorMap* tmC1, const GemmParams& p,
                                                uint32_t t_g, uint32_t t_u, int feat0, int nch, int row0, uint8_t* stg,
                                                int lane, int ch0 = 0, int step = 1) {
#pragma unroll 1
  for (int ch = ch0; ch < nch; ch += step) {
    const int feat = feat0 + ch * kChunk;
    if (feat >= p.f) break;
    uint32_t rg[32], ru[32];
    tc::tmem_ld_32x32(t_g + ch * kChunk, rg);
    tc::tmem_ld_32x32(t_u + ch * kChunk, ru);
    tc::tmem_ld_wait();
    float g[32], u[32], a[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      g[i] = __uint_as_float(rg[i]);
      u[i] = __uint_as_float(ru[i]);
      a[i] = g[i] * sigmoid_fast(g[i]) * u[i];
    }
    // lanes 0, 1, 2 each own one of the three stores (G, U, A), so the stores are issued and
    // their shared-memory reads awaited side by side
    if (lane < 3) tc::bulk_wait_read<0>();       // the previous chunk's stores have drained the tiles
    __syncwarp();
    stage_row_bf16(stg, lane, g);
    stage_row_bf16(stg + kBf16ChunkBytes, lane, u);
    stage_row_bf16(stg + 2 * kBf16ChunkBytes, lane, a);
    tc::fence_proxy_async();
    __syncwarp();
    if (lane == 0) tc::tma_store_2d(tmC0, stg, feat, row0);
    else if (lane == 1) tc::tma_store_2d(tmC0, stg + kBf16ChunkBytes, p.f + feat, row0);
    else if (lane == 2) tc::tma_store_2d(tmC1, stg + 2 * kBf16ChunkBytes, feat, row0);
    if (lane < 3) tc::bulk_commit();
  }
}

// Epilogue of a plain row-tile GEMM (down projection, second dgrad) for one warp's 32 rows: the
// accumulator is rounded to bf16, staged in a ring of four chunk tiles and stored (or add-reduced).
template <int MODE>
__device__ __forceinline__ void epilogue_rows(const CUtensorMap* tmC0, const GemmParams& p, uint32_t t_row, int col0,
                                              int ncols, int row0, uint8_t* stg, int lane, int& gchunk, int ch0 = 0,
                                              int step = 1) {
#pragma unroll 1
  for (int ch = ch0; ch < ncols / kChunk; ch += step) {
    const int col = col0 + ch * kChunk;
    if (col >= p.Ndim) break;
    uint32_t rr[32];
    tc::tmem_ld_32x32(t_row + ch * kChunk, rr);
    tc::tmem_ld_wait();
    float v[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(rr[i]);
    uint8_t* buf = stg + (gchunk++ & 3) * kBf16ChunkBytes;
    if (lane == 0) tc::bulk_wait_read<3>();      // the store issued four chunks ago has drained `buf`
    __syncwarp();
    stage_row_bf16(buf, lane, v);
    tc::fence_proxy_async();
    __syncwarp();
    if (lane == 0) {
      if (MODE == kFwd2 || p.overwrite) tc::tma_store_2d(tmC0, buf, col, row0);
      else tc::tma_reduce_add_2d(tmC0, buf, col, row0);
      tc::bulk_commit();
    }
  }
}

template <int MODE>
__global__ void __launch_bounds__(Traits<MODE>::kThreads, 1)
grouped_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const __grid_constant__ CUtensorMap tmB64,   // dgrad: 64 x 64 boxes of the weights (column slices)
                       const __grid_constant__ CUtensorMap tmC0, const __grid_constant__ CUtensorMap tmC1,
                       const GemmParams p) {
  using TR = Traits<MODE>;
  constexpr int kStages = TR::kStages;
  constexpr uint32_t kTmemCols = 2 * BN;            // two accumulators of BN fp32 columns

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kBarOffset);
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* tmem_full = empty_bar + kStages;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* epi_bar = tmem_empty + 2;               // [kEpiWarps][5] operand loads of the epilogue have landed
  uint64_t* staged_bar = epi_bar + 5 * kEpiWarps;   // [kEpiWarps][5] results are staged, ready to store
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(staged_bar + 5 * kEpiWarps);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_ptr + 1);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { tc::mbar_init(&full_bar[s], 1); tc::mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { tc::mbar_init(&tmem_full[a], 1); tc::mbar_init(&tmem_empty[a], MODE == kDgrad1 ? 2 * kEpiWarps : kEpiWarps); }
    for (int i = 0; i < 5 * kEpiWarps; ++i) { tc::mbar_init(&epi_bar[i], 1); tc::mbar_init(&staged_bar[i], 1); }
    *abort = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmA);
    tc::tma_prefetch_desc(&tmB);
    tc::tma_prefetch_desc(&tmC0);
    if constexpr (MODE == kFwd1 || MODE == kDgrad1 || MODE == kFwd2) tc::tma_prefetch_desc(&tmC1);
  }
  if (warp == 1) {
    tc::tmem_alloc(tmem_ptr, kTmemCols);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;

  int n_nt, n_mt;
  const int n_tiles = tiles_total<MODE>(p, n_nt, n_mt);
  const TailSplit ts = tail_split<MODE>(p, n_tiles);
  const int total = ts.units;                        // work units: whole tiles, then slices of the last round

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
        const TileCoord c = unit_coord<MODE>(p, ts, tile, n_nt, n_mt);
        if (!c.valid) continue;
        const int pe = p.expert_base + c.e;
        int layer = 0, r = 0, r_end = 0;              // wgrad: walks the rows of expert e, layer by layer
        if constexpr (!TR::kRowTiles) {
          if (p.offsets == nullptr) {
            r = c.e * p.Kdim;
            r_end = r + c.kblocks * BK;
          } else {
            r = p.offsets[c.e];
            r_end = p.offsets[c.e + 1];
          }
        }
        for (int kb = 0; kb < c.kblocks; ++kb) {
          if (!tc::mbar_wait(&empty_bar[stage], phase ^ 1u, abort)) { report_timeout(p, abort, 1); ok = false; break; }
          uint8_t* sA = smem + stage * kStageBytes;
          uint8_t* sB = sA + kABytes;
          tc::mbar_expect_tx(&full_bar[stage], kABytes + (uint32_t)c.ncols * (BK * 2));
          if constexpr (MODE == kFwd1) {
            tc::tma_load_2d(sA, &tmA, &full_bar[stage], kb * BK, c.mt * BM);
            tc::tma_load_3d(sB, &tmB, &full_bar[stage], kb * BK, c.nt * (BN / 2), 2 * pe);
          } else if constexpr (MODE == kFwd2) {
            tc::tma_load_2d(sA, &tmA, &full_bar[stage], kb * BK, c.mt * BM);
            if (c.ncols == BN) {
              tc::tma_load_2d(sB, &tmB, &full_bar[stage], kb * BK, pe * p.Ndim + c.col0);
            } else {                                  // a column slice: 64-row boxes of the weight (tmC1)
              for (int i = 0; i < c.ncols / 64; ++i)
                tc::tma_load_2d(sB + i * kMnBlockBytes, &tmC1, &full_bar[stage], kb * BK, pe * p.Ndim + c.col0 + 64 * i);
            }
          } else if constexpr (MODE == kDgrad1 || MODE == kDgrad2) {
            tc::tma_load_2d(sA, &tmA, &full_bar[stage], kb * BK, c.mt * BM);
            if (c.ncols == BN) {                      // the four 64-column blocks of the weights in one box
              tc::tma_load_3d(sB, &tmB, &full_bar[stage], 0, pe * p.Kdim + kb * BK, c.col0 / 64);
            } else {
              for (int i = 0; i < c.ncols / 64; ++i)
                tc::tma_load_2d(sB + i * kMnBlockBytes, &tmB64, &full_bar[stage], c.col0 + 64 * i,
                                pe * p.Kdim + kb * BK);
            }
          } else {
            while (r >= r_end) {                        // next layer that has rows for this expert
              ++layer;
              const int32_t* off = p.offsets + (int64_t)layer * (p.n_experts + 1);
              r = off[c.e];
              r_end = off[c.e + 1];
            }
            const int grow = layer * p.layer_stride_rows + r;
            tc::tma_load_3d(sA, &tmA, &full_bar[stage], 0, grow, c.mt * (BM / 64));   // two 64-column blocks
            tc::tma_load_3d(sB, &tmB, &full_bar[stage], 0, grow, c.nt * (BN / 64));   // four
            r += BK;
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // give loads already in flight time to land before the CTA retires
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t a_lbo = TR::kAMn ? kMnBlockBytes : 16, b_lbo = TR::kBMn ? kMnBlockBytes : 16;
      constexpr uint32_t a_step = (TR::kAMn ? 16 * 128 : 32) >> 4;   // descriptor units of 16 bytes per K = 16
      constexpr uint32_t b_step = (TR::kBMn ? 16 * 128 : 32) >> 4;
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
        const TileCoord c = unit_coord<MODE>(p, ts, tile, n_nt, n_mt);
        if (!c.valid) continue;
        const int acc = local & 1;
        const uint32_t acc_phase = (local >> 1) & 1;
        ++local;
        if (!tc::mbar_wait(&tmem_empty[acc], acc_phase ^ 1u, abort)) { report_timeout(p, abort, 2); break; }
        tc::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        const uint32_t idesc = tc::instr_desc_bf16(c.ncols, TR::kAMn, TR::kBMn);
        for (int kb = 0; kb < c.kblocks; ++kb) {
          if (!tc::mbar_wait(&full_bar[stage], phase, abort)) { report_timeout(p, abort, 3); ok = false; break; }
          tc::tc_fence_after_sync();
          const uint32_t aaddr = tc::smem_u32(smem + stage * kStageBytes);
          const uint64_t adesc = tc::smem_desc_sw128(aaddr, a_lbo, 1024);
          const uint64_t bdesc = tc::smem_desc_sw128(aaddr + kABytes, b_lbo, 1024);
#pragma unroll
          for (int j = 0; j < BK / 16; ++j)
            tc::umma_bf16(d_tmem, adesc + j * a_step, bdesc + j * b_step, idesc, (kb | j) != 0 ? 1u : 0u);
          tc::umma_commit(&empty_bar[stage]);            // frees the stage once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc::umma_commit(&tmem_full[acc]);        // accumulator complete
      }
    }
  } else if (MODE == kDgrad1 && warp >= 2 + 2 * kEpiWarps) {
    // ------------------------------------------------------------ dgrad1: operand mover of epilogue warp (warp - 4)
    // One lane per warp.  It keeps G and U of its epilogue warp's rows kAhead chunks ahead (TMA loads
    // into the ring) and writes each chunk back once the epilogue warp has turned it into dG, dU in
    // place (TMA stores), so that the epilogue warp itself never issues or awaits a copy.
    if constexpr (MODE == kDgrad1) {
      if (lane == 0) {
        const int ew = warp - (2 + 2 * kEpiWarps);
        const int quarter = (ew + 2) & 3;
        uint8_t* stg = smem + TR::kStagingOffset + ew * TR::kStagingPerWarp;
        uint64_t* full = epi_bar + kRing * ew;
        uint64_t* staged = staged_bar + kRing * ew;
        ChunkCursor<MODE> ld, st;
        ld.start(p, total, n_nt, n_mt, quarter);
        st.start(p, total, n_nt, n_mt, quarter);
        int fetched = 0, stored = 0;
        bool ok = true;
        while (st.tile < total && ok) {
          // A slot is refilled only after the store that last read it has drained: when chunk
          // `fetched` <= stored + 2 is fetched, that store (chunk fetched - 5) is at least three
          // bulk groups old, hence wait_group.read 1.
          while (fetched < stored + kAhead && ld.tile < total) {
            const int slot = fetched % kRing;
            uint8_t* buf = stg + slot * 2 * kBf16ChunkBytes;
            tc::bulk_wait_read<1>();
            tc::mbar_expect_tx(&full[slot], 2 * kBf16ChunkBytes);
            tc::tma_load_2d(buf, &tmC1, &full[slot], ld.col(), ld.row0);
            tc::tma_load_2d(buf + kBf16ChunkBytes, &tmC1, &full[slot], p.f + ld.col(), ld.row0);
            ++fetched;
            ld.next(p, total, n_nt, n_mt, quarter);
          }
          const int slot = stored % kRing;
          uint8_t* buf = stg + slot * 2 * kBf16ChunkBytes;
          if (!tc::mbar_wait(&staged[slot], (stored / kRing) & 1, abort)) { report_timeout(p, abort, 6); ok = false; break; }
          tc::tma_store_2d(&tmC0, buf, st.col(), st.row0);
          tc::tma_store_2d(&tmC0, buf + kBf16ChunkBytes, p.f + st.col(), st.row0);
          tc::bulk_commit();
          ++stored;
          st.next(p, total, n_nt, n_mt, quarter);
        }
        if (!ok)
          for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let loads already in flight land
        tc::bulk_wait<0>();
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    // Warp w owns TMEM lanes [32*(w%4), +32) = 32 rows of the tile.  Results are rounded,
    // staged in this warp's shared-memory tiles and leave through TMA stores; nothing
    // here synchronises with another warp except the two TMEM barriers.
    // (dgrad1 has two epilogue warps per 32 lanes: they share one ring and take alternate chunks)
    const int quarter = warp & 3;
    const int ew = (warp - 2) & 3;
    const int half = (warp - 2) >> 2;
    (void)half;
    uint8_t* stg = smem + TR::kStagingOffset + ew * TR::kStagingPerWarp;
    uint64_t* my_bar = epi_bar + kRing * ew;           // dgrad1: chunk n of this warp's stream is in slot n % kRing
    uint64_t* my_staged = staged_bar + kRing * ew;
    int gchunk = 0;                                    // chunks this warp has staged so far (ring position)
    (void)my_bar; (void)my_staged;
    int local = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
      const TileCoord c = unit_coord<MODE>(p, ts, tile, n_nt, n_mt);
      if (!c.valid) {
        if constexpr (MODE == kWgrad) {
          if (p.overwrite) {                           // no rows anywhere: the gradient of this tile is zero
            const int m0 = c.mt * BM + quarter * 32;
            if (m0 < p.Mdim) {
              if (lane == 0) tc::bulk_wait_read<0>();
              __syncwarp();
#pragma unroll
              for (int q = 0; q < 8; ++q) *f32_piece(stg, lane, q) = make_uint4(0, 0, 0, 0);
              tc::fence_proxy_async();
              __syncwarp();
              if (lane == 0) {
                for (int ch = 0; ch < BN / kChunk; ++ch) {
                  const int col = c.nt * BN + ch * kChunk;
                  if (col < p.Ndim) tc::tma_store_2d(&tmC0, stg, col, (p.expert_base + c.e) * p.Mdim + m0);
                }
                tc::bulk_commit();
                tc::bulk_wait_read<0>();
              }
              __syncwarp();
            }
          }
        }
        continue;
      }
      const int acc = local & 1;
      const uint32_t acc_phase = (local >> 1) & 1;
      ++local;
      const int row0 = c.mt * BM + quarter * 32;       // first row of this warp (row tiles: permuted row)

      int nch = 0;
      if constexpr (MODE == kDgrad1) nch = min(BN / kChunk, (p.f - c.nt * BN) / kChunk);
      if (!tc::mbar_wait(&tmem_full[acc], acc_phase, abort)) {
        if (lane == 0) report_timeout(p, abort, 4);
        break;
      }
      tc::tc_fence_after_sync();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * BN;

      if constexpr (MODE == kFwd1) {
        epilogue_swiglu(&tmC0, &tmC1, p, t_row, t_row + BN / 2, c.nt * (BN / 2), BN / 2 / kChunk, row0, stg, lane);
      } else if constexpr (MODE == kFwd2 || MODE == kDgrad2) {
        epilogue_rows<MODE>(&tmC0, p, t_row, c.col0, c.ncols, row0, stg, lane, gchunk);
      } else if constexpr (MODE == kDgrad1) {
#pragma unroll 1
        for (int ch = 0; ch < nch; ++ch) {
          if (((gchunk + ch) & 1) != half) continue;    // the other warp of this quarter takes it
          const int slot = (gchunk + ch) % kRing;
          const uint32_t slot_phase = ((gchunk + ch) / kRing) & 1;
          uint8_t* buf = stg + slot * 2 * kBf16ChunkBytes;
          uint32_t rr[32];
          tc::tmem_ld_32x32(t_row + ch * kChunk, rr);
          tc::tmem_ld_wait();
          if (!tc::mbar_wait(&my_bar[slot], slot_phase, abort)) {
            if (lane == 0) report_timeout(p, abort, 5);
            ok = false;
            break;
          }
          float g[32], u[32], dg[32], du[32];
          unstage_row_bf16(buf, lane, g);
          unstage_row_bf16(buf + kBf16ChunkBytes, lane, u);
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float dA = __uint_as_float(rr[i]);
            const float sig = sigmoid_fast(g[i]);
            const float sl = g[i] * sig;
            dg[i] = dA * u[i] * (sig + sl * (1.0f - sig));   // silu'(g) = sig (1 + g (1 - sig))
            du[i] = dA * sl;
          }
          stage_row_bf16(buf, lane, dg);               // in place: each lane rewrites the row it read
          stage_row_bf16(buf + kBf16ChunkBytes, lane, du);
          tc::fence_proxy_async();
          __syncwarp();
          if (lane == 0) tc::mbar_arrive(&my_staged[slot]);   // the operand mover stores the chunk
        }
        gchunk += nch;
        if (!ok) break;
      } else {
        const int m0 = row0;                           // row of dW[e]
        if (m0 < p.Mdim) {
          const int grow = (p.offsets ? (p.expert_base + c.e) * p.Mdim : 0) + m0;
#pragma unroll 1
          for (int ch = 0; ch < BN / kChunk; ++ch) {
            const int col = c.nt * BN + ch * kChunk;
            if (col >= p.Ndim) break;
            uint32_t rr[32];
            tc::tmem_ld_32x32(t_row + ch * kChunk, rr);
            tc::tmem_ld_wait();
            uint8_t* buf = stg + (gchunk++ & 1) * kF32ChunkBytes;
            if (lane == 0) tc::bulk_wait_read<1>();    // the store issued two chunks ago has drained `buf`
            __syncwarp();
#pragma unroll
            for (int q = 0; q < 8; ++q)
              *f32_piece(buf, lane, q) = make_uint4(rr[4 * q + 0], rr[4 * q + 1], rr[4 * q + 2], rr[4 * q + 3]);
            tc::fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              if (p.overwrite) tc::tma_store_2d(&tmC0, buf, col, grow);
              else tc::tma_reduce_add_2d(&tmC0, buf, col, grow);
              tc::bulk_commit();
            }
          }
        }
      }
      tc::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&tmem_empty[acc]);
    }
    if (!ok && lane == 0)
      for (int i = 0; i < 200; ++i) __nanosleep(1000);  // let loads already in flight land before the CTA retires
    if (lane < 3) tc::bulk_wait<0>();                  // every store has left shared memory and is complete
    __syncwarp();
  }

  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc::tc_fence_after_sync();
    tc::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------- weight gradient on CTA pairs
// dW[e] (+)= P_e^T Q_e with one tcgen05.mma.cta_group::2 of M = 256, N = 256 per K = 16: the two CTAs
// of a cluster own rows [0,128) and [128,256) of the 256 x 256 output tile (their own TMEM), each
// loads its 128 columns of P (A operand) and HALF of the 256 columns of Q (B operand), so a CTA
// moves 32 KB per k-block for the work that took 48 KB, and six stages fit instead of four.  The
// even CTA issues the MMAs; every TMA load counts its bytes on the even CTA's mbarrier (plain
// loads, no multicast); tcgen05.commit arrives on the stage / accumulator barriers of both CTAs.
constexpr int kPairStages = 6;
constexpr uint32_t kPairSmemTotal = kSmemTotal;
constexpr uint32_t kPairHalfBytes = 128 * BK * 2;            // 128 (M or N) x 64 (K) bf16
constexpr uint32_t kPairStageBytes = 2 * kPairHalfBytes;
static_assert(kPairStages * kPairStageBytes + kEpiWarps * 8192 == kBarOffset, "shared-memory budget");

__device__ __forceinline__ int wgrad_kblocks(const GemmParams& p, int e) {
  int kb = 0;
  for (int l = 0; l < p.n_layers; ++l) {
    const int32_t* off = p.offsets + (int64_t)l * (p.n_experts + 1);
    kb += (off[e + 1] - off[e]) / BK;
  }
  return kb;
}

// Tile of `pair` in `round` when a sorted tile list is dealt out forwards and backwards alternately.
__device__ __forceinline__ int snake_tile(int round, int pair, int n_pairs) {
  return round * n_pairs + ((round & 1) ? n_pairs - 1 - pair : pair);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
wgrad_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmC0, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kBarOffset);
  uint64_t* empty_bar = full_bar + kPairStages;
  uint64_t* tmem_full = empty_bar + kPairStages;
  uint64_t* tmem_empty = tmem_full + 2;
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(tmem_empty + 2);
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_ptr + 1);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int rank = (int)tc::cluster_ctarank();               // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPairStages; ++s) { tc::mbar_init(&full_bar[s], 1); tc::mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { tc::mbar_init(&tmem_full[a], 1); tc::mbar_init(&tmem_empty[a], 2 * kEpiWarps); }
    *abort = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmA);
    tc::tma_prefetch_desc(&tmB);
    tc::tma_prefetch_desc(&tmC0);
  }
  if (warp == 1) {
    tc::tmem_alloc_pair(tmem_ptr, 512);
    tc::tmem_relinquish_pair();
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync();                                        // both CTAs' barriers exist before any remote use
  tc::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;

  const int n_mt = (p.Mdim + 255) / 256, n_nt = (p.Ndim + 255) / 256;
  const int per_e = n_mt * n_nt;
  const int total = p.n_experts * per_e;

  // Ragged groups: the contraction length of a tile is its expert's row count over all layers.  The
  // experts are taken in order of decreasing length (ties by index) and dealt to the CTA pairs
  // boustrophedon-wise (first deal: pair 0 .. P-1, second deal: pair P-1 .. 0, ...), so that every deal holds
  // tiles of similar size, the long ones come first, and no pair collects the longest tile of every deal.
  uint16_t* order = reinterpret_cast<uint16_t*>(smem + kBarOffset + 512);   // [n_experts] i-th longest expert
  int* kb_of = reinterpret_cast<int*>(smem + kPairStages * kPairStageBytes);  // scratch in the (still idle) staging tiles
  for (int e = threadIdx.x; e < p.n_experts; e += blockDim.x) kb_of[e] = wgrad_kblocks(p, e);
  __syncthreads();
  for (int e = threadIdx.x; e < p.n_experts; e += blockDim.x) {
    const int mine = kb_of[e];
    int rank_e = 0;
    for (int o = 0; o < p.n_experts; ++o) {
      const int other = kb_of[o];
      rank_e += (other > mine || (other == mine && o < e)) ? 1 : 0;
    }
    order[rank_e] = (uint16_t)e;
  }
  __syncthreads();                                                           // kb_of is dead from here on

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (one in each CTA)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int round = 0; round * n_pairs < total && ok; ++round) {
        const int tile = snake_tile(round, pair, n_pairs);
        if (tile >= total) continue;
        const int e = order[tile / per_e], rem = tile % per_e, mt = rem / n_nt, nt = rem % n_nt;
        const int kblocks = wgrad_kblocks(p, e);
        int layer = 0, r = p.offsets[e], r_end = p.offsets[e + 1];
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!tc::mbar_wait(&empty_bar[stage], phase ^ 1u, abort)) { report_timeout(p, abort, 21); ok = false; break; }
          while (r >= r_end) {                          // next layer that has rows for this expert
            ++layer;
            const int32_t* off = p.offsets + (int64_t)layer * (p.n_experts + 1);
            r = off[e];
            r_end = off[e + 1];
          }
          const int grow = layer * p.layer_stride_rows + r;
          uint8_t* sA = smem + stage * kPairStageBytes;
          uint8_t* sB = sA + kPairHalfBytes;
          if (rank == 0) tc::mbar_expect_tx(&full_bar[stage], 2 * kPairStageBytes);   // both CTAs' bytes
          // this CTA's two 64-column blocks of each operand, one box each
          tc::tma_load_3d_pair(sA, &tmA, &full_bar[stage], 0, grow, mt * 4 + rank * 2);
          tc::tma_load_3d_pair(sB, &tmB, &full_bar[stage], 0, grow, nt * 4 + rank * 2);
          r += BK;
          if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok)
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = tc::instr_desc_bf16(256, true, true, 256);
      constexpr uint32_t kstep = (16 * 128) >> 4;             // descriptor units per K = 16 (MN-major)
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int round = 0; round * n_pairs < total && ok; ++round) {
        const int tile = snake_tile(round, pair, n_pairs);
        if (tile >= total) continue;
        const int kblocks = wgrad_kblocks(p, order[tile / per_e]);
        if (kblocks == 0) continue;
        const int acc = local & 1;
        const uint32_t acc_phase = (local >> 1) & 1;
        ++local;
        if (!tc::mbar_wait(&tmem_empty[acc], acc_phase ^ 1u, abort)) { report_timeout(p, abort, 22); break; }
        tc::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * 256;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!tc::mbar_wait(&full_bar[stage], phase, abort)) { report_timeout(p, abort, 23); ok = false; break; }
          tc::tc_fence_after_sync();
          const uint32_t aaddr = tc::smem_u32(smem + stage * kPairStageBytes);
          const uint64_t adesc = tc::smem_desc_sw128(aaddr, kMnBlockBytes, 1024);
          const uint64_t bdesc = tc::smem_desc_sw128(aaddr + kPairHalfBytes, kMnBlockBytes, 1024);
#pragma unroll
          for (int j = 0; j < BK / 16; ++j)
            tc::umma_bf16_pair(d_tmem, adesc + j * kstep, bdesc + j * kstep, idesc, (kb | j) != 0 ? 1u : 0u);
          tc::umma_commit_pair(&empty_bar[stage], 3);           // frees the stage in both CTAs
          if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc::umma_commit_pair(&tmem_full[acc], 3);       // accumulator complete, both CTAs
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue: this CTA's 128 rows of the tile
    const int quarter = warp & 3;
    uint8_t* stg = smem + kPairStages * kPairStageBytes + (warp - 2) * 8192;
    int gchunk = 0, local = 0;
    for (int round = 0; round * n_pairs < total; ++round) {
      const int tile = snake_tile(round, pair, n_pairs);
      if (tile >= total) continue;
      const int e = order[tile / per_e], rem = tile % per_e, mt = rem / n_nt, nt = rem % n_nt;
      const int m0 = mt * 256 + rank * 128 + quarter * 32;
      const int grow = (p.expert_base + e) * p.Mdim + m0;
      if (wgrad_kblocks(p, e) == 0) {
        if (p.overwrite && m0 < p.Mdim) {               // no rows anywhere: the gradient of this tile is zero
          if (lane == 0) tc::bulk_wait_read<0>();
          __syncwarp();
#pragma unroll
          for (int q = 0; q < 8; ++q) *f32_piece(stg, lane, q) = make_uint4(0, 0, 0, 0);
          tc::fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            for (int ch = 0; ch < 256 / kChunk; ++ch) {
              const int col = nt * 256 + ch * kChunk;
              if (col < p.Ndim) tc::tma_store_2d(&tmC0, stg, col, grow);
            }
            tc::bulk_commit();
            tc::bulk_wait_read<0>();
          }
          __syncwarp();
        }
        continue;
      }
      const int acc = local & 1;
      const uint32_t acc_phase = (local >> 1) & 1;
      ++local;
      if (!tc::mbar_wait(&tmem_full[acc], acc_phase, abort)) {
        if (lane == 0) report_timeout(p, abort, 24);
        break;
      }
      tc::tc_fence_after_sync();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * 256;
      if (m0 < p.Mdim) {
#pragma unroll 1
        for (int ch = 0; ch < 256 / kChunk; ++ch) {
          const int col = nt * 256 + ch * kChunk;
          if (col >= p.Ndim) break;
          uint32_t rr[32];
          tc::tmem_ld_32x32(t_row + ch * kChunk, rr);
          tc::tmem_ld_wait();
          uint8_t* buf = stg + (gchunk++ & 1) * kF32ChunkBytes;
          if (lane == 0) tc::bulk_wait_read<1>();        // the store issued two chunks ago has drained `buf`
          __syncwarp();
#pragma unroll
          for (int q = 0; q < 8; ++q)
            *f32_piece(buf, lane, q) = make_uint4(rr[4 * q + 0], rr[4 * q + 1], rr[4 * q + 2], rr[4 * q + 3]);
          tc::fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            if (p.overwrite) tc::tma_store_2d(&tmC0, buf, col, grow);
            else tc::tma_reduce_add_2d(&tmC0, buf, col, grow);
            tc::bulk_commit();
          }
        }
      }
      tc::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {                                   // the leader's MMA thread waits for all eight warps
        if (rank == 0) tc::mbar_arrive(&tmem_empty[acc]);
        else tc::mbar_arrive_leader(&tmem_empty[acc]);
      }
    }
    if (lane == 0) tc::bulk_wait<0>();
    __syncwarp();
  }

  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync();                                        // neither CTA leaves while the other may still signal it
  if (warp == 1) {
    tc::tc_fence_after_sync();
    tc::tmem_dealloc_pair(tmem_base, 512);
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcModule {
  EncodeTiledFn encode;
};

enum MapKind { kMapOperand, kMapBf16Chunk, kMapF32Chunk };

// Tensor map over a dense row-major tensor; dims/box innermost first, strides in elements.
//   kMapOperand   bf16, 128-byte swizzle (MMA operand tiles)
//   kMapBf16Chunk bf16, 64-byte swizzle  (32 x 32 epilogue chunks)
//   kMapF32Chunk  fp32, 128-byte swizzle (32 x 32 epilogue chunks of the weight gradient)
int make_tmap(const unipool_ctx* ctx, CUtensorMap* out, MapKind kind, const void* base, int rank,
              const uint64_t* dims, const uint64_t* strides_elems, const uint32_t* box) {
  const TcModule* mod = static_cast<const TcModule*>(ctx->tmap_cache);
  const uint64_t esz = kind == kMapF32Chunk ? 4 : 2;
  cuuint64_t gdims[3], gstrides[2];
  cuuint32_t gbox[3], estr[3] = {1, 1, 1};
  for (int i = 0; i < rank; ++i) { gdims[i] = dims[i]; gbox[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) gstrides[i] = strides_elems[i] * esz;
  UP_REQUIRE((reinterpret_cast<uintptr_t>(base) & 15) == 0, UNIPOOL_ERR_INVALID_ARG,
             "tensor base %p is not 16-byte aligned", base);
  CUresult r = mod->encode(out, kind == kMapF32Chunk ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                           (cuuint32_t)rank, const_cast<void*>(base), gdims, gstrides, gbox, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE,
                           kind == kMapBf16Chunk ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  UP_REQUIRE(r == CUDA_SUCCESS, UNIPOOL_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return UNIPOOL_OK;
}

int map_2d(const unipool_ctx* ctx, CUtensorMap* out, const void* base, uint64_t cols, uint64_t rows,
           uint32_t box_cols, uint32_t box_rows, MapKind kind = kMapOperand) {
  const uint64_t dims[2] = {cols, rows}, strides[1] = {cols};
  const uint32_t box[2] = {box_cols, box_rows};
  return make_tmap(ctx, out, kind, base, 2, dims, strides, box);
}

// MMA operand read along the contiguous dimension of a row-major matrix [k_rows, n_cols] ("MN-major"):
// the matrix seen as [n_cols / 64][k_rows][64], a box = `blocks` column blocks x 64 k-rows, laid out
// block after block (8 KiB each) - one copy instead of one per block.
int map_mn(const unipool_ctx* ctx, CUtensorMap* out, const void* base, uint64_t n_cols, uint64_t k_rows,
           uint32_t blocks) {
  const uint64_t dims[3] = {64, k_rows, n_cols / 64}, strides[2] = {n_cols, 64};
  const uint32_t box[3] = {64, 64, blocks};
  return make_tmap(ctx, out, kMapOperand, base, 3, dims, strides, box);
}

// 32 x 32 epilogue chunk map
int map_chunk(const unipool_ctx* ctx, CUtensorMap* out, const void* base, uint64_t cols, uint64_t rows,
              MapKind kind) {
  return map_2d(ctx, out, base, cols, rows, kChunk, 32, kind);
}

// ---------------------------------------------------------------- row-tile GEMMs on CTA pairs
// A 128 x 256 tile takes 48 KB of operands per k-block, most of it the expert's weights, which the
// other row tiles of the same expert fetch again, and an SM cannot pull more than ~100 GB/s out of
// L2.  Here two row tiles of ONE expert share a CTA pair: one tcgen05.mma.cta_group::2 of M = 256
// (128 rows per CTA, each in its own TMEM) and N = 256, each CTA loading its own 128 rows of A and
// HALF of the expert's 256 weight rows (B), 32 KB per k-block and CTA, six stages.  The odd last tile
// of a group is a half pair-tile: the M = 128 form of the same instruction, 64 rows per CTA (24 KB per
// k-block and CTA).  Scheduling, barriers and commits follow the weight-gradient pair kernel above; the
// epilogues are the single-CTA ones, addressed through the two accumulator layouts.
// Six operand stages and four epilogue warps: a variant with eight epilogue warps (two per TMEM lane
// quarter, taking alternate chunks) had to give one stage to their staging tiles and was 8 - 12 %
// slower - the main loop lives on the bytes it keeps in flight.
// The SwiGLU-derivative GEMM keeps its organisation of the single-CTA kernel (eight epilogue warps, one
// operand mover per TMEM lane quarter, G and U turned into dG and dU in place in a ring of chunk
// buffers): four operand stages, and a ring of six chunk pairs per quarter in the room the other two took.
template <int MODE> struct PairTraits {
  static constexpr bool kIo = MODE == kDgrad1;
  static constexpr int kStages = kIo ? 4 : 6;
  static constexpr int kEpiWarps = kIo ? 8 : 4;
  static constexpr int kThreads = 64 + 32 * kEpiWarps + (kIo ? 128 : 0);
  static constexpr uint32_t kStagingOffset = kStages * kPairStageBytes;
  static constexpr uint32_t kStagingPerQuarter = kIo ? 24576 : 8192;
  static_assert(kStagingOffset + 4 * kStagingPerQuarter == kBarOffset, "shared-memory budget");
};
constexpr int kPairRing = 6, kPairAhead = 3;           // dgrad1: ring slots per quarter, prefetch distance
static_assert(kPairRing * 2 * kBf16ChunkBytes == PairTraits<kDgrad1>::kStagingPerQuarter, "ring size");

// half: the pair-tile is ONE row tile (the odd last tile of a group): each CTA takes 64 of its rows and the
// MMA is the M = 128 form of cta_group::2.
struct PairTile { int e, mt, nt; bool half; };

// pair-tile q of the row space -> expert and first row tile; pp[e] = pair-tiles before expert e
__device__ __forceinline__ PairTile pair_tile(const GemmParams& p, const uint16_t* pp, int tile, int n_nt,
                                              int total_q, bool descending) {
  PairTile t;
  int q = tile / n_nt;
  t.nt = tile % n_nt;
  if (descending) q = total_q - 1 - q;
  int lo = 0, hi = p.n_experts - 1;                    // last e with pp[e] <= q
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if ((int)pp[mid] <= q) lo = mid; else hi = mid - 1;
  }
  t.e = lo;
  const int first = p.group_offsets[lo] / BM, n_tiles = (p.group_offsets[lo + 1] - p.group_offsets[lo]) / BM;
  const int i = 2 * (q - (int)pp[lo]);
  t.mt = first + i;
  t.half = i + 1 >= n_tiles;
  return t;
}

// dgrad1 on pairs: the chunks (32 rows x 32 columns of dA) that the epilogue warps of TMEM lane quarter
// `quarter` of CTA `rank` own in pair-tile t: first row, first column and how many (chunk i sits at TMEM
// column 32 i under both accumulator layouts described below).
__device__ __forceinline__ void pair_chunks(const GemmParams& p, const PairTile& t, int rank, int quarter, int& row0,
                                            int& col0, int& nch) {
  if (!t.half) {
    row0 = (t.mt + rank) * BM + quarter * 32;
    col0 = t.nt * BN;
    nch = min(BN / kChunk, (p.f - col0) / kChunk);
  } else {
    row0 = t.mt * BM + rank * (BM / 2) + (quarter & 1) * 32;
    col0 = t.nt * BN + (BN / 2) * (quarter >> 1);
    nch = max(0, min(BN / 2 / kChunk, (p.f - col0) / kChunk));
  }
}

// The (G, U) chunks of one lane quarter over all pair-tiles of this CTA pair, in the order the epilogue
// consumes them (see ChunkCursor).
struct PairChunkCursor {
  int tile, ch, nch, col0, row0;
  __device__ void seek(const GemmParams& p, const uint16_t* pp, int total, int n_nt, int total_q, int rank, int quarter) {
    while (tile < total) {
      pair_chunks(p, pair_tile(p, pp, tile, n_nt, total_q, false), rank, quarter, row0, col0, nch);
      ch = 0;
      if (nch > 0) return;
      tile += gridDim.x >> 1;
    }
  }
  __device__ void start(const GemmParams& p, const uint16_t* pp, int total, int n_nt, int total_q, int rank, int quarter) {
    tile = blockIdx.x >> 1; ch = 0; nch = 0; col0 = 0; row0 = 0;
    seek(p, pp, total, n_nt, total_q, rank, quarter);
  }
  __device__ void next(const GemmParams& p, const uint16_t* pp, int total, int n_nt, int total_q, int rank, int quarter) {
    if (++ch == nch) { tile += gridDim.x >> 1; seek(p, pp, total, n_nt, total_q, rank, quarter); }
  }
  __device__ int col() const { return col0 + ch * kChunk; }
};

// Accumulator layouts (read back with tcgen05.ld, lanes [32 w, 32 w + 32) for warp w of a CTA):
//   M = 256: the CTA's 128 rows are lanes 0..127, the tile's 256 columns TMEM columns 0..255;
//   M = 128: the CTA's 64 rows are lanes 0..63 for columns 0..127 AND lanes 64..127 for columns
//            128..255, both at TMEM columns 0..127.
// B halves: CTA r supplies columns [128 r, 128 r + 128) of the tile.  For the gate/up projection each
// half is [64 gate features | the same 64 up features], so that G and U of one element meet in one
// thread under both layouts.
template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PairTraits<MODE>::kThreads, 1)
row_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA64,
                const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmC0,
                const __grid_constant__ CUtensorMap tmC1, const GemmParams p) {
  static_assert(Traits<MODE>::kRowTiles, "row tiles");
  using PT = PairTraits<MODE>;
  constexpr int kRowPairStages = PT::kStages;
  constexpr int kRowPairEpiWarps = PT::kEpiWarps;
  constexpr bool kBMn = Traits<MODE>::kBMn;
  constexpr bool kDescending = MODE == kFwd2 || MODE == kDgrad2;      // see tile_coord
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kBarOffset);
  uint64_t* empty_bar = full_bar + kRowPairStages;
  uint64_t* tmem_full = empty_bar + kRowPairStages;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* epi_bar = tmem_empty + 2;                        // dgrad1: [4][kPairRing] a chunk's G and U have landed
  uint64_t* staged_bar = epi_bar + (PT::kIo ? 4 * kPairRing : 0);   // dgrad1: [4][kPairRing] dG and dU are staged
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(staged_bar + (PT::kIo ? 4 * kPairRing : 0));
  volatile int* abort = reinterpret_cast<volatile int*>(tmem_ptr + 1);
  static_assert((2 * PT::kStages + 4 + (PT::kIo ? 8 * kPairRing : 0)) * 8 + 8 <= 512, "barrier block");
  uint16_t* pp = reinterpret_cast<uint16_t*>(smem + kBarOffset + 512);       // [n_experts + 1]

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int rank = (int)tc::cluster_ctarank();               // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kRowPairStages; ++s) { tc::mbar_init(&full_bar[s], 1); tc::mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { tc::mbar_init(&tmem_full[a], 1); tc::mbar_init(&tmem_empty[a], 2 * kRowPairEpiWarps); }
    if constexpr (PT::kIo)
      for (int i = 0; i < 4 * kPairRing; ++i) { tc::mbar_init(&epi_bar[i], 1); tc::mbar_init(&staged_bar[i], 1); }
    *abort = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmA);
    tc::tma_prefetch_desc(&tmA64);
    tc::tma_prefetch_desc(&tmB);
    tc::tma_prefetch_desc(&tmC0);
    if constexpr (MODE == kFwd1 || MODE == kDgrad1) tc::tma_prefetch_desc(&tmC1);
  }
  if (warp == 1) {
    tc::tmem_alloc_pair(tmem_ptr, 512);
    tc::tmem_relinquish_pair();
  }
  // pair-tiles before each expert: an expert of n row tiles takes ceil(n / 2), the last one a half
  // pair-tile when n is odd
  for (int e = threadIdx.x; e <= p.n_experts; e += blockDim.x) {
    int before = 0;
    for (int o = 0; o < e; ++o) before += ((p.group_offsets[o + 1] - p.group_offsets[o]) / BM + 1) >> 1;
    pp[e] = (uint16_t)before;
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync();                                        // both CTAs' barriers exist before any remote use
  tc::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr;

  const int ncols = MODE == kFwd1 ? BN / 2 : BN;             // output columns (fwd1: features) per tile
  const int n_nt = (p.Ndim + ncols - 1) / ncols;
  const int total_q = pp[p.n_experts];
  const int total = total_q * n_nt;
  const int kblocks = p.Kdim / BK;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (one in each CTA)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; tile < total && ok; tile += n_pairs) {
        const PairTile t = pair_tile(p, pp, tile, n_nt, total_q, kDescending);
        const int pe = p.expert_base + t.e;
        const uint32_t tx = 2 * (kPairHalfBytes + (t.half ? kPairHalfBytes / 2 : kPairHalfBytes));
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!tc::mbar_wait(&empty_bar[stage], phase ^ 1u, abort)) { report_timeout(p, abort, 31); ok = false; break; }
          uint8_t* sA = smem + stage * kPairStageBytes;
          uint8_t* sB = sA + kPairHalfBytes;
          if (rank == 0) tc::mbar_expect_tx(&full_bar[stage], tx);              // both CTAs' bytes
          if (t.half) tc::tma_load_2d_pair(sA, &tmA64, &full_bar[stage], kb * BK, t.mt * BM + rank * (BM / 2));
          else tc::tma_load_2d_pair(sA, &tmA, &full_bar[stage], kb * BK, (t.mt + rank) * BM);
          if constexpr (MODE == kFwd1) {           // 64 gate features and the same 64 up features: W_gu as [2M][f][d]
            tc::tma_load_3d_pair(sB, &tmB, &full_bar[stage], kb * BK, t.nt * (BN / 2) + rank * 64, 2 * pe);
          } else if constexpr (MODE == kFwd2) {    // 128 rows of W_down
            tc::tma_load_2d_pair(sB, &tmB, &full_bar[stage], kb * BK, pe * p.Ndim + t.nt * BN + rank * (BN / 2));
          } else {                                 // two 64-column blocks of the MN-major weights (W_down, W_gu)
            tc::tma_load_3d_pair(sB, &tmB, &full_bar[stage], 0, pe * p.Kdim + kb * BK, t.nt * 4 + rank * 2);
          }
          if (++stage == kRowPairStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok)
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc_full = tc::instr_desc_bf16(BN, false, kBMn, 256);
      constexpr uint32_t idesc_half = tc::instr_desc_bf16(BN, false, kBMn, 128);
      constexpr uint32_t b_lbo = kBMn ? kMnBlockBytes : 16;
      constexpr uint32_t a_step = 32 >> 4;                                   // K-major: 32 bytes per K = 16
      constexpr uint32_t b_step = (kBMn ? 16 * 128 : 32) >> 4;
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int tile = pair; tile < total && ok; tile += n_pairs) {
        const PairTile t = pair_tile(p, pp, tile, n_nt, total_q, kDescending);
        const uint32_t idesc = t.half ? idesc_half : idesc_full;
        const int acc = local & 1;
        const uint32_t acc_phase = (local >> 1) & 1;
        ++local;
        if (!tc::mbar_wait(&tmem_empty[acc], acc_phase ^ 1u, abort)) { report_timeout(p, abort, 32); break; }
        tc::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!tc::mbar_wait(&full_bar[stage], phase, abort)) { report_timeout(p, abort, 33); ok = false; break; }
          tc::tc_fence_after_sync();
          const uint32_t aaddr = tc::smem_u32(smem + stage * kPairStageBytes);
          const uint64_t adesc = tc::smem_desc_sw128(aaddr, 16, 1024);
          const uint64_t bdesc = tc::smem_desc_sw128(aaddr + kPairHalfBytes, b_lbo, 1024);
#pragma unroll
          for (int j = 0; j < BK / 16; ++j)
            tc::umma_bf16_pair(d_tmem, adesc + j * a_step, bdesc + j * b_step, idesc, (kb | j) != 0 ? 1u : 0u);
          tc::umma_commit_pair(&empty_bar[stage], 3);           // frees the stage in both CTAs
          if (++stage == kRowPairStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc::umma_commit_pair(&tmem_full[acc], 3);       // accumulator complete, both CTAs
      }
    }
  } else if (PT::kIo && warp >= 2 + kRowPairEpiWarps) {
    // ------------------------------------------------------------ dgrad1: operand mover of one lane quarter
    // (one lane; see the single-CTA kernel: G and U are fetched kPairAhead chunks ahead into the quarter's
    // ring and written back as dG, dU once the epilogue warps have rewritten them in place)
    if constexpr (PT::kIo) {
      if (lane == 0) {
        const int ew = warp - (2 + kRowPairEpiWarps);
        const int quarter = (ew + 2) & 3;
        uint8_t* stg = smem + PT::kStagingOffset + ew * PT::kStagingPerQuarter;
        uint64_t* full = epi_bar + kPairRing * ew;
        uint64_t* staged = staged_bar + kPairRing * ew;
        PairChunkCursor ld, st;
        ld.start(p, pp, total, n_nt, total_q, rank, quarter);
        st.start(p, pp, total, n_nt, total_q, rank, quarter);
        int fetched = 0, stored = 0;
        bool ok = true;
        while (st.tile < total && ok) {
          // Chunk n uses slot n % kPairRing.  When chunk `fetched` < stored + kPairAhead is fetched, the
          // store that last read its slot (chunk fetched - kPairRing) is followed by at least
          // kPairRing - kPairAhead committed stores: all but that many must have drained.
          while (fetched < stored + kPairAhead && ld.tile < total) {
            const int slot = fetched % kPairRing;
            uint8_t* buf = stg + slot * 2 * kBf16ChunkBytes;
            tc::bulk_wait_read<kPairRing - kPairAhead - 1>();
            tc::mbar_expect_tx(&full[slot], 2 * kBf16ChunkBytes);
            tc::tma_load_2d(buf, &tmC1, &full[slot], ld.col(), ld.row0);
            tc::tma_load_2d(buf + kBf16ChunkBytes, &tmC1, &full[slot], p.f + ld.col(), ld.row0);
            ++fetched;
            ld.next(p, pp, total, n_nt, total_q, rank, quarter);
          }
          const int slot = stored % kPairRing;
          uint8_t* buf = stg + slot * 2 * kBf16ChunkBytes;
          if (!tc::mbar_wait(&staged[slot], (stored / kPairRing) & 1, abort)) { report_timeout(p, abort, 36); ok = false; break; }
          tc::tma_store_2d(&tmC0, buf, st.col(), st.row0);
          tc::tma_store_2d(&tmC0, buf + kBf16ChunkBytes, p.f + st.col(), st.row0);
          tc::bulk_commit();
          ++stored;
          st.next(p, pp, total, n_nt, total_q, rank, quarter);
        }
        if (!ok)
          for (int i = 0; i < 200; ++i) __nanosleep(1000);   // let loads already in flight land
        tc::bulk_wait<0>();
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue: this CTA's rows of the pair-tile
    // (dgrad1: two warps per lane quarter, warps w and w + 4, share the quarter's ring and take alternate chunks)
    const int quarter = warp & 3;
    const int ew = (warp - 2) & 3;
    uint8_t* stg = smem + PT::kStagingOffset + ew * PT::kStagingPerQuarter;
    int gchunk = 0, local = 0;
    (void)gchunk;
    bool ok = true;
    for (int tile = pair; tile < total && ok; tile += n_pairs) {
      const PairTile t = pair_tile(p, pp, tile, n_nt, total_q, kDescending);
      const int acc = local & 1;
      const uint32_t acc_phase = (local >> 1) & 1;
      ++local;
      if (!tc::mbar_wait(&tmem_full[acc], acc_phase, abort)) {
        if (lane == 0) report_timeout(p, abort, 34);
        break;
      }
      tc::tc_fence_after_sync();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * BN;
      if constexpr (MODE == kDgrad1) {
        const int half = (warp - 2) >> 2;
        uint64_t* my_bar = epi_bar + kPairRing * ew;
        uint64_t* my_staged = staged_bar + kPairRing * ew;
        int row0, col0, nch;
        pair_chunks(p, t, rank, quarter, row0, col0, nch);
#pragma unroll 1
        for (int ch = 0; ch < nch; ++ch) {
          if (((gchunk + ch) & 1) != half) continue;    // the other warp of this quarter takes it
          const int slot = (gchunk + ch) % kPairRing;
          const uint32_t slot_phase = ((gchunk + ch) / kPairRing) & 1;
          uint8_t* buf = stg + slot * 2 * kBf16ChunkBytes;
          uint32_t rr[32];
          tc::tmem_ld_32x32(t_row + ch * kChunk, rr);
          tc::tmem_ld_wait();
          if (!tc::mbar_wait(&my_bar[slot], slot_phase, abort)) {
            if (lane == 0) report_timeout(p, abort, 35);
            ok = false;
            break;
          }
          float g[32], u[32], dg[32], du[32];
          unstage_row_bf16(buf, lane, g);
          unstage_row_bf16(buf + kBf16ChunkBytes, lane, u);
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float dA = __uint_as_float(rr[i]);
            const float sig = sigmoid_fast(g[i]);
            const float sl = g[i] * sig;
            dg[i] = dA * u[i] * (sig + sl * (1.0f - sig));   // silu'(g) = sig (1 + g (1 - sig))
            du[i] = dA * sl;
          }
          stage_row_bf16(buf, lane, dg);               // in place: each lane rewrites the row it read
          stage_row_bf16(buf + kBf16ChunkBytes, lane, du);
          tc::fence_proxy_async();
          __syncwarp();
          if (lane == 0) tc::mbar_arrive(&my_staged[slot]);   // the operand mover stores the chunk
        }
        gchunk += nch;
        if (!ok) break;
      } else if (!t.half) {
        const int row0 = (t.mt + rank) * BM + quarter * 32;
        if constexpr (MODE == kFwd1) {
#pragma unroll 1
          for (int h = 0; h < 2; ++h)                    // the two B halves: features [64 h, 64 h + 64) of the tile
            epilogue_swiglu(&tmC0, &tmC1, p, t_row + 128 * h, t_row + 128 * h + 64, t.nt * (BN / 2) + 64 * h, 2, row0,
                            stg, lane);
        } else {
          epilogue_rows<MODE>(&tmC0, p, t_row, t.nt * BN, BN, row0, stg, lane, gchunk);
        }
      } else {
        const int h = quarter >> 1;                      // lanes 64..127 hold the second half of the columns
        const int row0 = t.mt * BM + rank * (BM / 2) + (quarter & 1) * 32;
        if constexpr (MODE == kFwd1)
          epilogue_swiglu(&tmC0, &tmC1, p, t_row, t_row + 64, t.nt * (BN / 2) + 64 * h, 2, row0, stg, lane);
        else if constexpr (MODE != kDgrad1)
          epilogue_rows<MODE>(&tmC0, p, t_row, t.nt * BN + 128 * h, BN / 2, row0, stg, lane, gchunk);
      }
      tc::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {                                   // the leader's MMA thread waits for both CTAs' epilogue warps
        if (rank == 0) tc::mbar_arrive(&tmem_empty[acc]);
        else tc::mbar_arrive_leader(&tmem_empty[acc]);
      }
    }
    if (!ok && lane == 0)
      for (int i = 0; i < 200; ++i) __nanosleep(1000);       // let loads already in flight land before the CTA retires
    if (lane < 3) tc::bulk_wait<0>();
    __syncwarp();
  }

  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync();                                        // neither CTA leaves while the other may still signal it
  if (warp == 1) {
    tc::tc_fence_after_sync();
    tc::tmem_dealloc_pair(tmem_base, 512);
  }
}

template <int MODE>
int launch(unipool_ctx* ctx, int phase, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmB64,
           const CUtensorMap& tmC0, const CUtensorMap& tmC1, const GemmParams& p, cudaStream_t s) {
  PhaseTimer pt(ctx, phase, 1, s);
  auto kern = grouped_gemm_tc_kernel<MODE>;
  UP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemTotal));
  kern<<<ctx->sm_count, Traits<MODE>::kThreads, kSmemTotal, s>>>(tmA, tmB, tmB64, tmC0, tmC1, p);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

// The four row-tile GEMMs (gate/up, down, both dgrads) of a call run either all on the single-CTA kernel or
// all on CTA pairs (the odd last tile of a group as a half pair-tile, M = 128).  Pairs move a third
// fewer operand bytes into the SMs.  Measured (interleaved runs, one B200), pairs against single per
// GEMM: -10 % at 32 row tiles per group, -3 .. -8 % at 4 - 7 tiles, none at 2.7 tiles (341 rows): a
// half pair-tile uses the tensor cores at half rate, and every third tile is one.  So: pairs when a
// batch of max_tokens gives the average expert four row tiles, single otherwise.  The pair schedule
// keeps 16-bit counts of pair-tiles.
bool rows_on_pairs(const unipool_ctx* ctx, int n_experts) {
  if (ctx->sm_count < 2 || ctx->row_capacity / (2 * BM) + n_experts >= 65535) return false;
  return (int64_t)ctx->cfg.max_tokens * ctx->cfg.top_k >= (int64_t)4 * BM * n_experts;
}

// One row-tile GEMM.  tmA / tmB / tmB64: the operand maps of the single-CTA kernel (tmB64: 64 x 64 boxes
// of the weights for the column slices of the second dgrad); tmA64 / tmBp: those of the pair kernel's
// half pair-tiles (64-row boxes of A) and of its B halves.
template <int MODE>
int launch_rows(unipool_ctx* ctx, int phase, bool pairs, const CUtensorMap& tmA, const CUtensorMap& tmA64,
                const CUtensorMap& tmB, const CUtensorMap& tmB64, const CUtensorMap& tmBp, const CUtensorMap& tmC0,
                const CUtensorMap& tmC1, const GemmParams& p, cudaStream_t s) {
  PhaseTimer pt(ctx, phase, 1, s);
  if (pairs) {
    auto kern = row_pair_kernel<MODE>;
    UP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmemTotal));
    kern<<<ctx->sm_count / 2 * 2, PairTraits<MODE>::kThreads, kPairSmemTotal, s>>>(tmA, tmA64, tmBp, tmC0, tmC1, p);
  } else {
    auto kern = grouped_gemm_tc_kernel<MODE>;
    UP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemTotal));
    kern<<<ctx->sm_count, Traits<MODE>::kThreads, kSmemTotal, s>>>(tmA, tmB, tmB64, tmC0, tmC1, p);
  }
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

// The pool weight gradient runs on CTA pairs.
int launch_wgrad(unipool_ctx* ctx, int phase, const CUtensorMap& tmP, const CUtensorMap& tmQ, const CUtensorMap& tmW,
                 const GemmParams& p, cudaStream_t s) {
  UP_REQUIRE(ctx->sm_count >= 2, UNIPOOL_ERR_UNSUPPORTED, "the weight gradient needs a device with CTA pairs");
  PhaseTimer pt(ctx, phase, 1, s);
  UP_CUDA(cudaFuncSetAttribute(wgrad_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmemTotal));
  wgrad_pair_kernel<<<ctx->sm_count / 2 * 2, kThreads, kPairSmemTotal, s>>>(tmP, tmQ, tmW, p);
  UP_LAUNCH_CHECK();
  return UNIPOOL_OK;
}

int wgrad_pair(unipool_ctx* ctx, const PoolWgradArgs& a, cudaStream_t s) {
  const int d = ctx->cfg.d_model, f = ctx->cfg.d_ff, M = ctx->cfg.pool_size;
  const uint64_t rows = (uint64_t)(a.n_layers > 1 ? (int64_t)a.n_layers * a.layer_stride_rows : ctx->row_capacity);
  GemmParams p{};
  p.offsets = a.offsets;
  p.n_experts = a.n_experts;
  p.expert_base = a.expert_base;
  p.n_layers = a.n_layers;
  p.layer_stride_rows = (int)a.layer_stride_rows;
  p.overwrite = a.overwrite ? 1 : 0;
  p.status = ctx->ws.status;
  CUtensorMap tmP, tmQ, tmW;
  int rc;
  if (a.dW_down != nullptr) {                     // dW_down[e] [d, f] (+)= dYp_e^T A_e
    if ((rc = map_mn(ctx, &tmP, a.dYp, d, rows, 2)) != UNIPOOL_OK) return rc;
    if ((rc = map_mn(ctx, &tmQ, a.A, f, rows, 2)) != UNIPOOL_OK) return rc;
    if ((rc = map_chunk(ctx, &tmW, a.dW_down, f, (uint64_t)M * d, kMapF32Chunk)) != UNIPOOL_OK) return rc;
    p.Mdim = d; p.Ndim = f;
    if ((rc = launch_wgrad(ctx, UNIPOOL_PH_WGRAD_DOWN, tmP, tmQ, tmW, p, s)) != UNIPOOL_OK) return rc;
  }
  if (a.dW_gu == nullptr) return UNIPOOL_OK;
  // dW_gu[e] [2f, d] (+)= dGU_e^T Xp_e
  if ((rc = map_mn(ctx, &tmP, a.dGU, 2 * f, rows, 2)) != UNIPOOL_OK) return rc;
  if ((rc = map_mn(ctx, &tmQ, a.Xp, d, rows, 2)) != UNIPOOL_OK) return rc;
  if ((rc = map_chunk(ctx, &tmW, a.dW_gu, d, (uint64_t)M * 2 * f, kMapF32Chunk)) != UNIPOOL_OK) return rc;
  p.Mdim = 2 * f; p.Ndim = d;
  return launch_wgrad(ctx, UNIPOOL_PH_WGRAD_GU, tmP, tmQ, tmW, p, s);
}

}  // namespace

int tc_module_init(unipool_ctx* ctx) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
  UP_REQUIRE(e == cudaSuccess && fn != nullptr && q == cudaDriverEntryPointSuccess, UNIPOOL_ERR_CUDA,
             "cuTensorMapEncodeTiled is not available from the driver (%s)", cudaGetErrorString(e));
  TcModule* mod = new TcModule{reinterpret_cast<EncodeTiledFn>(fn)};
  ctx->tmap_cache = mod;
  return UNIPOOL_OK;
}

void tc_module_destroy(unipool_ctx* ctx) {
  delete static_cast<TcModule*>(ctx->tmap_cache);
  ctx->tmap_cache = nullptr;
}

int expert_fwd_tc(unipool_ctx* ctx, const ExpertFwdArgs& a, cudaStream_t s) {
  const int d = ctx->cfg.d_model, f = ctx->cfg.d_ff, M = ctx->cfg.pool_size;
  const uint64_t cap = (uint64_t)ctx->row_capacity;
  GemmParams p{};
  p.offsets = a.offsets + a.n_experts;
  p.tile_expert = a.tile_expert;
  p.n_experts = a.n_experts;
  p.expert_base = a.expert_base;
  p.f = f;
  p.status = ctx->ws.status;
  p.group_offsets = a.offsets;
  const bool plan = rows_on_pairs(ctx, a.n_experts);
  CUtensorMap tmA, tmA64, tmB, tmBp, tmC0, tmC1;
  int rc;
  // GU = Xp [W_gate; W_up]^T with the SwiGLU epilogue.  B tile = 128 gate rows + 128 up rows of the
  // same features, fetched as one 3-D box over W_gu viewed as [2M, f, d] (CTA pairs: one half each,
  // 128 rows of W_gu viewed as [2M f, d]).
  if ((rc = map_2d(ctx, &tmA, a.Xp, d, cap, 64, BM)) != UNIPOOL_OK) return rc;
  if ((rc = map_2d(ctx, &tmA64, a.Xp, d, cap, 64, 64)) != UNIPOOL_OK) return rc;
  {
    const uint64_t dims[3] = {(uint64_t)d, (uint64_t)f, (uint64_t)2 * M};
    const uint64_t strides[2] = {(uint64_t)d, (uint64_t)f * d};
    const uint32_t box[3] = {64, BN / 2, 2}, box_pair[3] = {64, BN / 4, 2};
    if ((rc = make_tmap(ctx, &tmB, kMapOperand, a.W_gu, 3, dims, strides, box)) != UNIPOOL_OK) return rc;
    if ((rc = make_tmap(ctx, &tmBp, kMapOperand, a.W_gu, 3, dims, strides, box_pair)) != UNIPOOL_OK) return rc;
  }
  if ((rc = map_chunk(ctx, &tmC0, a.GU, 2 * f, cap, kMapBf16Chunk)) != UNIPOOL_OK) return rc;
  if ((rc = map_chunk(ctx, &tmC1, a.A, f, cap, kMapBf16Chunk)) != UNIPOOL_OK) return rc;
  p.Ndim = f; p.Kdim = d;
  if ((rc = launch_rows<kFwd1>(ctx, UNIPOOL_PH_EXPERT_FWD_GU, plan, tmA, tmA64, tmB, tmB, tmBp, tmC0, tmC1, p, s)) != UNIPOOL_OK)
    return rc;
  // Yp = A W_down^T
  if ((rc = map_2d(ctx, &tmA, a.A, f, cap, 64, BM)) != UNIPOOL_OK) return rc;
  if ((rc = map_2d(ctx, &tmA64, a.A, f, cap, 64, 64)) != UNIPOOL_OK) return rc;
  if ((rc = map_2d(ctx, &tmB, a.W_down, f, (uint64_t)M * d, 64, BN)) != UNIPOOL_OK) return rc;
  if ((rc = map_2d(ctx, &tmBp, a.W_down, f, (uint64_t)M * d, 64, BN / 2)) != UNIPOOL_OK) return rc;   // a CTA's half
  if ((rc = map_2d(ctx, &tmC1, a.W_down, f, (uint64_t)M * d, 64, 64)) != UNIPOOL_OK) return rc;       // column slices
  if ((rc = map_chunk(ctx, &tmC0, a.Yp, d, cap, kMapBf16Chunk)) != UNIPOOL_OK) return rc;
  p.Ndim = d; p.Kdim = f;
  return launch_rows<kFwd2>(ctx, UNIPOOL_PH_EXPERT_FWD_DOWN, plan, tmA, tmA64, tmB, tmB, tmBp, tmC0, tmC1, p, s);
}

int expert_bwd_tc(unipool_ctx* ctx, const ExpertBwdArgs& a, cudaStream_t s) {
  const int d = ctx->cfg.d_model, f = ctx->cfg.d_ff, M = ctx->cfg.pool_size;
  const uint64_t cap = (uint64_t)ctx->row_capacity;
  GemmParams p{};
  p.offsets = a.offsets + a.n_experts;
  p.tile_expert = a.tile_expert;
  p.n_experts = a.n_experts;
  p.expert_base = a.expert_base;
  p.f = f;
  p.status = ctx->ws.status;
  p.group_offsets = a.offsets;
  const bool plan = rows_on_pairs(ctx, a.n_experts);
  CUtensorMap tmA, tmA64, tmB, tmB64, tmBp, tmC0, tmC1;
  int rc;
  // dA = dYp W_down, fused with the SwiGLU derivative -> dGU
  if ((rc = map_2d(ctx, &tmA, a.dYp, d, cap, 64, BM)) != UNIPOOL_OK) return rc;
  if ((rc = map_2d(ctx, &tmA64, a.dYp, d, cap, 64, 64)) != UNIPOOL_OK) return rc;
  if ((rc = map_mn(ctx, &tmB, a.W_down, f, (uint64_t)M * d, BN / 64)) != UNIPOOL_OK) return rc;
  if ((rc = map_mn(ctx, &tmBp, a.W_down, f, (uint64_t)M * d, BN / 128)) != UNIPOOL_OK) return rc;
  if ((rc = map_2d(ctx, &tmB64, a.W_down, f, (uint64_t)M * d, 64, 64)) != UNIPOOL_OK) return rc;
  if ((rc = map_chunk(ctx, &tmC0, a.dGU, 2 * f, cap, kMapBf16Chunk)) != UNIPOOL_OK) return rc;
  if ((rc = map_chunk(ctx, &tmC1, a.GU, 2 * f, cap, kMapBf16Chunk)) != UNIPOOL_OK) return rc;
  p.Ndim = f; p.Kdim = d;
  rc = launch_rows<kDgrad1>(ctx, UNIPOOL_PH_DGRAD_DOWN, plan, tmA, tmA64, tmB, tmB64, tmBp, tmC0, tmC1, p, s);
  if (rc != UNIPOOL_OK) return rc;
  // dXp = dGU [W_gate; W_up]
  if ((rc = map_2d(ctx, &tmA, a.dGU, 2 * f, cap, 64, BM)) != UNIPOOL_OK) return rc;
  if ((rc = map_mn(ctx, &tmB, a.W_gu, d, (uint64_t)M * 2 * f, BN / 64)) != UNIPOOL_OK) return rc;
  if ((rc = map_mn(ctx, &tmBp, a.W_gu, d, (uint64_t)M * 2 * f, BN / 128)) != UNIPOOL_OK) return rc;
  if ((rc = map_2d(ctx, &tmB64, a.W_gu, d, (uint64_t)M * 2 * f, 64, 64)) != UNIPOOL_OK) return rc;
  if ((rc = map_chunk(ctx, &tmC0, a.dXp, d, cap, kMapBf16Chunk)) != UNIPOOL_OK) return rc;
  p.Ndim = d; p.Kdim = 2 * f; p.overwrite = 1;
  if ((rc = map_2d(ctx, &tmA64, a.dGU, 2 * f, cap, 64, 64)) != UNIPOOL_OK) return rc;
  rc = launch_rows<kDgrad2>(ctx, UNIPOOL_PH_DGRAD_GU, plan, tmA, tmA64, tmB, tmB64, tmBp, tmC0, tmC0, p, s);
  if (rc != UNIPOOL_OK) return rc;
  if (a.wgrad) {
    PoolWgradArgs w{1, 0, a.offsets, a.Xp, a.A, a.dYp, a.dGU, a.expert_base, a.n_experts, a.dW_gu, a.dW_down,
                    a.overwrite};
    return wgrad_pair(ctx, w, s);
  }
  return UNIPOOL_OK;
}

int pool_wgrad_tc(unipool_ctx* ctx, const PoolWgradArgs& a, cudaStream_t s) { return wgrad_pair(ctx, a, s); }

int tc_operand_map(unipool_ctx* ctx, void* out, const void* base, uint64_t cols, uint64_t rows, uint32_t box_rows) {
  return map_2d(ctx, static_cast<CUtensorMap*>(out), base, cols, rows, 64, box_rows);
}

// fp32 [rows, cols] map of 32 x 32 chunks with the 128-byte swizzle (epilogue-style stores)
int tc_f32_chunk_map(unipool_ctx* ctx, void* out, const void* base, uint64_t cols, uint64_t rows) {
  return map_chunk(ctx, static_cast<CUtensorMap*>(out), base, cols, rows, kMapF32Chunk);
}

// Router backward GEMMs (bf16 mode).  dz16 [T, Mp] bf16 (Mp = M rounded up to 64, pad columns
// zero), W16 [M, d] bf16, x [T, d] bf16:
//   dx [T, d] bf16 += dz16 W16        (row tiles, one group, TMA add-reduce into dx)
//   dW_r [M, d] fp32 += dz16^T x      (tokens split evenly over the CTAs, TMA add-reduce)
int router_bwd_gemms_tc(unipool_ctx* ctx, const void* dz16, int Mp, const void* W16, const void* x, int T, int M,
                        void* dx, float* dW_r, cudaStream_t s) {
  const int d = ctx->cfg.d_model;
  GemmParams p{};
  p.status = ctx->ws.status;
  p.n_experts = 1;
  CUtensorMap tmA, tmB, tmB64, tmC;
  int rc;
  if ((rc = map_2d(ctx, &tmA, dz16, Mp, T, 64, BM)) != UNIPOOL_OK) return rc;
  if ((rc = map_mn(ctx, &tmB, W16, d, M, BN / 64)) != UNIPOOL_OK) return rc;
  if ((rc = map_2d(ctx, &tmB64, W16, d, M, 64, 64)) != UNIPOOL_OK) return rc;
  if ((rc = map_chunk(ctx, &tmC, dx, d, T, kMapBf16Chunk)) != UNIPOOL_OK) return rc;
  p.Mdim = (T + BM - 1) / BM; p.Ndim = d; p.Kdim = Mp; p.overwrite = 0;
  if ((rc = launch<kDgrad2>(ctx, UNIPOOL_PH_ROUTE_BWD_DX, tmA, tmB, tmB64, tmC, tmC, p, s)) != UNIPOOL_OK) return rc;

  const int out_tiles = ((M + BM - 1) / BM) * ((d + BN - 1) / BN);
  const int t64 = (T + 63) / 64;
  int splits = ctx->sm_count / out_tiles;
  if (splits < 1) splits = 1;
  if (splits > t64) splits = t64;
  const int chunk = ((t64 + splits - 1) / splits) * 64;
  splits = (t64 * 64 + chunk - 1) / chunk;
  if ((rc = map_mn(ctx, &tmA, dz16, Mp, T, BM / 64)) != UNIPOOL_OK) return rc;
  if ((rc = map_mn(ctx, &tmB, x, d, T, BN / 64)) != UNIPOOL_OK) return rc;
  if ((rc = map_chunk(ctx, &tmC, dW_r, d, M, kMapF32Chunk)) != UNIPOOL_OK) return rc;
  p.n_experts = splits; p.n_layers = 1; p.uniform_rows = t64 * 64;
  p.Mdim = M; p.Ndim = d; p.Kdim = chunk; p.overwrite = 0;
  return launch<kWgrad>(ctx, UNIPOOL_PH_ROUTE_BWD_DW, tmA, tmB, tmB, tmC, tmC, p, s);
}

}  // namespace unipool
