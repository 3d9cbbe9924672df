// Persistent, warp-specialised bf16 GEMM main loop for sm_100a with pluggable epilogues.
//
//   warp 0      : TMA producer (one lane) - streams 128x64 A tiles and 256x64 B tiles into a
//                 4-stage shared-memory ring, 128-byte swizzled.
//   warp 1      : allocates tensor memory; one lane issues tcgen05.mma (128x256x16 per
//                 instruction) into one of two 256-column fp32 accumulators.
//   warps 2..5  : epilogue - each warp owns the 32 tensor-memory lanes (tile rows) that its
//                 rank modulo 4 may read, pulls the accumulator out in 32-column chunks and
//                 hands them to the epilogue functor.  While they drain accumulator a, the MMA
//                 warp already fills accumulator a^1.
//
// Either operand may be K-major (its global tensor is [rows, K], K contiguous) or MN-major
// (its global tensor is [K, rows], rows contiguous).  A K-major tile is one 2-D TMA box
// {64 k, rows}; an MN-major tile is one 3-D box {64 rows, 64 k, rows/64}, which lands in shared
// memory as rows/64 chunks of 8 KB, each chunk 64 k-lines of 128 bytes.
//
// Every wait is bounded: when one runs out the block raises a shared abort flag, every role
// leaves its loop, the status word is latched and the block still frees its tensor memory.
#pragma once
#include <cuda.h>

#include "ptx.cuh"

namespace rlh {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 64;
constexpr int kStages = 4;
constexpr int kAStageBytes = BM * BK * 2;
constexpr int kBStageBytes = BN * BK * 2;
constexpr int kStageBytes = kAStageBytes + kBStageBytes;
constexpr int kGemmThreads = 192;
constexpr int kGemmSmemBytes = kStages * kStageBytes + 1024;  // + slack for 1024-byte alignment
constexpr int kTmemCols = 512;
constexpr int kMaxSplit = 16;

// Device status word shared by all kernels of a context.
struct DevStatus {
  int code;    // rl_status value, 0 = ok (first error wins)
  int detail;  // where it happened
  int n_valid; // number of rows with mask != 0, written by the mask scan
  int pad;
};
constexpr int kStatusTokenRange = 7;
constexpr int kStatusTimeout = 8;

__device__ __forceinline__ void latch_status(DevStatus* st, int code, int detail) {
  if (atomicCAS(&st->code, 0, code) == 0) st->detail = detail;
}

struct GemmShape {
  // Extent of the M dimension: m_rows_cap, or when m_dyn != 0 the part of it that is covered by
  // valid rows: clamp(*n_valid - m_dyn_off, 0, m_rows_cap).  Same for K with the k_* fields.
  const int* n_valid;
  int m_rows_cap, m_dyn, m_dyn_off;
  int k_cap, k_dyn, k_dyn_off;
  int n_tiles;      // number of 256-wide column tiles
  int n_range;      // consecutive column tiles per work unit; 0 = choose so that units fill the SMs
  int skip_if_k0;   // nothing to do at all when K is empty (otherwise the epilogue sees zeros)
  // coordinate offsets into the operands' global tensors
  int a_mn_off, a_k_off, b_mn_off, b_k_off;
};

// Number of vocabulary ranges each 128-row tile is split into so that (row tiles x ranges) fills
// the machine: minimises waves * tiles-per-range, preferring fewer ranges on ties.
__host__ __device__ inline int choose_split(int m_tiles, int n_tiles, int n_ctas) {
  int best = 1;
  long best_cost = -1;
  for (int s = 1; s <= kMaxSplit && s <= n_tiles; ++s) {
    long units = (long)m_tiles * s;
    long waves = (units + n_ctas - 1) / n_ctas;
    long cost = waves * ((n_tiles + s - 1) / s);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
  }
  return best;
}

struct GemmExtents {
  int m_rows, m_tiles, k_blocks, n_range, n_ranges, n_units;
};

__device__ __forceinline__ GemmExtents gemm_extents(const GemmShape& sh) {
  GemmExtents e;
  int nv = sh.n_valid ? *sh.n_valid : 0;
  e.m_rows = sh.m_dyn ? min(max(nv - sh.m_dyn_off, 0), sh.m_rows_cap) : sh.m_rows_cap;
  int k_len = sh.k_dyn ? min(max(nv - sh.k_dyn_off, 0), sh.k_cap) : sh.k_cap;
  e.m_tiles = (e.m_rows + BM - 1) / BM;
  e.k_blocks = (k_len + BK - 1) / BK;
  int split = sh.n_range > 0 ? 0 : choose_split(e.m_tiles, sh.n_tiles, (int)gridDim.x);
  e.n_range = sh.n_range > 0 ? sh.n_range : (sh.n_tiles + split - 1) / max(split, 1);
  e.n_range = max(e.n_range, 1);
  e.n_ranges = (sh.n_tiles + e.n_range - 1) / e.n_range;
  e.n_units = e.m_tiles * e.n_ranges;
  if (sh.skip_if_k0 && e.k_blocks == 0) e.n_units = 0;
  return e;
}

// Epilogue functor contract (all methods run in the 128 epilogue threads, one tile row each):
//   struct Epi { struct Params; struct State;
//     static void begin_unit(const Params&, State&, int m_tile, int n_range_idx, int row_in_tile, int m_rows);
//     static void chunk(const Params&, State&, int m_tile, int n_tile, int chunk, int row_in_tile, int m_rows, const float (&v)[32]);
//     static void end_unit(const Params&, State&, int m_tile, int n_range_idx, int row_in_tile, int m_rows); };
template <class Epi, int A_MN, int B_MN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const GemmShape sh, const typename Epi::Params ep, DevStatus* status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kStages];
  __shared__ __align__(8) uint64_t bar_empty[kStages];
  __shared__ __align__(8) uint64_t bar_acc_full[2];
  __shared__ __align__(8) uint64_t bar_acc_empty[2];
  __shared__ __align__(8) uint64_t bar_drain;
  __shared__ uint32_t tmem_base_smem;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(smem_u32(&bar_acc_full[a]), 1); mbar_init(smem_u32(&bar_acc_empty[a]), 4); }
    mbar_init(smem_u32(&bar_drain), 1);
    abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_smem), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_smem;
  volatile int* abort_p = &abort_flag;

  const GemmExtents ex = gemm_extents(sh);

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < ex.n_units && ok; u += gridDim.x) {
        const int m = u % ex.m_tiles, nr = u / ex.m_tiles;
        const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
        for (int n = n0; n < n1 && ok; ++n) {
          for (int kb = 0; kb < ex.k_blocks; ++kb) {
            if (!mbar_wait_bounded(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_p)) {
              latch_status(status, kStatusTimeout, (1 << 28) | (blockIdx.x << 8) | stage);
              ok = false;
              break;
            }
            const uint32_t full = smem_u32(&bar_full[stage]);
            const uint32_t a_dst = tiles_base + stage * kAStageBytes;
            const uint32_t b_dst = tiles_base + kStages * kAStageBytes + stage * kBStageBytes;
            mbar_arrive_expect_tx(full, kStageBytes);
            if (A_MN) tma_load_3d(a_dst, &tmA, full, 0, sh.a_k_off + kb * BK, (sh.a_mn_off + m * BM) / 64);
            else      tma_load_2d(a_dst, &tmA, full, sh.a_k_off + kb * BK, sh.a_mn_off + m * BM);
            if (B_MN) tma_load_3d(b_dst, &tmB, full, 0, sh.b_k_off + kb * BK, (sh.b_mn_off + n * BN) / 64);
            else      tma_load_2d(b_dst, &tmB, full, sh.b_k_off + kb * BK, sh.b_mn_off + n * BN);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok) {
        // let copies that were already issued land before the block's shared memory goes away
        for (int s = 0; s < kStages; ++s) {
          uint32_t p = (s < stage) ? phase : (phase ^ 1u);
          for (int it = 0; it < 4096 && !mbar_try_wait(smem_u32(&bar_full[s]), p); ++it) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(BM, BN, A_MN, B_MN);
      // K-major: 8-row groups 1024 B apart, 32 bytes per 16-element k step.
      // MN-major: 64-row chunks 8192 B apart, 8-k-line groups 1024 B apart, 2048 B per k step.
      constexpr uint64_t a_hi = A_MN ? make_smem_desc_hi(8192, 1024) : make_smem_desc_hi(16, 1024);
      constexpr uint64_t b_hi = B_MN ? make_smem_desc_hi(8192, 1024) : make_smem_desc_hi(16, 1024);
      constexpr uint32_t a_kstep = A_MN ? 2048 : 32;
      constexpr uint32_t b_kstep = B_MN ? 2048 : 32;
      int stage = 0;
      uint32_t phase = 0;
      uint32_t t = 0;
      bool ok = true;
      if (ex.k_blocks > 0) {
        for (int u = blockIdx.x; u < ex.n_units && ok; u += gridDim.x) {
          const int nr = u / ex.m_tiles;
          const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
          for (int n = n0; n < n1 && ok; ++n, ++t) {
            const uint32_t a = t & 1u, round = t >> 1;
            if (!mbar_wait_bounded(smem_u32(&bar_acc_empty[a]), (round & 1u) ^ 1u, abort_p)) {
              latch_status(status, kStatusTimeout, (2 << 28) | (blockIdx.x << 8) | a);
              ok = false;
              break;
            }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + a * BN;
            for (int kb = 0; kb < ex.k_blocks; ++kb) {
              if (!mbar_wait_bounded(smem_u32(&bar_full[stage]), phase, abort_p)) {
                latch_status(status, kStatusTimeout, (3 << 28) | (blockIdx.x << 8) | stage);
                ok = false;
                break;
              }
              tc_fence_after();
              const uint32_t a_src = tiles_base + stage * kAStageBytes;
              const uint32_t b_src = tiles_base + kStages * kAStageBytes + stage * kBStageBytes;
#pragma unroll
              for (int k = 0; k < BK / 16; ++k) {
                umma_bf16(d_tmem, smem_desc(a_hi, a_src + k * a_kstep), smem_desc(b_hi, b_src + k * b_kstep),
                          idesc, (kb | k) != 0 ? 1u : 0u);
              }
              umma_commit(smem_u32(&bar_empty[stage]));
              if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
            if (ok) umma_commit(smem_u32(&bar_acc_full[a]));
          }
        }
      }
      // every UMMA issued above has to retire before tensor memory is released
      umma_commit(smem_u32(&bar_drain));
      bool drained = false;
      for (int it = 0; it < (1 << 22) && !drained; ++it) drained = mbar_try_wait(smem_u32(&bar_drain), 0) != 0;
      if (!drained) latch_status(status, kStatusTimeout, (4 << 28) | (blockIdx.x << 8));
    }
  } else {
    // ------------------------------------------------------------- epilogue warps
    const int q = warp & 3;
    const int row_in_tile = q * 32 + lane;
    typename Epi::State st;
    uint32_t t = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < ex.n_units && ok; u += gridDim.x) {
      const int m = u % ex.m_tiles, nr = u / ex.m_tiles;
      const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
      Epi::begin_unit(ep, st, m, nr, row_in_tile, ex.m_rows);
      for (int n = n0; n < n1 && ok; ++n, ++t) {
        const uint32_t a = t & 1u, round = t >> 1;
        if (ex.k_blocks > 0) {
          if (!mbar_wait_bounded(smem_u32(&bar_acc_full[a]), round & 1u, abort_p)) {
            latch_status(status, kStatusTimeout, (5 << 28) | (blockIdx.x << 8) | a);
            ok = false;
          }
          ok = __all_sync(0xffffffffu, ok);   // tensor-memory loads below need the whole warp
          if (!ok) break;
          tc_fence_after();
        }
        const uint32_t taddr = tmem_base + a * BN + (uint32_t(q * 32) << 16);
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          float v[32];
          if (ex.k_blocks > 0) {
            uint32_t r[32];
            tmem_ld_32x32(taddr + c * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0.f;
          }
          Epi::chunk(ep, st, m, n, c, row_in_tile, ex.m_rows, v);
        }
        if (ex.k_blocks > 0) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[a]));
        }
      }
      if (ok) Epi::end_unit(ep, st, m, nr, row_in_tile, ex.m_rows);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace rlh
