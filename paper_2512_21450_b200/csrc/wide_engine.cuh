// Wide-tile variant of the GEMM main loop for the long-K gradient products (dH = G W, dW = G^T H).
//
// A CTA pair works on a 256 x 512 output tile: both 256-column accumulators of tensor memory hold
// one tile, so every k-slice of A (16 KB per CTA) is used for twice as many flops as in the
// 256 x 256 engine and the operand bytes a CTA has to pull from L2 per flop drop by a quarter
// (48 KB instead of 64 KB per 2 x 128 x 256 x 64 multiply-adds).  The price is that the epilogue of
// a tile cannot overlap the main loop of the next one; with K of 17-19 thousand the epilogue is
// about 1 % of a tile.
//
// Per stage a CTA holds A (128 rows x 64 k) and two B boxes (128 output columns x 64 k each): box s
// (s = 0, 1) carries columns [512 n + 256 s + 128 rank, +128) of the tile, so that the M = 256,
// N = 256 UMMA number s reads its 256 columns half from each CTA of the pair exactly as in the
// 256 x 256 engine, and writes accumulator s (tensor-memory columns [256 s, 256 s + 256)).  Four
// stages of 48 KB.  Roles, barriers, bounded waits and the epilogue functor contract are those of
// gemm_kernel with CG = 2; the epilogue sees the two halves as column tiles 2 n and 2 n + 1.
// K slices and stream-K are not supported here (the launch code does not ask for them).
#pragma once
#include "gemm_engine.cuh"

namespace rlh {

constexpr int kWideBBoxBytes = (BN / 2) * BK * 2;                      // one B box of a CTA: 16 KB
constexpr int kWideStageBytes = kAStageBytes + 2 * kWideBBoxBytes;     // 48 KB

template <class Epi, int A_MN, int B_MN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_wide_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmC, const GemmShape sh, const typename Epi::Params ep,
                 DevStatus* status) {
  constexpr int kStages = (kTileSmemBytes - Epi::kStagingBytes) / kWideStageBytes;   // 4
  constexpr int kRingBytes = kStages * kWideStageBytes;
  constexpr uint32_t kTxBytes = uint32_t(kWideStageBytes) * 2;   // both CTAs' copies land on the even CTA's barrier
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kStages];
  __shared__ __align__(8) uint64_t bar_empty[kStages];
  __shared__ __align__(8) uint64_t bar_acc_full;
  __shared__ __align__(8) uint64_t bar_acc_empty[2];
  __shared__ __align__(8) uint64_t bar_drain;
  __shared__ uint32_t tmem_base_smem;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t rank = cluster_ctarank();
  const int worker = blockIdx.x / 2;
  const int n_workers = gridDim.x / 2;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
    mbar_init(smem_u32(&bar_acc_full), 1);
    for (int a = 0; a < 2; ++a) mbar_init(smem_u32(&bar_acc_empty[a]), 8);   // 4 epilogue warps in each CTA
    mbar_init(smem_u32(&bar_drain), 1);
    abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) { tmem_alloc_pair(smem_u32(&tmem_base_smem), kTmemCols); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_smem;
  volatile int* abort_p = &abort_flag;

  // sh.n_tiles counts 512-wide column tiles here
  const GemmExtents ex = gemm_extents(sh, sh.n_valid ? *sh.n_valid : 0, 2, n_workers);

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = worker; u < ex.n_units && ok; u += n_workers) {
        int mu, nr, ks, kb0, kb1;
        unit_coords(sh, ex, u, mu, nr, ks, kb0, kb1);
        const int m = mu * 2 + (int)rank;
        const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
        const int a_row = sh.a_mn_off + (sh.a_mn_slab ? ex.slab_off : 0) + m * BM;
        for (int n = n0; n < n1 && ok; ++n) {
          for (int kb = kb0; kb < kb1; ++kb) {
            if (!mbar_wait_bounded(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_p)) {
              latch_status(status, kStatusTimeout, (int)((10u << 28) | (blockIdx.x << 8) | (unsigned)stage));
              ok = false;
              break;
            }
            const uint32_t full_local = smem_u32(&bar_full[stage]);
            const uint32_t a_dst = tiles_base + stage * kWideStageBytes;
            const uint32_t b_dst = a_dst + kAStageBytes;
            const int b_k = sh.b_k_off + (sh.b_k_slab ? ex.slab_off : 0) + kb * BK;
            if (rank == 0) mbar_arrive_expect_tx(full_local, kTxBytes);
            const uint32_t full = mapa_cluster(full_local, 0);
            if (A_MN) tma_load_3d_pair(a_dst, &tmA, full, 0, sh.a_k_off + kb * BK, a_row / 64);
            else      tma_load_2d_pair(a_dst, &tmA, full, sh.a_k_off + kb * BK, a_row);
#pragma unroll
            for (int s = 0; s < 2; ++s) {
              const int b_row = sh.b_mn_off + n * (2 * BN) + s * BN + (int)rank * (BN / 2);
              if (B_MN) tma_load_3d_pair(b_dst + s * kWideBBoxBytes, &tmB, full, 0, b_k, b_row / 64);
              else      tma_load_2d_pair(b_dst + s * kWideBBoxBytes, &tmB, full, b_k, b_row);
            }
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok && rank == 0) {
        // let copies that were already issued land before the block's shared memory goes away
        for (int s = 0; s < kStages; ++s) {
          uint32_t p = (s < stage) ? phase : (phase ^ 1u);
          for (int it = 0; it < 4096 && !mbar_try_wait(smem_u32(&bar_full[s]), p); ++it) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer (even CTA of the pair)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(BM * 2, BN, A_MN, B_MN);
      constexpr uint64_t a_hi = A_MN ? make_smem_desc_hi(8192, 1024) : make_smem_desc_hi(16, 1024);
      constexpr uint64_t b_hi = B_MN ? make_smem_desc_hi(8192, 1024) : make_smem_desc_hi(16, 1024);
      constexpr uint32_t a_kstep = A_MN ? 2048 : 32;
      constexpr uint32_t b_kstep = B_MN ? 2048 : 32;
      int stage = 0;
      uint32_t phase = 0;
      uint32_t t = 0;   // wide tiles issued so far
      bool ok = true;
      if (ex.k_blocks > 0) {
        for (int u = worker; u < ex.n_units && ok; u += n_workers) {
          int mu, nr, ks, kb0, kb1;
          unit_coords(sh, ex, u, mu, nr, ks, kb0, kb1);
          if (kb1 <= kb0) continue;
          const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
          for (int n = n0; n < n1 && ok; ++n, ++t) {
            // both accumulators must have been drained by the epilogues of the previous tile
            for (int a = 0; a < 2 && ok; ++a) {
              if (!mbar_wait_bounded_cluster(smem_u32(&bar_acc_empty[a]), (t & 1u) ^ 1u, abort_p)) {
                latch_status(status, kStatusTimeout, (int)((11u << 28) | (blockIdx.x << 8) | (unsigned)a));
                ok = false;
              }
            }
            if (!ok) break;
            tc_fence_after();
            for (int kb = kb0; kb < kb1; ++kb) {
              if (!mbar_wait_bounded_cluster(smem_u32(&bar_full[stage]), phase, abort_p)) {
                latch_status(status, kStatusTimeout, (int)((12u << 28) | (blockIdx.x << 8) | (unsigned)stage));
                ok = false;
                break;
              }
              tc_fence_after();
              const uint32_t a_src = tiles_base + stage * kWideStageBytes;
              const uint32_t b_src = a_src + kAStageBytes;
#pragma unroll
              for (int k = 0; k < BK / 16; ++k) {
                const uint64_t da = smem_desc(a_hi, a_src + k * a_kstep);
                const uint32_t acc = (kb > kb0 || k > 0) ? 1u : 0u;
                umma_bf16_pair(tmem_base, da, smem_desc(b_hi, b_src + k * b_kstep), idesc, acc);
                umma_bf16_pair(tmem_base + BN, da, smem_desc(b_hi, b_src + kWideBBoxBytes + k * b_kstep), idesc, acc);
              }
              umma_commit_pair_mcast(smem_u32(&bar_empty[stage]), 3);
              if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
            if (ok) umma_commit_pair_mcast(smem_u32(&bar_acc_full), 3);
          }
        }
      }
      // every UMMA issued above has to retire before tensor memory is released
      umma_commit_pair(smem_u32(&bar_drain));
      bool drained = false;
      for (int it = 0; it < (1 << 22) && !drained; ++it) drained = mbar_try_wait(smem_u32(&bar_drain), 0) != 0;
      if (!drained) latch_status(status, kStatusTimeout, (int)((13u << 28) | (blockIdx.x << 8)));
    }
  } else {
    // ------------------------------------------------------------- epilogue warps (both CTAs)
    const int q = warp & 3;
    const int row_in_tile = q * 32 + lane;
    const uint32_t staging = tiles_base + kRingBytes + q * kStagingPerWarp;
    typename Epi::State st;
    Epi::init(st);
    uint32_t t = 0;
    bool ok = true;
    for (int u = worker; u < ex.n_units && ok; u += n_workers) {
      int mu, nr, ks, kb0, kb1;
      unit_coords(sh, ex, u, mu, nr, ks, kb0, kb1);
      const bool has_k = kb1 > kb0;   // an empty K range contributes zeros
      const int m = mu * 2 + (int)rank;
      const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
      Epi::begin_unit(ep, st, m, nr, row_in_tile, ex.m_rows, ex.slab_off, ks);
      for (int n = n0; n < n1 && ok; ++n, t += has_k ? 1u : 0u) {
        if (has_k) {
          if (!mbar_wait_bounded_cluster(smem_u32(&bar_acc_full), t & 1u, abort_p)) {
            latch_status(status, kStatusTimeout, (int)((14u << 28) | (blockIdx.x << 8)));
            ok = false;
          }
          ok = __all_sync(0xffffffffu, ok);   // tensor-memory loads below need the whole warp
          if (!ok) break;
          tc_fence_after();
        }
        for (int s = 0; s < 2; ++s) {
          const uint32_t taddr = tmem_base + s * BN + (uint32_t(q * 32) << 16);
#pragma unroll 1
          for (int c = 0; c < BN / 32; ++c) {
            float v[32];
            if (has_k) {
              uint32_t r[32];
              tmem_ld_32x32(taddr + c * 32, r);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = 0.f;
            }
            Epi::chunk(ep, st, m, 2 * n + s, c, row_in_tile, ex.m_rows, v, &tmC, staging);
          }
          if (has_k) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
              if (rank != 0) mbar_arrive_cluster(mapa_cluster(smem_u32(&bar_acc_empty[s]), 0));
              else           mbar_arrive(smem_u32(&bar_acc_empty[s]));
            }
          }
        }
      }
      if (ok) Epi::end_unit(ep, st, m, nr, row_in_tile, ex.m_rows);
    }
    Epi::finish(st);
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // the pair's UMMAs have retired and both epilogues are done
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

}  // namespace rlh
