// Two-product variant of the GEMM main loop, for the full-distribution KL to a reference policy
// (section 2.2 / 3.1: Omega = beta * sum_t KL(pi_theta(.|s_t) || pi_ref(.|s_t))).
//
// For every 128x256 (per CTA) output tile it forms BOTH logit tiles the KL needs,
//     Z  = H  W^T      (policy,    K = d)      -> tensor-memory columns [0, 256)
//     Zr = Hr Wr^T     (reference, K = d_ref)  -> tensor-memory columns [256, 512)
// and hands the epilogue matching 32-column chunks of the two.  The two accumulators are both
// busy for the whole tile, so the epilogue of a tile and the MMAs of the next one do not overlap
// here (they do in the single-product engine); the warp roles, the operand ring, the CTA-pair
// protocol and the bounded waits are the same as there.  All four operands are K-major.
#pragma once
#include "gemm_engine.cuh"

namespace rlh {

// Epilogue contract: as in gemm_engine.cuh, except that chunk receives the policy chunk v and the
// reference chunk vr:  chunk(p, st, m_tile, n_tile, c, row_in_tile, m_rows, v, vr, tmC, staging).
template <class Epi, int CG>
__global__ void __launch_bounds__(kGemmThreads, 1)
dual_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2,
                 const __grid_constant__ CUtensorMap tmC, const GemmShape sh, const int k2_len,
                 const typename Epi::Params ep, DevStatus* status) {
  using Cfg = StageCfg<CG, Epi::kStagingBytes>;
  constexpr int kStages = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kMaxStages];
  __shared__ __align__(8) uint64_t bar_empty[kMaxStages];
  __shared__ __align__(8) uint64_t bar_acc_full;
  __shared__ __align__(8) uint64_t bar_acc_empty;
  __shared__ __align__(8) uint64_t bar_drain;
  __shared__ uint32_t tmem_base_smem;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t rank = CG == 2 ? cluster_ctarank() : 0u;
  const int worker = blockIdx.x / CG;
  const int n_workers = gridDim.x / CG;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
    mbar_init(smem_u32(&bar_acc_full), 1);
    mbar_init(smem_u32(&bar_acc_empty), 4 * CG);
    mbar_init(smem_u32(&bar_drain), 1);
    abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
    prefetch_tmap(&tmA2);
    prefetch_tmap(&tmB2);
  }
  if (warp == 1) {
    if (CG == 2) { tmem_alloc_pair(smem_u32(&tmem_base_smem), kTmemCols); tmem_relinquish_pair(); }
    else         { tmem_alloc(smem_u32(&tmem_base_smem), kTmemCols);      tmem_relinquish(); }
  }
  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_smem;
  volatile int* abort_p = &abort_flag;

  const GemmExtents ex = gemm_extents(sh, sh.n_valid ? *sh.n_valid : 0, CG, n_workers);
  const int k2_blocks = (k2_len + BK - 1) / BK;

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = worker; u < ex.n_units && ok; u += n_workers) {
        int mu, nr, ks, kb0, kb1;
        unit_coords(sh, ex, u, mu, nr, ks, kb0, kb1);
        const int m = mu * CG + (int)rank;
        const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
        const int a_row = sh.a_mn_off + (sh.a_mn_slab ? ex.slab_off : 0) + m * BM;
        for (int n = n0; n < n1 && ok; ++n) {
          const int b_row = sh.b_mn_off + n * BN + (int)rank * Cfg::kBRows;
          for (int prod = 0; prod < 2 && ok; ++prod) {
            const CUtensorMap* ta = prod ? &tmA2 : &tmA;
            const CUtensorMap* tb = prod ? &tmB2 : &tmB;
            const int nkb = prod ? k2_blocks : ex.k_blocks;
            for (int kb = 0; kb < nkb; ++kb) {
              if (!mbar_wait_bounded(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_p)) {
                latch_status(status, kStatusTimeout, (int)((9u << 28) | (blockIdx.x << 8) | (unsigned)stage));
                ok = false;
                break;
              }
              const uint32_t full_local = smem_u32(&bar_full[stage]);
              const uint32_t a_dst = tiles_base + stage * Cfg::kStageBytes;
              const uint32_t b_dst = a_dst + kAStageBytes;
              if (CG == 1) {
                mbar_arrive_expect_tx(full_local, Cfg::kTxBytes);
                tma_load_2d(a_dst, ta, full_local, kb * BK, a_row);
                tma_load_2d(b_dst, tb, full_local, kb * BK, b_row);
              } else {
                if (rank == 0) mbar_arrive_expect_tx(full_local, Cfg::kTxBytes);
                const uint32_t full = mapa_cluster(full_local, 0);
                tma_load_2d_pair(a_dst, ta, full, kb * BK, a_row);
                tma_load_2d_pair(b_dst, tb, full, kb * BK, b_row);
              }
              if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
          }
        }
      }
      if (!ok && (CG == 1 || rank == 0)) {
        for (int s = 0; s < kStages; ++s) {
          uint32_t p = (s < stage) ? phase : (phase ^ 1u);
          for (int it = 0; it < 4096 && !mbar_try_wait(smem_u32(&bar_full[s]), p); ++it) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer (even CTA of a pair)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(BM * CG, BN, 0, 0);
      constexpr uint64_t d_hi = make_smem_desc_hi(16, 1024);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t t = 0;
      bool ok = true;
      if (ex.k_blocks > 0 && k2_blocks > 0) {
        for (int u = worker; u < ex.n_units && ok; u += n_workers) {
          int mu, nr, ks, kb0, kb1;
          unit_coords(sh, ex, u, mu, nr, ks, kb0, kb1);
          const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
          for (int n = n0; n < n1 && ok; ++n, ++t) {
            if (!mbar_wait_bounded_cluster(smem_u32(&bar_acc_empty), (t & 1u) ^ 1u, abort_p)) {
              latch_status(status, kStatusTimeout, (int)((10u << 28) | (blockIdx.x << 8)));
              ok = false;
              break;
            }
            tc_fence_after();
            for (int prod = 0; prod < 2 && ok; ++prod) {
              const uint32_t d_tmem = tmem_base + prod * BN;
              const int nkb = prod ? k2_blocks : ex.k_blocks;
              for (int kb = 0; kb < nkb; ++kb) {
                if (!mbar_wait_bounded_cluster(smem_u32(&bar_full[stage]), phase, abort_p)) {
                  latch_status(status, kStatusTimeout, (int)((11u << 28) | (blockIdx.x << 8) | (unsigned)stage));
                  ok = false;
                  break;
                }
                tc_fence_after();
                const uint32_t a_src = tiles_base + stage * Cfg::kStageBytes;
                const uint32_t b_src = a_src + kAStageBytes;
#pragma unroll
                for (int k = 0; k < BK / 16; ++k) {
                  const uint64_t da = smem_desc(d_hi, a_src + k * 32), db = smem_desc(d_hi, b_src + k * 32);
                  if (CG == 2) umma_bf16_pair(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
                  else         umma_bf16(d_tmem, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
                }
                if (CG == 2) umma_commit_pair_mcast(smem_u32(&bar_empty[stage]), 3);
                else         umma_commit(smem_u32(&bar_empty[stage]));
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
              }
            }
            if (ok) {
              if (CG == 2) umma_commit_pair_mcast(smem_u32(&bar_acc_full), 3);
              else         umma_commit(smem_u32(&bar_acc_full));
            }
          }
        }
      }
      if (CG == 2) umma_commit_pair(smem_u32(&bar_drain));
      else         umma_commit(smem_u32(&bar_drain));
      bool drained = false;
      for (int it = 0; it < (1 << 22) && !drained; ++it) drained = mbar_try_wait(smem_u32(&bar_drain), 0) != 0;
      if (!drained) latch_status(status, kStatusTimeout, (int)((12u << 28) | (blockIdx.x << 8)));
    }
  } else {
    // ------------------------------------------------------------- epilogue warps (both CTAs)
    const int q = warp & 3;
    const int row_in_tile = q * 32 + lane;
    const uint32_t staging = tiles_base + Cfg::kRingBytes + q * kStagingPerWarp;
    typename Epi::State st;
    Epi::init(st);
    uint32_t t = 0;
    bool ok = true;
    const bool has_k = ex.k_blocks > 0 && k2_blocks > 0;
    for (int u = worker; u < ex.n_units && ok && has_k; u += n_workers) {
      int mu, nr, ks, kb0, kb1;
      unit_coords(sh, ex, u, mu, nr, ks, kb0, kb1);
      const int m = mu * CG + (int)rank;
      const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
      Epi::begin_unit(ep, st, m, nr, row_in_tile, ex.m_rows, ex.slab_off, ks);
      for (int n = n0; n < n1 && ok; ++n, ++t) {
        if (!mbar_wait_bounded_cluster(smem_u32(&bar_acc_full), t & 1u, abort_p)) {
          latch_status(status, kStatusTimeout, (int)((13u << 28) | (blockIdx.x << 8)));
          ok = false;
        }
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + (uint32_t(q * 32) << 16);
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32], rr[32];
          tmem_ld_32x32(taddr + c * 32, r);
          tmem_ld_32x32(taddr + BN + c * 32, rr);
          tmem_ld_wait();
          float v[32], vr[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) { v[i] = __uint_as_float(r[i]); vr[i] = __uint_as_float(rr[i]); }
          Epi::chunk(ep, st, m, n, c, row_in_tile, ex.m_rows, v, vr, &tmC, staging);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (CG == 2 && rank != 0) mbar_arrive_cluster(mapa_cluster(smem_u32(&bar_acc_empty), 0));
          else                      mbar_arrive(smem_u32(&bar_acc_empty));
        }
      }
      if (ok) Epi::end_unit(ep, st, m, nr, row_in_tile, ex.m_rows);
    }
    Epi::finish(st);
  }

  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (CG == 2) tmem_dealloc_pair(tmem_base, kTmemCols);
    else         tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace rlh
