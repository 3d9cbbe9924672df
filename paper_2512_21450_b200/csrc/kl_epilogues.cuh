// Epilogues of the two-product tile mode of the GEMM engine: full-distribution KL(pi_theta || pi_ref) per token
// (section 2.2 "KL-to-reference", section 3.1 Omega) and its gradient with respect to the logits.
#pragma once
#include "epilogues.cuh"

namespace rlh {

// ---------------------------------------------------------------------------------------------
// Forward: the statistics of EpiStats for the policy logits z, plus
//   D  = sum_j exp(z_j - M) zr_j          (so that sum_j p_j (z_j - zr_j) = (A - D) / S)
//   Mr, Sr = running max and sum exp(zr - Mr) of the reference logits (for lse_ref).
// Two float4 per (range, row): {M, S, A, z_y} and {D, Mr, Sr, 0}.
struct EpiStatsKL {
  static constexpr int kStagingBytes = 0;
  struct Params {
    const int* tokens_c;
    float4* partials;
    float4* partials2;
    int part_stride;
    int V;
  };
  struct State {
    float m, s, a, zy, dsum, mr, sr;
    int y;
  };
  __device__ static __forceinline__ void init(State&) {}
  __device__ static __forceinline__ void finish(State&) {}
  __device__ static __forceinline__ void begin_unit(const Params& p, State& st, int m_tile, int, int row_in_tile,
                                                    int m_rows, int, int) {
    st.m = -CUDART_INF_F; st.s = 0.f; st.a = 0.f; st.zy = 0.f; st.dsum = 0.f;
    st.mr = -CUDART_INF_F; st.sr = 0.f;
    const int row = m_tile * BM + row_in_tile;
    st.y = row < m_rows ? p.tokens_c[row] : -1;
  }
  __device__ static __forceinline__ void chunk(const Params& p, State& st, int, int n_tile, int c, int, int,
                                               const float (&v)[32], const float (&vr)[32], const CUtensorMap*,
                                               uint32_t) {
    const int col0 = n_tile * BN + c * 32;
    const int nvalid = p.V - col0;
    if (nvalid <= 0) return;
    float cmax = -CUDART_INF_F, rmax = -CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      cmax = i < nvalid ? fmaxf(cmax, v[i]) : cmax;
      rmax = i < nvalid ? fmaxf(rmax, vr[i]) : rmax;
    }
    const float newm = fmaxf(st.m, cmax), newr = fmaxf(st.mr, rmax);
    const float scale = ex2_approx((st.m - newm) * kLog2e), scale_r = ex2_approx((st.mr - newr) * kLog2e);
    const float mL = newm * kLog2e, rL = newr * kLog2e;
    float cs = 0.f, ca = 0.f, cd = 0.f, csr = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const float e = i < nvalid ? ex2_approx(fmaf(v[i], kLog2e, -mL)) : 0.f;
      const float er = i < nvalid ? ex2_approx(fmaf(vr[i], kLog2e, -rL)) : 0.f;
      cs += e;
      ca = fmaf(e, v[i], ca);
      cd = fmaf(e, vr[i], cd);
      csr += er;
    }
    st.s = fmaf(st.s, scale, cs);
    st.a = fmaf(st.a, scale, ca);
    st.dsum = fmaf(st.dsum, scale, cd);
    st.m = newm;
    st.sr = fmaf(st.sr, scale_r, csr);
    st.mr = newr;
    const unsigned rel = (unsigned)(st.y - col0);
    if (rel < 32u && (int)rel < nvalid) {
      float z = 0.f;
#pragma unroll
      for (int i = 0; i < 32; ++i) z = (rel == (unsigned)i) ? v[i] : z;
      st.zy = z;
    }
  }
  __device__ static __forceinline__ void end_unit(const Params& p, State& st, int m_tile, int nr, int row_in_tile,
                                                  int m_rows) {
    const int row = m_tile * BM + row_in_tile;
    if (row < m_rows) {
      p.partials[(size_t)nr * p.part_stride + row] = make_float4(st.m, st.s, st.a, st.zy);
      p.partials2[(size_t)nr * p.part_stride + row] = make_float4(st.dsum, st.mr, st.sr, 0.f);
    }
  }
};

// ---------------------------------------------------------------------------------------------
// Backward: g_tj = cp_t (p_tj - 1[j = y_t]) + cb_t p_tj (log p_tj - log q_tj - KL_t)
//                  + ce_t p_tj (log p_tj + Ent_t),   cb_t = w_t beta,
// written to the bf16 slab exactly as EpiGrad does (swizzled staging + TMA bulk stores).
struct EpiGradKL {
  static constexpr int kStagingBytes = 4 * kStagingPerWarp;
  struct Params {
    const int* tokens_c;
    const float* lse;
    const float* lse_ref;
    const float* ent;
    const float* kl;
    const float* cp;
    const float* cb;
    const float* ce;
    int V;
    int vocab_base;
  };
  struct State {
    float lse, lse_ref, ent, kl, cp, cb, ce;
    int y;
    bool valid;
    uint32_t n_issued;
  };
  __device__ static __forceinline__ void init(State& st) { st.n_issued = 0; }
  __device__ static __forceinline__ void finish(State& st) {
    if ((threadIdx.x & 31) == 0 && st.n_issued) bulk_wait_group_all();
    __syncwarp();
  }
  __device__ static __forceinline__ void begin_unit(const Params& p, State& st, int m_tile, int, int row_in_tile,
                                                    int m_rows, int slab_off, int) {
    const int rl = m_tile * BM + row_in_tile;
    st.valid = rl < m_rows;
    const int gr = slab_off + rl;
    st.lse = st.valid ? p.lse[gr] : 0.f;
    st.lse_ref = st.valid ? p.lse_ref[gr] : 0.f;
    st.ent = st.valid ? p.ent[gr] : 0.f;
    st.kl = st.valid ? p.kl[gr] : 0.f;
    st.cp = st.valid ? p.cp[gr] : 0.f;
    st.cb = st.valid ? p.cb[gr] : 0.f;
    st.ce = st.valid ? p.ce[gr] : 0.f;
    st.y = st.valid ? p.tokens_c[gr] : -1;
  }
  __device__ static __forceinline__ void chunk(const Params& p, State& st, int m_tile, int n_tile, int c,
                                               int row_in_tile, int m_rows, const float (&v)[32],
                                               const float (&vr)[32], const CUtensorMap* tmG, uint32_t staging) {
    if (m_tile * BM >= ((m_rows + BM - 1) / BM) * BM) return;
    const int col_l = n_tile * BN + c * 32;
    const int col_g = p.vocab_base + col_l;
    const int nvalid = p.V - col_g;
    float g[32];
    if (!st.valid || nvalid <= 0) {
#pragma unroll
      for (int i = 0; i < 32; ++i) g[i] = 0.f;
    } else {
      const float base = st.cp + st.ce * st.ent - st.cb * st.kl;   // terms that do not depend on j
      const float k_lp = st.cb + st.ce;                              // coefficient of log p_j
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float lp = v[i] - st.lse;
        const float lq = vr[i] - st.lse_ref;
        g[i] = ex2_approx(lp * kLog2e) * (fmaf(k_lp, lp, base) - st.cb * lq);
      }
      const unsigned rel = (unsigned)(st.y - col_g);
      if (rel < 32u) {
#pragma unroll
        for (int i = 0; i < 32; ++i) g[i] = (rel == (unsigned)i) ? g[i] - st.cp : g[i];
      }
      if (nvalid < 32) {
#pragma unroll
        for (int i = 0; i < 32; ++i) g[i] = i < nvalid ? g[i] : 0.f;
      }
    }
    const int lane = threadIdx.x & 31;
    const uint32_t buf = staging + (st.n_issued & 1u) * 4096u;
    if ((c & 1) == 0) {
      if (lane == 0) bulk_wait_group_read<1>();
      __syncwarp();
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      __nv_bfloat162 b0 = __floats2bfloat162_rn(g[8 * j + 0], g[8 * j + 1]);
      __nv_bfloat162 b1 = __floats2bfloat162_rn(g[8 * j + 2], g[8 * j + 3]);
      __nv_bfloat162 b2 = __floats2bfloat162_rn(g[8 * j + 4], g[8 * j + 5]);
      __nv_bfloat162 b3 = __floats2bfloat162_rn(g[8 * j + 6], g[8 * j + 7]);
      const uint32_t jj = uint32_t(4 * (c & 1) + j);
      const uint32_t addr = buf + lane * 128u + ((jj ^ uint32_t(lane & 7)) << 4);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(*reinterpret_cast<uint32_t*>(&b0)),
                   "r"(*reinterpret_cast<uint32_t*>(&b1)), "r"(*reinterpret_cast<uint32_t*>(&b2)),
                   "r"(*reinterpret_cast<uint32_t*>(&b3))
                   : "memory");
    }
    if (c & 1) {
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        tma_store_2d(tmG, buf, col_l - 32, m_tile * BM + (row_in_tile - lane));
        bulk_commit_group();
      }
      st.n_issued++;
    }
  }
  __device__ static __forceinline__ void end_unit(const Params&, State&, int, int, int, int) {}
};

}  // namespace rlh
