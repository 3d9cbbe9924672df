// Epilogue functors of the GEMM engine.  Each of the 128 epilogue threads owns one row of the
// 128x256 accumulator tile and receives it in chunks of 32 consecutive columns.
#pragma once
#include <math_constants.h>

#include "gemm_engine.cuh"

namespace rlh {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// One MUFU instruction: 2^x, denormal results flushed to zero (arguments here are <= 0 up to
// rounding, results in [0, 1]); -inf gives 0.
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---------------------------------------------------------------------------------------------
// Forward statistics (policy over the vocabulary, section 2.2): for its row and the vocabulary
// range of the work unit, keeps the running maximum M, S = sum exp(z-M), A = sum exp(z-M) z and
// the logit of the sampled token.  Logits never leave the chip; one float4 per (range, row) does.
struct EpiStats {
  static constexpr int kStagingBytes = 0;
  struct Params {
    const int* tokens_c;   // [rows] compact sampled-token ids
    float4* partials;      // [n_ranges][part_stride]
    int part_stride;
    int V;
  };
  struct State {
    float m, s, a, zy;
    int y;
  };
  __device__ static __forceinline__ void begin_unit(const Params& p, State& st, int m_tile, int, int row_in_tile,
                                                    int m_rows, int, int) {
    st.m = -CUDART_INF_F;
    st.s = 0.f;
    st.a = 0.f;
    st.zy = 0.f;
    const int row = m_tile * BM + row_in_tile;
    st.y = row < m_rows ? p.tokens_c[row] : -1;
  }
  __device__ static __forceinline__ void init(State&) {}
  __device__ static __forceinline__ void finish(State&) {}
  __device__ static __forceinline__ void chunk(const Params& p, State& st, int, int n_tile, int c, int, int,
                                               const float (&v)[32], const CUtensorMap*, uint32_t) {
    const int col0 = n_tile * BN + c * 32;
    const int nvalid = p.V - col0;
    if (nvalid <= 0) return;
    float cmax = -CUDART_INF_F;
    if (nvalid >= 32) {
#pragma unroll
      for (int i = 0; i < 32; i += 2) cmax = fmaxf(cmax, fmaxf(v[i], v[i + 1]));
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) cmax = i < nvalid ? fmaxf(cmax, v[i]) : cmax;
    }
    const float newm = fmaxf(st.m, cmax);
    const float scale = ex2_approx((st.m - newm) * kLog2e);
    const float mL = newm * kLog2e;
    float cs = 0.f, ca = 0.f;
    if (nvalid >= 32) {
      // two columns per instruction (packed fp32 pairs): e = 2^(z*log2e - M*log2e), S += e, A += e*z
      const float2 l2 = make_float2(kLog2e, kLog2e), nm2 = make_float2(-mL, -mL);
      float2 cs2 = make_float2(0.f, 0.f), ca2 = make_float2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < 32; i += 2) {
        const float2 z2 = make_float2(v[i], v[i + 1]);
        const float2 t2 = __ffma2_rn(z2, l2, nm2);
        const float2 e2 = make_float2(ex2_approx(t2.x), ex2_approx(t2.y));
        cs2 = __fadd2_rn(cs2, e2);
        ca2 = __ffma2_rn(e2, z2, ca2);
      }
      cs = cs2.x + cs2.y;
      ca = ca2.x + ca2.y;
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float e = i < nvalid ? ex2_approx(fmaf(v[i], kLog2e, -mL)) : 0.f;
        cs += e;
        ca = fmaf(e, v[i], ca);
      }
    }
    st.s = fmaf(st.s, scale, cs);
    st.a = fmaf(st.a, scale, ca);
    st.m = newm;
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
    if (row < m_rows) p.partials[(size_t)nr * p.part_stride + row] = make_float4(st.m, st.s, st.a, st.zy);
  }
};

// ---------------------------------------------------------------------------------------------
// Gradient with respect to the logits for one slab of rows x vocabulary columns, rounded to
// bf16 and written to the slab scratch (row-major) by bulk tensor stores: each epilogue warp packs
// two consecutive 32-column chunks of its 32 rows into a 128-byte-swizzled 32x64 bf16 box in
// shared memory (two boxes per warp) and one lane hands the box to the TMA unit:
//   g_tj = cp_t (p_tj - 1[j = y_t]) + ce_t p_tj (log p_tj + Ent_t),  p_tj = exp(z_tj - lse_t)
// cp_t = -w_t dloss_t/dlogp_t and ce_t = w_t ent_coef come from the per-token loss kernel.
// Rows past the valid rows of the slab and columns past V are written as zero.
struct EpiGrad {
  static constexpr int kStagingBytes = 4 * kStagingPerWarp;
  struct Params {
    const int* tokens_c;
    const float* lse;
    const float* ent;
    const float* cp;
    const float* ce;
    int V;
    int vocab_base;  // global column of the slab's column 0
  };
  struct State {
    float lse, ent, cp, ce;
    int y;
    bool valid;
    uint32_t n_issued;   // boxes handed to the TMA unit so far (selects the staging buffer)
  };
  __device__ static __forceinline__ void begin_unit(const Params& p, State& st, int m_tile, int, int row_in_tile,
                                                    int m_rows, int slab_off, int) {
    const int rl = m_tile * BM + row_in_tile;
    st.valid = rl < m_rows;
    const int gr = slab_off + rl;   // compact row of this slab row
    st.lse = st.valid ? p.lse[gr] : 0.f;
    st.ent = st.valid ? p.ent[gr] : 0.f;
    st.cp = st.valid ? p.cp[gr] : 0.f;
    st.ce = st.valid ? p.ce[gr] : 0.f;
    st.y = st.valid ? p.tokens_c[gr] : -1;
  }
  __device__ static __forceinline__ void init(State& st) { st.n_issued = 0; }
  __device__ static __forceinline__ void finish(State& st) {
    if ((threadIdx.x & 31) == 0 && st.n_issued) bulk_wait_group_all();
    __syncwarp();
  }
  __device__ static __forceinline__ void chunk(const Params& p, State& st, int m_tile, int n_tile, int c,
                                               int row_in_tile, int m_rows, const float (&v)[32],
                                               const CUtensorMap* tmG, uint32_t staging) {
    // a CTA pair may own a 128-row tile that lies wholly past the slab's rows: nothing to write
    if (m_tile * BM >= ((m_rows + BM - 1) / BM) * BM) return;
    const int col_l = n_tile * BN + c * 32;
    const int col_g = p.vocab_base + col_l;
    const int nvalid = p.V - col_g;
    float g[32];
    if (!st.valid || nvalid <= 0) {
#pragma unroll
      for (int i = 0; i < 32; ++i) g[i] = 0.f;
    } else {
      if (st.ce == 0.f) {
        // packed fp32 pairs: p = 2^(z*log2e - lse*log2e), g = cp * p
        const float2 l2 = make_float2(kLog2e, kLog2e), nl2 = make_float2(-st.lse * kLog2e, -st.lse * kLog2e);
        const float2 cp2 = make_float2(st.cp, st.cp);
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float2 t2 = __ffma2_rn(make_float2(v[i], v[i + 1]), l2, nl2);
          const float2 g2 = __fmul2_rn(make_float2(ex2_approx(t2.x), ex2_approx(t2.y)), cp2);
          g[i] = g2.x;
          g[i + 1] = g2.y;
        }
      } else {
        // entropy term as well, still two columns per instruction:
        // g = p * (ce * (z - lse) + (ce * Ent + cp))
        const float2 l2 = make_float2(kLog2e, kLog2e), nl2 = make_float2(-st.lse * kLog2e, -st.lse * kLog2e);
        const float2 nlse2 = make_float2(-st.lse, -st.lse), ce2 = make_float2(st.ce, st.ce);
        const float k = fmaf(st.ce, st.ent, st.cp);
        const float2 k2 = make_float2(k, k);
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float2 z2 = make_float2(v[i], v[i + 1]);
          const float2 t2 = __ffma2_rn(z2, l2, nl2);
          const float2 e2 = make_float2(ex2_approx(t2.x), ex2_approx(t2.y));
          const float2 w2 = __ffma2_rn(ce2, __fadd2_rn(z2, nlse2), k2);
          const float2 g2 = __fmul2_rn(e2, w2);
          g[i] = g2.x;
          g[i + 1] = g2.y;
        }
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
      // first half of a new box: the store issued from this buffer two boxes ago must have read it
      if (lane == 0) bulk_wait_group_read<1>();
      __syncwarp();
    }
    // row `lane` of the box is 128 bytes = 8 chunks of 8 bf16; chunk j sits at position j ^ (row & 7)
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

// ---------------------------------------------------------------------------------------------
// Plain fp32 output tile: C[slice][row_base + row, col] = acc (+ previous value when accumulating).
// Each epilogue warp stages its 32x32 chunk in shared memory (128-byte swizzled, two buffers) and
// one lane hands it to the TMA unit: a bulk tensor store, or a bulk tensor reduce-add when
// accumulating.  The output is seen through a 3-D fp32 tensor map {columns, rows, K slices}, which
// also clips rows past the tensor.  Every element is written by exactly one tile per launch, so
// the result does not depend on timing.
struct EpiAcc {
  static constexpr int kStagingBytes = 4 * kStagingPerWarp;
  struct Params {
    int n_cols;
    int accumulate;
    int row_base;
    int slice_add;   // stream-K launches: output slices past the first are always added to
  };
  struct State {
    int k_slice;
    uint32_t n_issued;   // chunks handed to the TMA unit so far (selects the staging buffer)
  };
  __device__ static __forceinline__ void init(State& st) { st.n_issued = 0; }
  __device__ static __forceinline__ void finish(State& st) {
    if ((threadIdx.x & 31) == 0 && st.n_issued) bulk_wait_group_all();
    __syncwarp();
  }
  __device__ static __forceinline__ void begin_unit(const Params&, State& st, int, int, int, int, int, int k_slice) {
    st.k_slice = k_slice;
  }
  __device__ static __forceinline__ void chunk(const Params& p, State& st, int m_tile, int n_tile, int c,
                                               int row_in_tile, int m_rows, const float (&v)[32],
                                               const CUtensorMap* tmC, uint32_t staging) {
    const int lane = threadIdx.x & 31;
    const int row0 = m_tile * BM + (row_in_tile - lane);   // first row of this warp's 32
    const int col0 = n_tile * BN + c * 32;
    if (row0 >= m_rows || col0 >= p.n_cols) return;        // warp-uniform
    const uint32_t buf = staging + (st.n_issued & 1u) * 4096u;
    // the store issued from this buffer two chunks ago must have finished reading it
    if (lane == 0) bulk_wait_group_read<1>();
    __syncwarp();
    // row `lane` of the box: 8 chunks of 16 bytes, chunk j stored at position j ^ (row & 7)
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint32_t addr = buf + lane * 128u + (uint32_t((j ^ (lane & 7)) << 4));
      asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v[4 * j]), "f"(v[4 * j + 1]),
                   "f"(v[4 * j + 2]), "f"(v[4 * j + 3])
                   : "memory");
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
      if (p.accumulate || (p.slice_add && st.k_slice > 0)) tma_reduce_add_3d(tmC, buf, col0, p.row_base + row0, st.k_slice);
      else              tma_store_3d(tmC, buf, col0, p.row_base + row0, st.k_slice);
      bulk_commit_group();
    }
    st.n_issued++;
  }
  __device__ static __forceinline__ void end_unit(const Params&, State&, int, int, int, int) {}
};

}  // namespace rlh
