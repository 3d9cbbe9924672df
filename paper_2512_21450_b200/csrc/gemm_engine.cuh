// Persistent, warp-specialised bf16 GEMM main loop for sm_100a with pluggable epilogues.  One
// kernel template serves every tensor-core pass of the library; a tile mode picks how the two
// 256-column fp32 accumulators of tensor memory are used.
//
//   warp 0      : TMA producer (one lane) - streams A and B k-slices (64 elements of K) into a
//                 shared-memory ring, 128-byte swizzled; a ring stage holds one k-slice, or two for
//                 the 256-column pair tiles (see StageCfg::kKSub).
//   warp 1      : allocates tensor memory; one lane issues tcgen05.mma.
//   warps 2..5  : epilogue - each warp owns the 32 tensor-memory lanes (tile rows) that its
//                 rank modulo 4 may read, pulls the accumulator out in 32-column chunks and
//                 hands them to the epilogue functor.
//
// Tile modes (per CTA 128 accumulator rows):
//   kTileSquare : a tile is 256 columns wide and lives in ONE accumulator; tile t uses accumulator
//                 t & 1, so the MMAs of tile t + 1 overlap the epilogue of tile t.  Used where K is
//                 short and the epilogue heavy (forward statistics, gradient of the logits).
//   kTileWide   : a tile is 512 columns wide and fills BOTH accumulators; a stage holds A and two B
//                 boxes, every k-slice of A feeds two UMMAs, so a CTA pulls a quarter fewer operand
//                 bytes from L2 per flop; the epilogue of a tile no longer overlaps the next main
//                 loop (about 1 % of a tile at K of 17-19 thousand).  CTA pairs only.  Used for the
//                 two long-K gradient products dH = G W and dW = G^T H.
//   kTileDual   : a tile is 256 columns wide and BOTH accumulators hold it, one per product:
//                 Z = A B^T (K = k_len) and Z2 = A2 B2^T (K = k2_len) of the same rows and columns,
//                 whose 32-column chunks reach the epilogue side by side.  Used for the
//                 full-distribution KL (policy and reference logits).  All operands K-major.
//
// CG = 1: one CTA per 128-row tile (4 stages of 16 KB A + 32 KB B).
// CG = 2: a cluster of two CTAs (one SM pair) per 256-row tile.  Each CTA stages its own 128 rows
//         of A and 128 of every 256 columns of B, the even CTA issues tcgen05.mma.cta_group::2
//         (M = 256) which reads both halves of B and writes 128 accumulator rows into each CTA's
//         tensor memory; both CTAs run their own epilogue.  All TMA completions of a stage are
//         counted on the even CTA's barrier; stage-free and accumulator-ready signals reach both
//         CTAs through one tcgen05.commit; the odd CTA's epilogue reports its accumulator drained
//         to the even CTA with a remote mbarrier arrive.  Every TMA load is addressed to the
//         shared memory of the CTA that issues it.
//
// Either operand may be K-major (its global tensor is [rows, K], K contiguous) or MN-major
// (its global tensor is [K, rows], rows contiguous).  A K-major tile is one 2-D TMA box
// {64 k, rows}; an MN-major tile is one 3-D box {64 rows, 64 k, rows/64}, which lands in shared
// memory as rows/64 panels of 8 KB, each panel 64 k-lines of 128 bytes.
//
// All three roles walk the same list of work units (UnitWalk), so K slices, stream-K balancing and
// row groups exist for every tile mode.  Every wait is bounded: when one runs out the block raises
// a shared abort flag, every role leaves its loop, the status word is latched and the block still
// frees its tensor memory.
#pragma once
#include <cuda.h>

#include "ptx.cuh"

namespace rlh {

constexpr int BM = 128;   // accumulator rows per CTA
constexpr int BN = 256;   // accumulator columns
constexpr int BK = 64;
constexpr int kAStageBytes = BM * BK * 2;
constexpr int kGemmThreads = 192;
constexpr int kTileSmemBytes = 224 * 1024;             // operand ring + epilogue staging
constexpr int kGemmSmemBytes = kTileSmemBytes + 1024;  // + slack for 1024-byte alignment
constexpr int kStagingPerWarp = 8192;                  // two 32x32 fp32 boxes per epilogue warp
constexpr int kTmemCols = 512;
constexpr int kMaxSplit = 16;   // most column ranges per row tile when the split is chosen to fill the machine
constexpr int kFwdRange = 8;    // column tiles per work unit when there is plenty of work

enum TileMode { kTileSquare = 0, kTileWide = 1, kTileDual = 2 };

// kStaging: bytes of shared memory the epilogue keeps for itself behind the ring.
template <int CG, int MODE, int kStaging>
struct StageCfg {
  static constexpr int kBRows = BN / CG;                    // B rows (output columns) of one box staged per CTA
  static constexpr int kBBytes = kBRows * BK * 2;
  static constexpr int kBBoxes = MODE == kTileWide ? 2 : 1; // B boxes per k-slice
  static constexpr int kSliceBytes = kAStageBytes + kBBoxes * kBBytes;   // one k-slice of 64: A box, then the B boxes
  // k-slices per ring stage.  The MMA issuer is one thread whose chain per stage - wait, fence, UMMAs, commit - has
  // to stay shorter than the tensor work it hands out; a 256-column pair tile has only 512 tensor clocks per
  // k-slice, so its stages hold two k-slices (eight UMMAs per barrier round trip, as a wide tile has).
  static constexpr int kKSub = (CG == 2 && MODE != kTileWide) ? 2 : 1;
  static constexpr int kStageBytes = kKSub * kSliceBytes;
  static constexpr int kStages = (kTileSmemBytes - kStaging) / kStageBytes;   // 4 (CG = 1); 3 (square pairs); 4 (wide)
  static constexpr int kRingBytes = kStages * kStageBytes;
  static constexpr uint32_t kTxBytes = uint32_t(kStageBytes) * CG;  // bytes counted on the issuing CTA's barrier
};
constexpr int kMaxStages = 7;

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
  // With n_range == 0 and n_range_hi > 0 the range length is chosen in [n_range_lo, n_range_hi] by choose_range():
  // always (n_range_always != 0) or only when there is plenty of work (otherwise the split that fills the SMs).
  int n_range_lo, n_range_hi, n_range_always;
  int skip_if_k0;   // nothing to do at all when K is empty (otherwise the epilogue sees zeros)
  int n_fastest;    // 1: consecutive units walk the column ranges of one row tile first
  // Row slabs of the backward pass: when slab_cap > 0 the valid rows are cut into
  // ceil(n_valid / slab_cap) slabs of equal size (a multiple of 256, at most slab_cap) and this
  // launch works on slab slab_index: its row offset replaces m_dyn_off / k_dyn_off, and is added
  // to the A row coordinate (a_mn_slab) or the B k coordinate (b_k_slab).
  int slab_cap, slab_index, a_mn_slab, b_k_slab;
  // K split: when k_split_max > 1 every output tile may be cut into up to k_split_max slices of
  // the K range, each a work unit of its own that adds into its own output buffer (the epilogue
  // gets the slice index); the slice count is chosen on the device to even out the last wave.
  int k_split_max;
  // Stream-K: when set (and the tiles are not cut by k_split, n_range == 1) and the tile count is
  // not a multiple of the worker count, the tiles of the last full wave and of the ragged wave
  // after it are balanced: their (tile, k-block) iterations, tile-major, are cut into one
  // contiguous share per worker, so every worker gets the same amount of tensor-core work.  A
  // tile that straddles two shares is finished by two workers: the part that starts at k-block 0
  // goes to output slice 0, the part that ends the tile is ADDED to output slice 1 (which the
  // caller zeroes beforehand), so each output element still has exactly one writer per slice and
  // launch.  Every share holds at least one whole tile's worth of iterations, so a tile has at
  // most two parts.
  int stream_k;
  // Row groups (only when the units are walked rows-first, n_fastest == 0): when m_group > 0 the row
  // tiles are taken at most m_group at a time (in groups of equal size) and all column ranges are
  // walked for one group before the next group starts, so that the A panels the CTAs running at any
  // moment keep re-reading stay in L2; B is then fetched once per group instead of once per launch.
  int m_group;
  // coordinate offsets into the operands' global tensors
  int a_mn_off, a_k_off, b_mn_off, b_k_off;
};

// Number of vocabulary ranges each row tile is split into so that (row tiles x ranges) fills the
// machine: minimises waves * tiles-per-range, preferring fewer ranges on ties.  m_units = row
// tiles of 128*CG rows, n_workers = CTAs (CG = 1) or CTA pairs (CG = 2).
__host__ __device__ inline int choose_split(int m_units, int n_tiles, int n_workers) {
  int best = 1;
  long best_cost = -1;
  for (int s = 1; s <= kMaxSplit && s <= n_tiles; ++s) {
    long units = (long)m_units * s;
    long waves = (units + n_workers - 1) / n_workers;
    long cost = waves * ((n_tiles + s - 1) / s);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
  }
  return best;
}

// Column tiles per work unit, in [lo, hi], for a pass whose units all cost the same per tile: minimises the time of
// the busiest worker, estimated as (waves of units) x (range length), with 5 % of a tile charged per unit for what
// the roles do between units (unit coordinates on the MMA issuer's serial chain, per-row loads of the epilogue).
// Measured on the gradient-of-the-logits pass (148 column tiles, 66 row tiles, 74 workers): ranges of 1 / 2 / 4 / 8
// tiles take 8.02 / 7.86 / 7.80 / 7.90 ms.
__host__ __device__ inline int choose_range(int m_units, int n_tiles, int n_workers, int lo, int hi) {
  int best = lo;
  long best_cost = -1;
  for (int nr = lo; nr <= hi; ++nr) {
    const long ranges = (n_tiles + nr - 1) / nr;
    const long waves = ((long)m_units * ranges + n_workers - 1) / n_workers;
    const long cost = waves * (100 * nr + 5);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = nr; }
  }
  return best;
}

struct GemmExtents {
  int m_rows, m_units, k_blocks, n_range, n_ranges, n_units, slab_off, k_split, kb_per, stream_k, m_group;
};

// Number of K slices per tile (1..smax) that minimises the number of waves the tiles take on
// n_workers workers, charging about 1 % per extra slice for the extra output traffic.
__host__ __device__ inline int choose_k_split(long tiles, int n_workers, int smax) {
  int best = 1;
  long best_cost = -1;
  for (int sp = 1; sp <= smax && sp <= 4; ++sp) {
    const long waves = (tiles * sp + n_workers - 1) / n_workers;
    const long cost = waves * (12 / sp) * (100 + sp - 1);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = sp; }
  }
  return best;
}

// Offset and row count of slab `index` when n_valid rows are cut into equal slabs of at most cap rows.
__host__ __device__ inline void slab_extent(int n_valid, int cap, int index, int& off, int& rows) {
  int n_slabs = (n_valid + cap - 1) / cap;
  if (n_slabs < 1) n_slabs = 1;
  int per = ((n_valid + n_slabs - 1) / n_slabs + 255) / 256 * 256;
  if (per > cap) per = cap;
  off = index * per;
  rows = n_valid - off;
  rows = rows < 0 ? 0 : (rows > per ? per : rows);
}

// cg = CTAs per output row tile, n_workers = gridDim.x / cg.
__host__ __device__ inline GemmExtents gemm_extents(const GemmShape& sh, int n_valid, int cg, int n_workers) {
  GemmExtents e;
  e.slab_off = 0;
  int m, k;
  if (sh.slab_cap > 0) {
    slab_extent(n_valid, sh.slab_cap, sh.slab_index, e.slab_off, m);
    k = m;
  } else {
    m = n_valid - sh.m_dyn_off;
    k = n_valid - sh.k_dyn_off;
  }
  m = m < 0 ? 0 : (m > sh.m_rows_cap ? sh.m_rows_cap : m);
  e.m_rows = sh.m_dyn ? m : sh.m_rows_cap;
  k = k < 0 ? 0 : (k > sh.k_cap ? sh.k_cap : k);
  const int k_len = sh.k_dyn ? k : sh.k_cap;
  e.m_units = (e.m_rows + BM * cg - 1) / (BM * cg);
  e.k_blocks = (k_len + BK - 1) / BK;
  const bool plenty = (long)e.m_units * ((sh.n_tiles + kFwdRange - 1) / kFwdRange) >= 4L * n_workers;
  if (sh.n_range > 0) {
    e.n_range = sh.n_range;
  } else if (sh.n_range_hi > 0 && (sh.n_range_always || plenty)) {
    e.n_range = choose_range(e.m_units, sh.n_tiles, n_workers, sh.n_range_lo > 0 ? sh.n_range_lo : 1, sh.n_range_hi);
  } else if (plenty) {
    // plenty of work: short fixed ranges, walked rows-first, keep every worker within a few
    // column tiles of the others, so the B operand is fetched from DRAM about once
    e.n_range = kFwdRange;
  } else {
    const int split = choose_split(e.m_units, sh.n_tiles, n_workers);
    e.n_range = (sh.n_tiles + split - 1) / split;
  }
  if (e.n_range < 1) e.n_range = 1;
  e.n_ranges = (sh.n_tiles + e.n_range - 1) / e.n_range;
  e.n_units = e.m_units * e.n_ranges;
  e.k_split = sh.k_split_max > 1 ? choose_k_split((long)e.n_units, n_workers, sh.k_split_max) : 1;
  e.kb_per = (e.k_blocks + e.k_split - 1) / e.k_split;
  e.n_units *= e.k_split;
  if (sh.skip_if_k0 && e.k_blocks == 0) e.n_units = 0;
  // row groups of equal size: as few groups as the budget of sh.m_group row tiles allows
  e.m_group = 0;
  if (sh.m_group > 0 && !sh.n_fastest && sh.m_group < e.m_units) {
    const int n_groups = (e.m_units + sh.m_group - 1) / sh.m_group;
    e.m_group = (e.m_units + n_groups - 1) / n_groups;
  }
  e.stream_k = (sh.stream_k && e.k_split == 1 && e.n_range == 1 && e.k_blocks > 0 && e.n_units >= n_workers &&
                e.n_units % n_workers != 0) ? 1 : 0;
  return e;
}

// Unit u -> row tile mu, column range nr and the K-block range [kb0, kb1) of its K slice ks.
__host__ __device__ inline void unit_coords(const GemmShape& sh, const GemmExtents& ex, int u, int& mu, int& nr,
                                            int& ks, int& kb0, int& kb1) {
  ks = u % ex.k_split;
  u /= ex.k_split;
  kb0 = ks * ex.kb_per;
  kb1 = kb0 + ex.kb_per < ex.k_blocks ? kb0 + ex.kb_per : ex.k_blocks;
  if (sh.n_fastest) {
    nr = u % ex.n_ranges; mu = u / ex.n_ranges;
  } else if (ex.m_group > 0) {
    const int per_group = ex.m_group * ex.n_ranges;
    const int gi = u / per_group, r = u - gi * per_group;
    const int m0 = gi * ex.m_group;
    const int gsz = ex.m_group < ex.m_units - m0 ? ex.m_group : ex.m_units - m0;
    mu = m0 + r % gsz; nr = r / gsz;
  } else {
    mu = u % ex.m_units;  nr = u / ex.m_units;
  }
}

// The work units of one worker, in the order all three roles of a CTA walk them.
// Plain: units worker, worker + n_workers, ... decoded by unit_coords.  Stream-K: all full waves
// but the last are walked the same way (CTAs that run together then share operand panels); the
// remaining tiles (between one and two per worker) are balanced: their (tile, k-block) iterations,
// tile-major, are cut into one contiguous share per worker, one unit per tile a share touches; ks
// is then the output slice of the part: 0 when it starts at k-block 0, else 1.
struct UnitWalk {
  const GemmShape& sh;
  const GemmExtents& ex;
  int n_workers, u, plain_units;
  long long it, it_end;
  __host__ __device__ inline UnitWalk(const GemmShape& sh_, const GemmExtents& ex_, int worker, int n_workers_)
      : sh(sh_), ex(ex_), n_workers(n_workers_), u(worker), plain_units(ex_.n_units), it(0), it_end(0) {
    if (ex.stream_k) {
      plain_units = (ex.n_units / n_workers - 1) * n_workers;
      const long long total = (long long)(ex.n_units - plain_units) * ex.k_blocks;
      it = total * worker / n_workers;
      it_end = total * (worker + 1) / n_workers;
    }
  }
  __host__ __device__ inline bool next(int& mu, int& nr, int& ks, int& kb0, int& kb1) {
    if (u < plain_units) {
      unit_coords(sh, ex, u, mu, nr, ks, kb0, kb1);
      u += n_workers;
      return true;
    }
    if (it >= it_end) return false;
    const int t_rel = (int)(it / ex.k_blocks);
    kb0 = (int)(it - (long long)t_rel * ex.k_blocks);
    const long long left = it_end - it;
    kb1 = (left < (long long)(ex.k_blocks - kb0)) ? kb0 + (int)left : ex.k_blocks;
    ks = kb0 > 0 ? 1 : 0;
    it += kb1 - kb0;
    const int tile = plain_units + t_rel;
    if (sh.n_fastest) { nr = tile % ex.n_ranges; mu = tile / ex.n_ranges; }
    else              { mu = tile % ex.m_units;  nr = tile / ex.m_units; }
    return true;
  }
};

// Epilogue functor contract (all methods run in the 128 epilogue threads, one tile row each):
//   struct Epi { struct Params; struct State;
//     static void begin_unit(const Params&, State&, int m_tile, int n_range_idx, int row_in_tile, int m_rows, int slab_off, int k_slice);
//     static void chunk(const Params&, State&, int m_tile, int n_tile, int chunk, int row_in_tile, int m_rows, const float (&v)[32],
//                       const CUtensorMap* out_map, uint32_t staging);
//     static void end_unit(const Params&, State&, int m_tile, int n_range_idx, int row_in_tile, int m_rows);
//     static void init(State&); static void finish(State&);     // once per kernel, per thread
//     static constexpr int kStagingBytes;                      // shared memory behind the ring (0 or 32 KB) };
//   kTileDual: chunk receives the chunk of the second product as well (..., v, v2, out_map, staging).
// m_tile counts 128-row tiles, n_tile 256-column tiles (a wide tile n covers column tiles 2n and 2n + 1;
// sh.n_tiles then counts 512-wide tiles).  tmA2 / tmB2 / k2_len are read by kTileDual only.
template <class Epi, int A_MN, int B_MN, int CG, int MODE>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2,
            const __grid_constant__ CUtensorMap tmC, const GemmShape sh, const int k2_len,
            const typename Epi::Params ep, DevStatus* status) {
  static_assert(MODE != kTileWide || CG == 2, "wide tiles run on CTA pairs");
  static_assert(MODE != kTileDual || (A_MN == 0 && B_MN == 0), "the two-product mode takes K-major operands");
  using Cfg = StageCfg<CG, MODE, Epi::kStagingBytes>;
  constexpr int kStages = Cfg::kStages;
  constexpr int kProducts = MODE == kTileDual ? 2 : 1;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kMaxStages];
  __shared__ __align__(8) uint64_t bar_empty[kMaxStages];
  __shared__ __align__(8) uint64_t bar_acc_full[2];
  __shared__ __align__(8) uint64_t bar_acc_empty[2];
  __shared__ __align__(8) uint64_t bar_drain;
  __shared__ uint32_t tmem_base_smem;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t rank = CG == 2 ? cluster_ctarank() : 0u;   // position in the CTA pair
  const int worker = blockIdx.x / CG;
  const int n_workers = gridDim.x / CG;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(smem_u32(&bar_acc_full[a]), 1); mbar_init(smem_u32(&bar_acc_empty[a]), 4 * CG); }
    mbar_init(smem_u32(&bar_drain), 1);
    abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
    if (MODE == kTileDual) { prefetch_tmap(&tmA2); prefetch_tmap(&tmB2); }
  }
  if (warp == 1) {
    if (CG == 2) { tmem_alloc_pair(smem_u32(&tmem_base_smem), kTmemCols); tmem_relinquish_pair(); }
    else         { tmem_alloc(smem_u32(&tmem_base_smem), kTmemCols);      tmem_relinquish(); }
  }
  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync_all();   // the peer's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_smem;
  volatile int* abort_p = &abort_flag;

  const GemmExtents ex = gemm_extents(sh, sh.n_valid ? *sh.n_valid : 0, CG, n_workers);
  const int k2_blocks = MODE == kTileDual ? (k2_len + BK - 1) / BK : 0;
  // the two-product mode has nothing to do unless both products have a K range
  const bool run = MODE != kTileDual || (ex.k_blocks > 0 && k2_blocks > 0);

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer (both CTAs)
    if (lane == 0 && run) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      UnitWalk walk(sh, ex, worker, n_workers);
      int mu, nr, ks, kb0, kb1;
      while (ok && walk.next(mu, nr, ks, kb0, kb1)) {
        const int m = mu * CG + (int)rank;
        const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
        const int a_row = sh.a_mn_off + (sh.a_mn_slab ? ex.slab_off : 0) + m * BM;
        for (int n = n0; n < n1 && ok; ++n) {
          for (int prod = 0; prod < kProducts && ok; ++prod) {
            const CUtensorMap* ta = prod ? &tmA2 : &tmA;
            const CUtensorMap* tb = prod ? &tmB2 : &tmB;
            const int lo = prod ? 0 : kb0, hi = prod ? k2_blocks : kb1;
            for (int kb = lo; kb < hi; kb += Cfg::kKSub) {
              if (!mbar_wait_bounded(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_p)) {
                latch_status(status, kStatusTimeout, (1 << 28) | (blockIdx.x << 8) | stage);
                ok = false;
                break;
              }
              const uint32_t full_local = smem_u32(&bar_full[stage]);
              // the even CTA's barrier counts the bytes of both CTAs' copies
              if (CG == 1 || rank == 0) mbar_arrive_expect_tx(full_local, Cfg::kTxBytes);
              const uint32_t full = CG == 2 ? mapa_cluster(full_local, 0) : full_local;
              // A stage always receives all its k-slices: one that lies past the K range of the unit is loaded all
              // the same (past the tensor it reads as zeros) and the issuer leaves it out.
#pragma unroll
              for (int j = 0; j < Cfg::kKSub; ++j) {
                const uint32_t a_dst = tiles_base + stage * Cfg::kStageBytes + j * Cfg::kSliceBytes;
                const uint32_t b_dst = a_dst + kAStageBytes;
                const int a_k = (prod ? 0 : sh.a_k_off) + (kb + j) * BK;
                const int b_k = (prod ? 0 : sh.b_k_off + (sh.b_k_slab ? ex.slab_off : 0)) + (kb + j) * BK;
                if (CG == 1) {
                  if (A_MN) tma_load_3d(a_dst, ta, full, 0, a_k, a_row / 64);
                  else      tma_load_2d(a_dst, ta, full, a_k, a_row);
                } else {
                  if (A_MN) tma_load_3d_pair(a_dst, ta, full, 0, a_k, a_row / 64);
                  else      tma_load_2d_pair(a_dst, ta, full, a_k, a_row);
                }
#pragma unroll
                for (int s = 0; s < Cfg::kBBoxes; ++s) {
                  const int b_row = sh.b_mn_off + (n * Cfg::kBBoxes + s) * BN + (int)rank * Cfg::kBRows;
                  const uint32_t dst = b_dst + s * Cfg::kBBytes;
                  if (CG == 1) {
                    if (B_MN) tma_load_3d(dst, tb, full, 0, b_k, b_row / 64);
                    else      tma_load_2d(dst, tb, full, b_k, b_row);
                  } else {
                    if (B_MN) tma_load_3d_pair(dst, tb, full, 0, b_k, b_row / 64);
                    else      tma_load_2d_pair(dst, tb, full, b_k, b_row);
                  }
                }
              }
              if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
          }
        }
      }
      if (!ok && (CG == 1 || rank == 0)) {
        // let copies that were already issued land before the block's shared memory goes away
        for (int s = 0; s < kStages; ++s) {
          uint32_t p = (s < stage) ? phase : (phase ^ 1u);
          for (int it = 0; it < 4096 && !mbar_try_wait(smem_u32(&bar_full[s]), p); ++it) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer (even CTA of a pair)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(BM * CG, BN, A_MN, B_MN);
      // K-major: 8-row groups 1024 B apart, 32 bytes per 16-element k step.
      // MN-major: 64-row panels 8192 B apart, 8-k-line groups 1024 B apart, 2048 B per k step.
      constexpr uint64_t a_hi = A_MN ? make_smem_desc_hi(8192, 1024) : make_smem_desc_hi(16, 1024);
      constexpr uint64_t b_hi = B_MN ? make_smem_desc_hi(8192, 1024) : make_smem_desc_hi(16, 1024);
      constexpr uint32_t a_kstep = A_MN ? 2048 : 32;
      constexpr uint32_t b_kstep = B_MN ? 2048 : 32;
      // The issuing thread is a serial chain - wait for a stage, fence, eight UMMAs (four on single-CTA tiles), commit -
      // that has to stay shorter than the tensor work it hands out (1024 clocks per stage of a pair tile).  Besides
      // the two k-slices per stage of the 256-column tiles, two things keep it short: the barrier of the NEXT stage is polled before the UMMAs of this one are issued, so the
      // latency of that poll hides behind them (`ready` carries its answer into the next round, also across tiles);
      // and descriptors, barrier addresses and stage offsets are kept as running 32-bit words instead of being
      // rebuilt from the stage index.
      constexpr uint32_t a_hi32 = uint32_t(a_hi >> 32), b_hi32 = uint32_t(b_hi >> 32);
      constexpr uint32_t a_lo_const = uint32_t(a_hi), b_lo_const = uint32_t(b_hi);   // bits [16, 30): leading offset
      const uint32_t ring_lo = (tiles_base & 0x3FFFFu) >> 4;
      int stage = 0;
      uint32_t phase = 0;
      uint32_t ready = 0;   // 1: the full barrier of `stage` is already known to have completed at `phase`
      uint32_t t = 0;   // tiles issued so far
      bool ok = true;
      if (run && ex.k_blocks > 0) {
        UnitWalk walk(sh, ex, worker, n_workers);
        int mu, nr, ks, kb0, kb1;
        while (ok && walk.next(mu, nr, ks, kb0, kb1)) {
          if (kb1 <= kb0) continue;   // empty K slice: the epilogue handles it without an accumulator
          const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
          for (int n = n0; n < n1 && ok; ++n, ++t) {
            // square tiles alternate between the accumulators; the other modes need both drained
            const uint32_t a = MODE == kTileSquare ? (t & 1u) : 0u;
            const uint32_t par = MODE == kTileSquare ? (((t >> 1) & 1u) ^ 1u) : ((t & 1u) ^ 1u);
            for (uint32_t w = a; w < (MODE == kTileWide ? 2u : a + 1u) && ok; ++w) {
              if (!mbar_wait_bounded_cluster(smem_u32(&bar_acc_empty[w]), par, abort_p)) {
                latch_status(status, kStatusTimeout, (2 << 28) | (blockIdx.x << 8) | w);
                ok = false;
              }
            }
            if (!ok) break;
            tc_fence_after();
            for (int prod = 0; prod < kProducts && ok; ++prod) {
              const uint32_t d_tmem = tmem_base + (MODE == kTileDual ? prod : a) * BN;
              const int lo = prod ? 0 : kb0, hi = prod ? k2_blocks : kb1;
              for (int kb = lo; kb < hi; kb += Cfg::kKSub) {
                if (!ready && !mbar_wait_bounded_cluster(smem_u32(&bar_full[stage]), phase, abort_p)) {
                  latch_status(status, kStatusTimeout, (3 << 28) | (blockIdx.x << 8) | stage);
                  ok = false;
                  break;
                }
                // poll the next ring position now; the answer is looked at after this stage's UMMAs are out
                const int nstage = stage + 1 == kStages ? 0 : stage + 1;
                const uint32_t nphase = stage + 1 == kStages ? phase ^ 1u : phase;
                const uint32_t peek = mbar_try_wait_cluster(smem_u32(&bar_full[nstage]), nphase);
                tc_fence_after();
                const uint32_t a_lo = a_lo_const | (ring_lo + uint32_t(stage) * (Cfg::kStageBytes >> 4));
                const uint32_t b_lo = b_lo_const | (ring_lo + uint32_t(stage) * (Cfg::kStageBytes >> 4) + (kAStageBytes >> 4));
#pragma unroll
                for (int j = 0; j < Cfg::kKSub; ++j) {
                  if (j > 0 && kb + j >= hi) break;   // a k-slice past the unit's K range was loaded but is not used
#pragma unroll
                  for (int k = 0; k < BK / 16; ++k) {
                    const uint32_t acc = (kb > lo || j > 0 || k > 0) ? 1u : 0u;
#pragma unroll
                    for (int s = 0; s < Cfg::kBBoxes; ++s)
                      umma_bf16_words<CG>(d_tmem + s * BN, a_lo + (j * Cfg::kSliceBytes + k * a_kstep) / 16, a_hi32,
                                          b_lo + (j * Cfg::kSliceBytes + s * Cfg::kBBytes + k * b_kstep) / 16, b_hi32,
                                          idesc, acc);
                  }
                }
                if (CG == 2) umma_commit_pair_mcast(smem_u32(&bar_empty[stage]), 3);
                else         umma_commit(smem_u32(&bar_empty[stage]));
                stage = nstage;
                phase = nphase;
                ready = peek;
              }
            }
            if (ok) {
              if (CG == 2) umma_commit_pair_mcast(smem_u32(&bar_acc_full[a]), 3);
              else         umma_commit(smem_u32(&bar_acc_full[a]));
            }
          }
        }
      }
      // every UMMA issued above has to retire before tensor memory is released
      if (CG == 2) umma_commit_pair(smem_u32(&bar_drain));
      else         umma_commit(smem_u32(&bar_drain));
      bool drained = false;
      for (int it = 0; it < (1 << 22) && !drained; ++it) drained = mbar_try_wait(smem_u32(&bar_drain), 0) != 0;
      if (!drained) latch_status(status, kStatusTimeout, (4 << 28) | (blockIdx.x << 8));
    }
  } else {
    // ------------------------------------------------------------- epilogue warps (both CTAs)
    const int q = warp & 3;
    const int row_in_tile = q * 32 + lane;
    const uint32_t staging = tiles_base + Cfg::kRingBytes + q * kStagingPerWarp;   // this warp's epilogue staging
    typename Epi::State st;
    Epi::init(st);
    uint32_t t = 0;
    bool ok = true;
    UnitWalk walk(sh, ex, worker, n_workers);
    int mu, nr, ks, kb0, kb1;
    while (ok && run && walk.next(mu, nr, ks, kb0, kb1)) {
      const bool has_k = kb1 > kb0;   // an empty K slice contributes zeros
      const int m = mu * CG + (int)rank;
      const int n0 = nr * ex.n_range, n1 = min(n0 + ex.n_range, sh.n_tiles);
      Epi::begin_unit(ep, st, m, nr, row_in_tile, ex.m_rows, ex.slab_off, ks);
      for (int n = n0; n < n1 && ok; ++n, t += has_k ? 1u : 0u) {
        const uint32_t a = MODE == kTileSquare ? (t & 1u) : 0u;
        if (has_k) {
          const uint32_t par = MODE == kTileSquare ? ((t >> 1) & 1u) : (t & 1u);
          if (!mbar_wait_bounded_cluster(smem_u32(&bar_acc_full[a]), par, abort_p)) {
            latch_status(status, kStatusTimeout, (5 << 28) | (blockIdx.x << 8) | a);
            ok = false;
          }
          ok = __all_sync(0xffffffffu, ok);   // tensor-memory loads below need the whole warp
          if (!ok) break;
          tc_fence_after();
        }
#pragma unroll 1
        for (int s = 0; s < Cfg::kBBoxes; ++s) {
          const uint32_t acc_i = a + (uint32_t)s;   // accumulator this half of the tile sits in
          const uint32_t taddr = tmem_base + acc_i * BN + (uint32_t(q * 32) << 16);
#pragma unroll 1
          for (int c = 0; c < BN / 32; ++c) {
            float v[32];
            if constexpr (MODE == kTileDual) {
              uint32_t r[32], r2[32];
              tmem_ld_32x32(taddr + c * 32, r);
              tmem_ld_32x32(taddr + BN + c * 32, r2);
              tmem_ld_wait();
              float v2[32];
#pragma unroll
              for (int i = 0; i < 32; ++i) { v[i] = __uint_as_float(r[i]); v2[i] = __uint_as_float(r2[i]); }
              Epi::chunk(ep, st, m, n, c, row_in_tile, ex.m_rows, v, v2, &tmC, staging);
            } else {
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
              Epi::chunk(ep, st, m, n * Cfg::kBBoxes + s, c, row_in_tile, ex.m_rows, v, &tmC, staging);
            }
          }
          if (has_k) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
              if (CG == 2 && rank != 0) mbar_arrive_cluster(mapa_cluster(smem_u32(&bar_acc_empty[acc_i]), 0));
              else                      mbar_arrive(smem_u32(&bar_acc_empty[acc_i]));
            }
          }
        }
      }
      if (ok) Epi::end_unit(ep, st, m, nr, row_in_tile, ex.m_rows);
    }
    Epi::finish(st);   // e.g. wait for bulk stores that still read this warp's staging memory
  }

  tc_fence_before();
  __syncthreads();
  if (CG == 2) cluster_sync_all();   // the pair's UMMAs have retired and both epilogues are done
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (CG == 2) tmem_dealloc_pair(tmem_base, kTmemCols);
    else         tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace rlh
