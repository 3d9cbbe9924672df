// C ABI of the fused LM-head log-probability + GRPO policy-loss library: argument checks,
// workspace layout, tensor-map construction and the launch sequences.  All arithmetic of the
// path runs in the kernels of gemm_engine.cuh / epilogues.cuh / small_kernels.cuh.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "rlhead.h"
#include "small_kernels.cuh"
#include "cluster_probe.cuh"

using namespace rlh;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kProfMax = 1 << 16;   // timed launch groups kept between two rl_profile_read calls
constexpr int kProfKinds = 9;    // 0 forward statistics, 1 dlogits, 2 dH, 3 dW, 4 mask scan, 5 row gather,
                                 // 6 merge + loss, 7 dH scatter, 8 advantages

struct rl_ctx {
  int device;
  int n_sm;
  cudaStream_t stream;
  DevStatus* dstatus;  // device
  void* ws;
  size_t ws_bytes;
  EncodeTiledFn encode;
  int slab_rows;  // rows of one gradient slab (multiple of 128)
  int slab_cols;  // vocabulary columns of one gradient slab (multiple of 256)
  int cta_group;  // 1: one CTA per 128x256 tile; 2: CTA pairs on 256x256 tiles
  int dh_k_slices;  // upper bound on the K slices of the dH pass (1 = tiles are not cut)
  long long row_group_bytes;  // forward / dlogits: bytes of A panels walked together (0 = all row tiles at once)
  int wide_tiles;   // 1: dH and dW run on 256 x 512 tiles (both accumulators hold one tile)
  int dh_stream_k;  // 1: the dH pass balances its tiles over the SMs by stream-K (needs a second accumulator buffer)
  int grid[3];    // persistent grid for cta_group 1 and 2 (index = cta_group)
  int grid_full[3];   // the same before rl_set_max_ctas() capped it
  rl_dw_slab_hook dw_hook;   // called after the launch that completes a slab of dW rows was enqueued
  void* dw_hook_user;
  long long launches;  // kernels launched by this context so far
  // optional per-kernel timing: event pairs around every tensor-core launch, by kernel kind
  int prof_on;
  int prof_used;
  // pipelined host-buffer steps: a copy stream, per-slot events and pinned result words (created on first use)
  cudaStream_t copy_stream;
  cudaEvent_t copy_done[2], step_done[2];
  float* pinned_out[2];
  int slot_busy[2];
  int* prof_kind;                 // [kProfMax], allocated when profiling is first switched on
  cudaEvent_t (*prof_ev)[2];      // [kProfMax][2], events created on first use
};

namespace {

constexpr long long kRowGroupBytes = 36ll << 20;   // A panels walked together by the rows-first passes (L2 is 126 MB)
constexpr int kSlabRowsMax = 32768;        // rows of one gradient slab
// Device words a context owns besides the workspace: the status record, a few scalars of the small kernels
// (byte 64: batch statistics, 96: longest response, 128: valid-row count of rl_token_loss) and, from byte 256 on,
// the block partials of rl_token_loss.
constexpr int kTokenLossBlocks = 1024;
constexpr size_t kStatusBytes = 256 + (size_t)kTokenLossBlocks * kLossSums * sizeof(double);
constexpr int kAdvRowsMinGroups = 2048;     // from this many groups on, GRPO advantages run one thread per group
constexpr int kDhSplitMax = 4;             // most K slices (separate fp32 accumulators) of the dH pass
constexpr int kSlabColsMax = 148 * 256;    // vocabulary columns of one gradient slab (148 tiles of 256: two per SM pair)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// fp32 accumulator buffers of the dH pass: one per K slice, or two when stream-K balancing is on
inline bool dh_uses_stream_k(const rl_ctx* c) { return c->dh_stream_k && c->dh_k_slices == 1; }
inline int dh_buffers(const rl_ctx* c) { return dh_uses_stream_k(c) ? 2 : c->dh_k_slices; }

struct WsLayout {
  int Tpad, Ts, Vs;
  size_t scan_counts, row_map, tokens_c, logp_c, lse_c, ent_c, cp_c, ce_c, partials, block_sums, Hc, G, dH_acc, staging, total;
  size_t Hc_ref, partials2, lse_ref_c, kl_c, cb_c;   // only with a reference model (full KL)
};

// Reference-model operands of the full-distribution KL (all NULL / 0 when it is not used).
struct KlRef {
  const void* H_ref;
  int64_t ldH_ref;
  const void* W_ref;
  int64_t ldW_ref;
  int64_t d_ref;
};

// Device copies of one step's host inputs (H, tokens, old, ref, adv, mask, rewards, offsets) and its result words.
struct HostStage {
  void* H;
  int32_t* tok;
  float *old_lp, *ref_lp, *adv;
  uint8_t* mask;
  float* out;       // [16]: loss, 7 unused, 8 metrics
  float *rew, *advseq;
  int32_t* off;
};
inline size_t carve_stage(char* base, int64_t T, int64_t d, HostStage* hs) {
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 1024); return base ? base + at : nullptr; };
  HostStage h;
  h.H = take((size_t)T * d * 2);
  h.tok = reinterpret_cast<int32_t*>(take((size_t)T * 4));
  h.old_lp = reinterpret_cast<float*>(take((size_t)T * 4));
  h.ref_lp = reinterpret_cast<float*>(take((size_t)T * 4));
  h.adv = reinterpret_cast<float*>(take((size_t)T * 4));
  h.mask = reinterpret_cast<uint8_t*>(take((size_t)T));
  h.out = reinterpret_cast<float*>(take(64));
  h.rew = reinterpret_cast<float*>(take((size_t)T * 4));
  h.advseq = reinterpret_cast<float*>(take((size_t)T * 4));
  h.off = reinterpret_cast<int32_t*>(take((size_t)(T + 1) * 4));
  if (hs) *hs = h;
  return o;
}

// host_slots > 0 adds room for that many sets of host-call inputs behind the scratch proper.
WsLayout ws_layout(const rl_ctx* c, int64_t T, int64_t d, int64_t V, int host_slots, int64_t d_ref = 0) {
  WsLayout L;
  L.Tpad = (int)align_up((size_t)(T > 0 ? T : 1), 128);
  L.Ts = L.Tpad < c->slab_rows ? L.Tpad : c->slab_rows;
  const int Vpad = (int)align_up((size_t)V, 256);
  L.Vs = Vpad < c->slab_cols ? Vpad : c->slab_cols;
  size_t o = 0;
  size_t n_part_ranges = kMaxSplit;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 1024); return at; };
  L.scan_counts = take(((size_t)L.Tpad / 4096 + 2) * 4);
  L.row_map = take((size_t)L.Tpad * 4);
  L.tokens_c = take((size_t)L.Tpad * 4);
  L.logp_c = take((size_t)L.Tpad * 4);
  L.lse_c = take((size_t)L.Tpad * 4);
  L.ent_c = take((size_t)L.Tpad * 4);
  L.cp_c = take((size_t)L.Tpad * 4);
  L.ce_c = take((size_t)L.Tpad * 4);
  {
    // one float4 per (column range, row): at most kMaxSplit ranges, or one per kFwdRange column tiles
    const size_t by_range = (size_t)(((V + BN - 1) / BN + kFwdRange - 1) / kFwdRange);
    n_part_ranges = by_range > (size_t)kMaxSplit ? by_range : (size_t)kMaxSplit;
    L.partials = take(n_part_ranges * L.Tpad * sizeof(float4));
  }
  L.block_sums = take((size_t)1024 * kLossSums * sizeof(double));
  L.Hc = take((size_t)L.Tpad * d * 2);
  L.G = take((size_t)L.Ts * L.Vs * 2);
  L.dH_acc = take((size_t)dh_buffers(c) * L.Ts * d * 4);
  L.Hc_ref = L.partials2 = L.lse_ref_c = L.kl_c = L.cb_c = 0;
  if (d_ref > 0) {
    L.Hc_ref = take((size_t)L.Tpad * d_ref * 2);
    L.partials2 = take((size_t)n_part_ranges * L.Tpad * sizeof(float4));
    L.lse_ref_c = take((size_t)L.Tpad * 4);
    L.kl_c = take((size_t)L.Tpad * 4);
    L.cb_c = take((size_t)L.Tpad * 4);
  }
  L.staging = o;
  o += (size_t)host_slots * carve_stage(nullptr, T, d, nullptr);
  L.total = o;
  return L;
}

// K-major operand: global tensor [rows, k] with k contiguous, row stride ld elements.
bool map_kmajor(rl_ctx* c, CUtensorMap* m, const void* base, uint64_t rows, uint64_t k, uint64_t ld,
                uint32_t box_rows) {
  cuuint64_t dims[2] = {k, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t es[2] = {1, 1};
  return c->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// MN-major operand: global tensor [k, mn] with mn contiguous (a multiple of 64), row stride ld.
// Seen by TMA as {64, k, mn/64} so that one box {64, 64, chunks} fetches `chunks` 64-wide panels.
bool map_mnmajor(rl_ctx* c, CUtensorMap* m, const void* base, uint64_t k_rows, uint64_t mn, uint64_t ld,
                 uint32_t chunks) {
  cuuint64_t dims[3] = {64, k_rows, mn / 64};
  cuuint64_t strides[2] = {ld * 2, 128};
  cuuint32_t box[3] = {64, 64, chunks};
  cuuint32_t es[3] = {1, 1, 1};
  return c->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 output seen by the accumulate epilogue: {cols, rows, slices} with 32x32 boxes, 128-byte
// swizzled in shared memory.  slices > 1: identical [rows, ld] buffers slice_rows rows apart.
bool map_out_f32(rl_ctx* c, CUtensorMap* m, const float* base, uint64_t rows, uint64_t cols, uint64_t ld,
                 uint64_t slices, uint64_t slice_rows) {
  cuuint64_t dims[3] = {cols, rows, slices};
  cuuint64_t strides[2] = {ld * 4, slice_rows * ld * 4};
  cuuint32_t box[3] = {32, 32, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return c->encode(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 [rows, cols] slab written by the dlogits epilogue in 32-row x 64-column boxes.
bool map_out_bf16(rl_ctx* c, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint64_t ld) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {64, 32};
  cuuint32_t es[2] = {1, 1};
  return c->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <class Epi, int A_MN, int B_MN, int CG, int MODE>
cudaError_t set_smem_attr_one() {
  return cudaFuncSetAttribute(gemm_kernel<Epi, A_MN, B_MN, CG, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kGemmSmemBytes);
}
// square tiles, single CTAs and CTA pairs
template <class Epi, int A_MN, int B_MN>
cudaError_t set_smem_attr() {
  cudaError_t e = set_smem_attr_one<Epi, A_MN, B_MN, 1, kTileSquare>();
  return e != cudaSuccess ? e : set_smem_attr_one<Epi, A_MN, B_MN, 2, kTileSquare>();
}
template <class Epi>
cudaError_t set_smem_attr_dual() {
  cudaError_t e = set_smem_attr_one<Epi, 0, 0, 1, kTileDual>();
  return e != cudaSuccess ? e : set_smem_attr_one<Epi, 0, 0, 2, kTileDual>();
}

// Rows of B that one CTA stages per k-slice (box height of a K-major B map) and the number of
// 64-wide panels of an MN-major B map, for the context's CTA grouping.
inline uint32_t b_box_rows(const rl_ctx* c) { return BN / c->cta_group; }
inline uint32_t b_box_panels(const rl_ctx* c) { return BN / 64 / c->cta_group; }

// Optional timing of a group of launches: event pair on the context's stream, tagged with a kind.
int prof_begin(rl_ctx* c, int kind) {
  if (!(c->prof_on && c->prof_ev && kind >= 0 && kind < kProfKinds && c->prof_used < kProfMax)) return -1;
  const int i = c->prof_used;
  for (int e = 0; e < 2; ++e)
    if (!c->prof_ev[i][e]) cudaEventCreate(&c->prof_ev[i][e]);
  cudaEventRecord(c->prof_ev[i][0], c->stream);
  return i;
}
void prof_end(rl_ctx* c, int i, int kind) {
  if (i < 0) return;
  cudaEventRecord(c->prof_ev[i][1], c->stream);
  c->prof_kind[i] = kind;
  c->prof_used = i + 1;
}

// One launch of the tensor-core engine in tile mode MODE on the context's persistent grid (CTA pairs
// when cta_group is 2; wide tiles exist for pairs only).  a2 / b2 / k2_len: second product (kTileDual).
template <class Epi, int A_MN, int B_MN, int MODE>
void launch_tiles(rl_ctx* c, int kind, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& a2,
                  const CUtensorMap& b2, const CUtensorMap& out, const GemmShape& sh, int k2_len,
                  const typename Epi::Params& ep) {
  const int prof = prof_begin(c, kind);
  if (c->cta_group == 2) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(c->grid[2]);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = kGemmSmemBytes;
    cfg.stream = c->stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, gemm_kernel<Epi, A_MN, B_MN, 2, MODE>, a, b, a2, b2, out, sh, k2_len, ep, c->dstatus);
  } else if constexpr (MODE != kTileWide) {
    gemm_kernel<Epi, A_MN, B_MN, 1, MODE><<<c->grid[1], kGemmThreads, kGemmSmemBytes, c->stream>>>(
        a, b, a2, b2, out, sh, k2_len, ep, c->dstatus);
  }
  c->launches++;
  prof_end(c, prof, kind);
}

template <class Epi, int A_MN, int B_MN>
void launch_gemm(rl_ctx* c, int kind, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& out,
                 const GemmShape& sh, const typename Epi::Params& ep) {
  launch_tiles<Epi, A_MN, B_MN, kTileSquare>(c, kind, a, b, a, b, out, sh, 0, ep);
}

// 256 x 512 tiles on CTA pairs; sh.n_tiles counts 512-wide column tiles.
inline bool use_wide(const rl_ctx* c) { return c->wide_tiles && c->cta_group == 2; }

template <class Epi, int A_MN, int B_MN>
void launch_wide(rl_ctx* c, int kind, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& out,
                 const GemmShape& sh, const typename Epi::Params& ep) {
  launch_tiles<Epi, A_MN, B_MN, kTileWide>(c, kind, a, b, a, b, out, sh, 0, ep);
}

template <class Epi>
void launch_dual(rl_ctx* c, int kind, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& a2,
                 const CUtensorMap& b2, const CUtensorMap& out, const GemmShape& sh, int k2_len,
                 const typename Epi::Params& ep) {
  launch_tiles<Epi, 0, 0, kTileDual>(c, kind, a, b, a2, b2, out, sh, k2_len, ep);
}

rl_status check_hw(const void* H, int64_t ldH, const void* W, int64_t ldW, int64_t T, int64_t d, int64_t V) {
  if (T < 0 || d <= 0 || V <= 0) return RL_ERR_INVALID_ARG;
  if (T > 0 && (!H || !W)) return RL_ERR_INVALID_ARG;
  if (d % 64 != 0) return RL_ERR_SHAPE;
  if (T >= (int64_t(1) << 30) || V >= (int64_t(1) << 30)) return RL_ERR_SHAPE;
  if (ldH < d || ldW < d) return RL_ERR_SHAPE;
  if (ldH % 8 != 0 || ldW % 8 != 0) return RL_ERR_ALIGNMENT;
  if ((reinterpret_cast<uintptr_t>(H) & 15) || (reinterpret_cast<uintptr_t>(W) & 15)) return RL_ERR_ALIGNMENT;
  return RL_OK;
}

rl_status check_ws(rl_ctx* c, const WsLayout& L) {
  if (!c->ws || c->ws_bytes < L.total) return RL_ERR_WORKSPACE;
  return RL_OK;
}

// Vocabulary-parallel call: W holds the vocabulary ids [vocab_off, vocab_off + V) of V_total and the
// per-token statistics of the whole vocabulary come from the caller.
struct ShardArgs {
  int64_t vocab_off, V_total;
  const float* logp;
  const float* entropy;
  const float* lse;
};

// Row tiles per group for the rows-first passes: as many A panels (one row tile x K, bf16) as fit the byte budget.
inline int row_group_tiles(const rl_ctx* c, int64_t k) {
  if (c->row_group_bytes <= 0) return 0;
  const long long panel = (long long)BM * c->cta_group * k * 2;
  const long long n = c->row_group_bytes / panel;
  return n < 1 ? 1 : (n > (1 << 20) ? (1 << 20) : (int)n);
}

inline rl_status cuda_ok() { return cudaGetLastError() == cudaSuccess ? RL_OK : RL_ERR_CUDA; }

// Which part of the forward stage a call needs, and where its rows of W sit in the vocabulary.
struct FwdPlan {
  bool scan = true;          // mask scan (false: the row map of an earlier call on this workspace is reused)
  bool stats = true;         // tensor-core pass that leaves per-range statistics in the workspace
  int64_t vocab_off = 0;     // first vocabulary id of W's rows (vocabulary-parallel head)
  int64_t V_total = 0;       // size of the whole vocabulary for the token-range check (0: V)
};

// Mask scan + row compaction + forward statistics.  Leaves per-range partials in the workspace.
rl_status run_forward(rl_ctx* c, const WsLayout& L, const void* H, int64_t ldH, const void* W, int64_t ldW,
                      const int32_t* tokens, const uint8_t* mask, int64_t T, int64_t d, int64_t V,
                      GemmShape* shape_out, const KlRef* kl = nullptr, const FwdPlan& plan = FwdPlan()) {
  char* ws = static_cast<char*>(c->ws);
  int* row_map = reinterpret_cast<int*>(ws + L.row_map);
  int* tokens_c = reinterpret_cast<int*>(ws + L.tokens_c);
  __nv_bfloat16* Hc = reinterpret_cast<__nv_bfloat16*>(ws + L.Hc);
  if (plan.scan) {
    const int pr = prof_begin(c, 4);
    int* block_counts = reinterpret_cast<int*>(ws + L.scan_counts);
    const int n_blocks = (int)((T + kScanRowsPerBlock - 1) / kScanRowsPerBlock);
    mask_count_kernel<<<n_blocks, kScanThreads, 0, c->stream>>>(mask, (int)T, block_counts);
    mask_offsets_kernel<<<1, 1024, 0, c->stream>>>(block_counts, n_blocks, c->dstatus);
    mask_write_kernel<<<n_blocks, kScanThreads, 0, c->stream>>>(mask, (int)T, block_counts, row_map);
    prof_end(c, pr, 4);
    c->launches += 3;
  }
  const int pr_gather = prof_begin(c, 5);
  gather_rows_kernel<<<c->n_sm * 4, 256, 0, c->stream>>>(static_cast<const __nv_bfloat16*>(H), ldH, (int)d, row_map,
                                                         tokens, (int)(plan.V_total > 0 ? plan.V_total : V),
                                                         (int)plan.vocab_off, Hc, tokens_c, c->dstatus);
  prof_end(c, pr_gather, 5);
  c->launches += 1;
  if (!plan.stats) {
    memset(shape_out, 0, sizeof(*shape_out));
    return cuda_ok();
  }
  CUtensorMap tmA, tmB;
  if (!map_kmajor(c, &tmA, Hc, (uint64_t)L.Tpad, (uint64_t)d, (uint64_t)d, BM)) return RL_ERR_CUDA;
  if (!map_kmajor(c, &tmB, W, (uint64_t)V, (uint64_t)d, (uint64_t)ldW, b_box_rows(c))) return RL_ERR_CUDA;
  GemmShape sh;
  memset(&sh, 0, sizeof(sh));
  sh.n_valid = &c->dstatus->n_valid;
  sh.m_rows_cap = L.Tpad;
  sh.m_dyn = 1;
  sh.k_cap = (int)d;
  sh.n_tiles = (int)((V + BN - 1) / BN);
  sh.n_range = 0;  // split chosen on the device from the number of valid rows
  sh.m_group = row_group_tiles(c, d + (kl ? kl->d_ref : 0));
  EpiStats::Params ep;
  ep.tokens_c = tokens_c;
  ep.partials = reinterpret_cast<float4*>(ws + L.partials);
  ep.part_stride = L.Tpad;
  ep.V = (int)V;
  if (!kl) {
    launch_gemm<EpiStats, 0, 0>(c, 0, tmA, tmB, tmA, sh, ep);   // no output map
  } else {
    // full KL: compact the reference hidden states with the same row map and form both logit
    // tiles per output tile
    __nv_bfloat16* Hc_ref = reinterpret_cast<__nv_bfloat16*>(ws + L.Hc_ref);
    gather_plain_kernel<<<c->n_sm * 4, 256, 0, c->stream>>>(static_cast<const __nv_bfloat16*>(kl->H_ref), kl->ldH_ref,
                                                            (int)kl->d_ref, row_map, Hc_ref, c->dstatus);
    c->launches++;
    CUtensorMap tmA2, tmB2;
    if (!map_kmajor(c, &tmA2, Hc_ref, (uint64_t)L.Tpad, (uint64_t)kl->d_ref, (uint64_t)kl->d_ref, BM)) return RL_ERR_CUDA;
    if (!map_kmajor(c, &tmB2, kl->W_ref, (uint64_t)V, (uint64_t)kl->d_ref, (uint64_t)kl->ldW_ref, b_box_rows(c)))
      return RL_ERR_CUDA;
    EpiStatsKL::Params ek;
    ek.tokens_c = tokens_c;
    ek.partials = ep.partials;
    ek.partials2 = reinterpret_cast<float4*>(ws + L.partials2);
    ek.part_stride = L.Tpad;
    ek.V = (int)V;
    launch_dual<EpiStatsKL>(c, 0, tmA, tmB, tmA2, tmB2, tmA, sh, (int)kl->d_ref, ek);
  }
  *shape_out = sh;
  return cuda_ok();
}

}  // namespace

extern "C" {

const char* rl_status_string(rl_status s) {
  switch (s) {
    case RL_OK: return "ok";
    case RL_ERR_INVALID_ARG: return "invalid argument";
    case RL_ERR_SHAPE: return "unsupported shape";
    case RL_ERR_ALIGNMENT: return "pointer or leading dimension not aligned for TMA";
    case RL_ERR_WORKSPACE: return "workspace missing or too small";
    case RL_ERR_CUDA: return "CUDA call failed";
    case RL_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x";
    case RL_ERR_TOKEN_RANGE: return "token id outside [0,V) on a valid row";
    case RL_ERR_TIMEOUT: return "bounded wait inside a kernel ran out";
  }
  return "unknown status";
}

rl_status rl_create(rl_ctx** out, int device) {
  if (!out) return RL_ERR_INVALID_ARG;
  *out = nullptr;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return RL_ERR_CUDA;
  if (prop.major != 10) return RL_ERR_UNSUPPORTED_ARCH;
  if (cudaSetDevice(device) != cudaSuccess) return RL_ERR_CUDA;
  rl_ctx* c = new (std::nothrow) rl_ctx();
  if (!c) return RL_ERR_CUDA;
  c->device = device;
  c->n_sm = prop.multiProcessorCount;
  c->stream = nullptr;
  c->ws = nullptr;
  c->ws_bytes = 0;
  c->slab_rows = kSlabRowsMax;
  c->slab_cols = kSlabColsMax;
  c->cta_group = 1;
  c->dh_k_slices = 1;
  c->dh_stream_k = 0;
  c->wide_tiles = 1;
  c->row_group_bytes = kRowGroupBytes;
  c->grid[0] = 0;
  c->grid[1] = c->n_sm;
  c->grid[2] = c->n_sm / 2 * 2;
  c->launches = 0;
  c->prof_on = 0;
  c->prof_used = 0;
  c->prof_kind = nullptr;
  c->prof_ev = nullptr;
  c->copy_stream = nullptr;
  for (int i = 0; i < 2; ++i) { c->copy_done[i] = nullptr; c->step_done[i] = nullptr; c->pinned_out[i] = nullptr; c->slot_busy[i] = 0; }
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess) {
    delete c;
    return RL_ERR_CUDA;
  }
  c->encode = reinterpret_cast<EncodeTiledFn>(fn);
  // device block: status word, then two doubles for batch statistics
  if (cudaMalloc(&c->dstatus, kStatusBytes) != cudaSuccess) { delete c; return RL_ERR_CUDA; }
  cudaMemset(c->dstatus, 0, kStatusBytes);
  bool ok = set_smem_attr<EpiStats, 0, 0>() == cudaSuccess && set_smem_attr<EpiGrad, 0, 0>() == cudaSuccess &&
            set_smem_attr<EpiAcc, 0, 0>() == cudaSuccess && set_smem_attr<EpiAcc, 0, 1>() == cudaSuccess &&
            set_smem_attr<EpiAcc, 1, 0>() == cudaSuccess && set_smem_attr<EpiAcc, 1, 1>() == cudaSuccess &&
            set_smem_attr_dual<EpiStatsKL>() == cudaSuccess && set_smem_attr_dual<EpiGradKL>() == cudaSuccess &&
            set_smem_attr_one<EpiAcc, 0, 0, 2, kTileWide>() == cudaSuccess &&
            set_smem_attr_one<EpiAcc, 0, 1, 2, kTileWide>() == cudaSuccess &&
            set_smem_attr_one<EpiAcc, 1, 0, 2, kTileWide>() == cudaSuccess &&
            set_smem_attr_one<EpiAcc, 1, 1, 2, kTileWide>() == cudaSuccess;
  if (!ok) { cudaFree(c->dstatus); delete c; return RL_ERR_CUDA; }
  {
    // how many CTA pairs can be resident at once (pairs must share a TPC): the persistent grid
    // of the paired kernels must not exceed it
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(c->grid[2]);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = kGemmSmemBytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&n_clusters, gemm_kernel<EpiAcc, 0, 0, 2, kTileSquare>, &cfg) == cudaSuccess &&
        n_clusters > 0) {
      if (2 * n_clusters < c->grid[2]) c->grid[2] = 2 * n_clusters;
    } else {
      cudaGetLastError();
      c->grid[2] = 0;   // paired kernels unavailable
    }
    if (c->grid[2] >= 2) c->cta_group = 2;   // default: CTA pairs
  }
  for (int i = 0; i < 3; ++i) c->grid_full[i] = c->grid[i];
  c->dw_hook = nullptr;
  c->dw_hook_user = nullptr;
  *out = c;
  return RL_OK;
}

rl_status rl_destroy(rl_ctx* c) {
  if (!c) return RL_ERR_INVALID_ARG;
  if (c->prof_ev) {
    for (int i = 0; i < kProfMax; ++i)
      for (int e = 0; e < 2; ++e)
        if (c->prof_ev[i][e]) cudaEventDestroy(c->prof_ev[i][e]);
    delete[] c->prof_ev;
    delete[] c->prof_kind;
  }
  if (c->copy_stream) {
    cudaStreamSynchronize(c->copy_stream);
    cudaStreamDestroy(c->copy_stream);
    for (int i = 0; i < 2; ++i) {
      cudaEventDestroy(c->copy_done[i]);
      cudaEventDestroy(c->step_done[i]);
      cudaFreeHost(c->pinned_out[i]);
    }
  }
  cudaFree(c->dstatus);
  delete c;
  return RL_OK;
}

rl_status rl_set_stream(rl_ctx* c, void* s) {
  if (!c) return RL_ERR_INVALID_ARG;
  c->stream = static_cast<cudaStream_t>(s);
  return RL_OK;
}

rl_status rl_workspace_bytes(rl_ctx* c, int64_t T, int64_t d, int64_t V, size_t* bytes) {
  if (!c || !bytes || T < 0 || d <= 0 || V <= 0) return RL_ERR_INVALID_ARG;
  *bytes = ws_layout(c, T, d, V, false).total;
  return RL_OK;
}

rl_status rl_workspace_bytes_kl(rl_ctx* c, int64_t T, int64_t d, int64_t V, int64_t d_ref, size_t* bytes) {
  if (!c || !bytes || T < 0 || d <= 0 || V <= 0 || d_ref <= 0) return RL_ERR_INVALID_ARG;
  *bytes = ws_layout(c, T, d, V, false, d_ref).total;
  return RL_OK;
}

rl_status rl_workspace_bytes_host(rl_ctx* c, int64_t T, int64_t d, int64_t V, size_t* bytes) {
  if (!c || !bytes || T < 0 || d <= 0 || V <= 0) return RL_ERR_INVALID_ARG;
  *bytes = ws_layout(c, T, d, V, true).total;
  return RL_OK;
}

rl_status rl_set_cta_group(rl_ctx* c, int cta_group) {
  if (!c) return RL_ERR_INVALID_ARG;
  if (cta_group != 1 && cta_group != 2) return RL_ERR_INVALID_ARG;
  if (cta_group == 2 && c->grid[2] < 2) return RL_ERR_UNSUPPORTED_ARCH;
  c->cta_group = cta_group;
  return RL_OK;
}

rl_status rl_set_max_ctas(rl_ctx* c, int max_ctas) {
  if (!c || max_ctas < 0) return RL_ERR_INVALID_ARG;
  if (max_ctas == 0) {
    for (int i = 0; i < 3; ++i) c->grid[i] = c->grid_full[i];
    return RL_OK;
  }
  if (max_ctas < 2) return RL_ERR_INVALID_ARG;
  c->grid[1] = max_ctas < c->grid_full[1] ? max_ctas : c->grid_full[1];
  const int pairs = max_ctas / 2 * 2;
  c->grid[2] = pairs < c->grid_full[2] ? pairs : c->grid_full[2];
  return RL_OK;
}

rl_status rl_set_dw_slab_hook(rl_ctx* c, rl_dw_slab_hook hook, void* user) {
  if (!c) return RL_ERR_INVALID_ARG;
  c->dw_hook = hook;
  c->dw_hook_user = hook ? user : nullptr;
  return RL_OK;
}

rl_status rl_set_dh_k_slices(rl_ctx* c, int max_slices) {
  if (!c) return RL_ERR_INVALID_ARG;
  if (max_slices < 1 || max_slices > kDhSplitMax) return RL_ERR_INVALID_ARG;
  c->dh_k_slices = max_slices;
  return RL_OK;
}

rl_status rl_set_row_group_bytes(rl_ctx* c, int64_t bytes) {
  if (!c || bytes < 0) return RL_ERR_INVALID_ARG;
  c->row_group_bytes = bytes;
  return RL_OK;
}

rl_status rl_set_wide_tiles(rl_ctx* c, int on) {
  if (!c) return RL_ERR_INVALID_ARG;
  c->wide_tiles = on ? 1 : 0;
  return RL_OK;
}

rl_status rl_set_dh_stream_k(rl_ctx* c, int on) {
  if (!c) return RL_ERR_INVALID_ARG;
  c->dh_stream_k = on ? 1 : 0;
  return RL_OK;
}

rl_status rl_launch_count(rl_ctx* c, int64_t* n) {
  if (!c || !n) return RL_ERR_INVALID_ARG;
  *n = c->launches;
  return RL_OK;
}

rl_status rl_set_profiling(rl_ctx* c, int on) {
  if (!c) return RL_ERR_INVALID_ARG;
  if (on && !c->prof_ev) {
    c->prof_kind = new (std::nothrow) int[kProfMax];
    c->prof_ev = new (std::nothrow) cudaEvent_t[kProfMax][2];
    if (!c->prof_kind || !c->prof_ev) {
      delete[] c->prof_kind;
      delete[] c->prof_ev;
      c->prof_kind = nullptr;
      c->prof_ev = nullptr;
      return RL_ERR_CUDA;
    }
    memset(c->prof_ev, 0, sizeof(cudaEvent_t) * 2 * kProfMax);
  }
  c->prof_on = on ? 1 : 0;
  c->prof_used = 0;
  return RL_OK;
}

rl_status rl_profile_read(rl_ctx* c, double* ms, int64_t* launches) {
  if (!c || !ms || !launches) return RL_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return RL_ERR_CUDA;
  for (int k = 0; k < kProfKinds; ++k) { ms[k] = 0.0; launches[k] = 0; }
  for (int i = 0; i < c->prof_used; ++i) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, c->prof_ev[i][0], c->prof_ev[i][1]) != cudaSuccess) return RL_ERR_CUDA;
    ms[c->prof_kind[i]] += t;
    launches[c->prof_kind[i]]++;
  }
  c->prof_used = 0;
  return RL_OK;
}

rl_status rl_set_slab_limits(rl_ctx* c, int max_rows, int max_cols) {
  if (!c) return RL_ERR_INVALID_ARG;
  if (max_rows == 0) max_rows = kSlabRowsMax;
  if (max_cols == 0) max_cols = kSlabColsMax;
  if (max_rows < 128 || max_rows % 128 != 0 || max_cols < 256 || max_cols % 256 != 0) return RL_ERR_SHAPE;
  if ((int64_t)max_rows * max_cols > (int64_t(1) << 31)) return RL_ERR_SHAPE;
  c->slab_rows = max_rows;
  c->slab_cols = max_cols;
  return RL_OK;
}

rl_status rl_set_workspace(rl_ctx* c, void* p, size_t bytes) {
  if (!c) return RL_ERR_INVALID_ARG;
  if (p && (reinterpret_cast<uintptr_t>(p) & 255)) return RL_ERR_ALIGNMENT;
  c->ws = p;
  c->ws_bytes = p ? bytes : 0;
  return RL_OK;
}

rl_status rl_last_device_status(rl_ctx* c, int32_t* detail) {
  if (!c) return RL_ERR_INVALID_ARG;
  DevStatus h;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return RL_ERR_CUDA;
  if (cudaMemcpy(&h, c->dstatus, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return RL_ERR_CUDA;
  if (detail) *detail = h.detail;
  if (h.code != 0) {
    int zero[2] = {0, 0};
    cudaMemcpy(c->dstatus, zero, sizeof(zero), cudaMemcpyHostToDevice);
  }
  return static_cast<rl_status>(h.code);
}

rl_status rl_grpo_advantages_ex(rl_ctx* c, const float* rewards, int64_t n_seq, int group_size, int ddof,
                                float eps_std, const int32_t* seq_offsets, int64_t T, float* adv_seq,
                                float* adv_tok) {
  if (!c || n_seq < 0 || (n_seq > 0 && (!rewards || !adv_seq))) return RL_ERR_INVALID_ARG;
  if ((ddof != 0 && ddof != 1) || !(eps_std >= 0.f)) return RL_ERR_INVALID_ARG;
  if ((adv_tok != nullptr) != (seq_offsets != nullptr) || T < 0) return RL_ERR_INVALID_ARG;
  if (group_size < 2 || n_seq % group_size != 0 || n_seq >= (int64_t(1) << 31)) return RL_ERR_SHAPE;
  if (n_seq == 0) return RL_OK;
  const int n_groups = (int)(n_seq / group_size);
  const int warps = 8;
  int seg = 32;   // lanes per group, as the kernel computes it
  while (seg > 1 && (seg >> 1) >= group_size) seg >>= 1;
  const int groups_per_block = warps * (32 / seg);
  const int pr_adv = prof_begin(c, 8);
  // many groups of 4, 8, ... 32 responses in 16-byte aligned arrays: one thread per group; else shuffle segments
  const bool rows_path = n_groups >= kAdvRowsMinGroups && group_size % 4 == 0 && group_size <= 32 &&
                         ((reinterpret_cast<uintptr_t>(rewards) | reinterpret_cast<uintptr_t>(adv_seq)) & 15) == 0;
  if (rows_path) {
    const int blocks = (n_groups + 255) / 256;
    const float4* r4 = reinterpret_cast<const float4*>(rewards);
    float4* a4 = reinterpret_cast<float4*>(adv_seq);
    switch (group_size / 4) {
      case 1: grpo_adv_rows_kernel<1><<<blocks, 256, 0, c->stream>>>(r4, n_groups, ddof, eps_std, a4); break;
      case 2: grpo_adv_rows_kernel<2><<<blocks, 256, 0, c->stream>>>(r4, n_groups, ddof, eps_std, a4); break;
      case 3: grpo_adv_rows_kernel<3><<<blocks, 256, 0, c->stream>>>(r4, n_groups, ddof, eps_std, a4); break;
      case 4: grpo_adv_rows_kernel<4><<<blocks, 256, 0, c->stream>>>(r4, n_groups, ddof, eps_std, a4); break;
      case 5: grpo_adv_rows_kernel<5><<<blocks, 256, 0, c->stream>>>(r4, n_groups, ddof, eps_std, a4); break;
      case 6: grpo_adv_rows_kernel<6><<<blocks, 256, 0, c->stream>>>(r4, n_groups, ddof, eps_std, a4); break;
      case 7: grpo_adv_rows_kernel<7><<<blocks, 256, 0, c->stream>>>(r4, n_groups, ddof, eps_std, a4); break;
      default: grpo_adv_rows_kernel<8><<<blocks, 256, 0, c->stream>>>(r4, n_groups, ddof, eps_std, a4); break;
    }
  } else {
    grpo_adv_kernel<<<(n_groups + groups_per_block - 1) / groups_per_block, warps * 32, 0, c->stream>>>(
        rewards, n_groups, group_size, ddof, eps_std, adv_seq);
  }
  c->launches++;
  if (adv_tok) {
    if (T > 0) {
      const long long rows_per_block = (long long)kBroadcastSweeps * 1024;
      long long blocks = (T + rows_per_block - 1) / rows_per_block;
      if (blocks > (long long)c->n_sm * 32) blocks = (long long)c->n_sm * 32;
      broadcast_adv_kernel<<<(int)blocks, 256, 0, c->stream>>>(adv_seq, seq_offsets, (int)n_seq, (long long)T, adv_tok);
      c->launches++;
    }
  }
  prof_end(c, pr_adv, 8);
  return cuda_ok();
}

rl_status rl_advantages(rl_ctx* c, int estimator, const float* rewards, const int32_t* lengths, int64_t n_seq,
                        int group_size, float eps_std, float* adv_seq) {
  if (!c || n_seq < 0 || (n_seq > 0 && (!rewards || !adv_seq))) return RL_ERR_INVALID_ARG;
  if (estimator < RL_ADV_GRPO || estimator > RL_ADV_REINFORCE_PP || !(eps_std >= 0.f)) return RL_ERR_INVALID_ARG;
  if (estimator == RL_ADV_OPO && n_seq > 0 && !lengths) return RL_ERR_INVALID_ARG;
  if (estimator == RL_ADV_GRPO)
    return rl_grpo_advantages_ex(c, rewards, n_seq, group_size, 1, eps_std, nullptr, 0, adv_seq, nullptr);
  const int min_group = estimator == RL_ADV_RLOO ? 2 : 1;
  if (group_size < min_group || n_seq % group_size != 0 || n_seq >= (int64_t(1) << 31)) return RL_ERR_SHAPE;
  if (n_seq == 0) return RL_OK;
  const int n_groups = (int)(n_seq / group_size);
  const int warps = 8;
  const int pr = prof_begin(c, 8);
  group_baseline_kernel<<<(n_groups + warps - 1) / warps, warps * 32, 0, c->stream>>>(rewards, lengths, n_groups,
                                                                                      group_size, estimator, adv_seq);
  c->launches++;
  if (estimator == RL_ADV_REINFORCE_PP) {
    double* stats = reinterpret_cast<double*>(reinterpret_cast<char*>(c->dstatus) + 64);
    batch_stats_kernel<<<1, 1024, 0, c->stream>>>(adv_seq, (long long)n_seq, stats);
    int blocks = (int)((n_seq + 255) / 256);
    if (blocks > 4096) blocks = 4096;
    batch_normalise_kernel<<<blocks, 256, 0, c->stream>>>(adv_seq, (long long)n_seq, stats, eps_std);
    c->launches += 2;
  }
  prof_end(c, pr, 8);
  return cuda_ok();
}

rl_status rl_token_loss(rl_ctx* c, const float* logp, const float* entropy, const float* old_logp,
                        const float* ref_logp, const float* adv, const uint8_t* mask, int64_t T, float eps_low,
                        float eps_high, float beta, float ent_coef, const float* token_weight, const void* token_count,
                        float* loss, float* dlogp, float* dentropy, float* metrics_out) {
  if (!c || T < 0 || !loss) return RL_ERR_INVALID_ARG;
  if (!(eps_low >= 0.f && eps_low < 1.f) || !(eps_high >= 0.f) || !(beta >= 0.f) || !(ent_coef >= 0.f))
    return RL_ERR_INVALID_ARG;
  if (T > 0 && (!logp || !old_logp || !adv)) return RL_ERR_INVALID_ARG;
  if (T > 0 && beta != 0.f && !ref_logp) return RL_ERR_INVALID_ARG;
  if (T > 0 && ent_coef != 0.f && !entropy) return RL_ERR_INVALID_ARG;
  cudaStream_t st = c->stream;
  if (T == 0) {
    cudaMemsetAsync(loss, 0, 4, st);
    if (metrics_out) cudaMemsetAsync(metrics_out, 0, 32, st);
    return cuda_ok();
  }
  char* base = reinterpret_cast<char*>(c->dstatus);
  unsigned long long* count = reinterpret_cast<unsigned long long*>(base + 128);
  double* block_sums = reinterpret_cast<double*>(base + 256);
  const int pr = prof_begin(c, 6);
  if (mask) {
    cudaMemsetAsync(count, 0, 8, st);
    long long cb = (T / 16 + 255) / 256 + 1;
    if (cb > (long long)c->n_sm * 8) cb = (long long)c->n_sm * 8;
    count_valid_kernel<<<(int)cb, 256, 0, st>>>(mask, (long long)T, count);
    c->launches++;
  }
  TokenLossParams p;
  memset(&p, 0, sizeof(p));
  p.logp = logp; p.entropy = entropy; p.old_logp = old_logp; p.ref_logp = beta != 0.f ? ref_logp : nullptr;
  p.adv = adv; p.mask = mask; p.token_weight = token_weight;
  p.count = token_count ? reinterpret_cast<const unsigned long long*>(token_count) : (mask ? count : nullptr);
  p.n_known = (unsigned long long)T;
  p.T = (long long)T;
  p.eps_low = eps_low; p.eps_high = eps_high; p.beta = beta; p.ent_coef = ent_coef;
  p.dlogp = dlogp; p.dentropy = dentropy; p.block_sums = block_sums;
  long long blocks = ((T + 3) / 4 + kLossThreads - 1) / kLossThreads;
  if (blocks > kTokenLossBlocks) blocks = kTokenLossBlocks;
  if (blocks > (long long)c->n_sm * 4) blocks = (long long)c->n_sm * 4;   // one wave: four blocks are resident per SM
  uintptr_t all = reinterpret_cast<uintptr_t>(logp) | reinterpret_cast<uintptr_t>(old_logp) | reinterpret_cast<uintptr_t>(adv) |
                  reinterpret_cast<uintptr_t>(entropy) | reinterpret_cast<uintptr_t>(p.ref_logp) |
                  reinterpret_cast<uintptr_t>(token_weight) | reinterpret_cast<uintptr_t>(dlogp) |
                  reinterpret_cast<uintptr_t>(dentropy);
  const bool vec = (all & 15) == 0 && (reinterpret_cast<uintptr_t>(mask) & 3) == 0;
  if (vec) token_loss_kernel<true><<<(int)blocks, kLossThreads, 0, st>>>(p);
  else     token_loss_kernel<false><<<(int)blocks, kLossThreads, 0, st>>>(p);
  finalize_token_loss_kernel<<<1, 32 * kLossSums, 0, st>>>(block_sums, (int)blocks, loss, metrics_out, mask ? count : nullptr,
                                               (unsigned long long)T);
  c->launches += 2;
  prof_end(c, pr, 6);
  return cuda_ok();
}

rl_status rl_grpo_advantages(rl_ctx* c, const float* rewards, int64_t n_seq, int group_size, float* adv_seq) {
  return rl_grpo_advantages_ex(c, rewards, n_seq, group_size, 1, 1e-6f, nullptr, 0, adv_seq, nullptr);
}

rl_status rl_kl_shaped_returns(rl_ctx* c, const float* seq_value, const float* logp, const float* ref_logp,
                               const float* kl_tok, const uint8_t* mask, const int32_t* seq_offsets, int64_t n_seq,
                               int64_t T, float beta, float gamma, int kl_estimate, float* shaped_reward,
                               float* returns) {
  if (!c || n_seq < 0 || T < 0 || n_seq >= (int64_t(1) << 31) || T >= (int64_t(1) << 31)) return RL_ERR_INVALID_ARG;
  if (kl_estimate < RL_KL_K1 || kl_estimate > RL_KL_GIVEN || !(beta >= 0.f) || !(gamma >= 0.f)) return RL_ERR_INVALID_ARG;
  if (T == 0) return RL_OK;
  if (!returns) return RL_ERR_INVALID_ARG;
  if (n_seq == 0) {
    cudaMemsetAsync(returns, 0, (size_t)T * 4, c->stream);
    if (shaped_reward) cudaMemsetAsync(shaped_reward, 0, (size_t)T * 4, c->stream);
    return cuda_ok();
  }
  if (!seq_value || !seq_offsets) return RL_ERR_INVALID_ARG;
  if (kl_estimate == RL_KL_GIVEN ? !kl_tok : (!logp || !ref_logp)) return RL_ERR_INVALID_ARG;
  const int warps = 8;
  long long blocks = (n_seq + warps - 1) / warps;
  if (blocks > (long long)c->n_sm * 64) blocks = (long long)c->n_sm * 64;
  const int pr = prof_begin(c, 8);
  zero_outside_ranges_kernel<<<c->n_sm, 256, 0, c->stream>>>(seq_offsets, (int)n_seq, (long long)T, returns,
                                                             shaped_reward);
  kl_shaped_returns_kernel<<<(int)blocks, warps * 32, 0, c->stream>>>(seq_value, logp, ref_logp, kl_tok, mask,
                                                                      seq_offsets, (int)n_seq, beta, gamma, kl_estimate,
                                                                      shaped_reward, returns);
  prof_end(c, pr, 8);
  c->launches += 2;
  return cuda_ok();
}

rl_status rl_mask_scan(rl_ctx* c, const uint8_t* mask, int64_t T, int32_t* row_map, int32_t* n_valid) {
  if (!c || T < 0 || T >= (int64_t(1) << 31) || !n_valid || (T > 0 && !row_map)) return RL_ERR_INVALID_ARG;
  if (T == 0) return cudaMemsetAsync(n_valid, 0, 4, c->stream) == cudaSuccess ? RL_OK : RL_ERR_CUDA;
  const int n_blocks = (int)((T + kScanRowsPerBlock - 1) / kScanRowsPerBlock);
  if (!c->ws || c->ws_bytes < ((size_t)n_blocks + 2) * 4) return RL_ERR_WORKSPACE;
  int* block_counts = static_cast<int*>(c->ws);
  const int pr = prof_begin(c, 4);
  mask_count_kernel<<<n_blocks, kScanThreads, 0, c->stream>>>(mask, (int)T, block_counts);
  mask_offsets_kernel<<<1, 1024, 0, c->stream>>>(block_counts, n_blocks, c->dstatus);
  mask_write_kernel<<<n_blocks, kScanThreads, 0, c->stream>>>(mask, (int)T, block_counts, row_map);
  prof_end(c, pr, 4);
  c->launches += 3;
  if (cudaMemcpyAsync(n_valid, &c->dstatus->n_valid, 4, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess)
    return RL_ERR_CUDA;
  return cuda_ok();
}

rl_status rl_token_logprobs(rl_ctx* c, const void* H, int64_t ldH, const void* W, int64_t ldW, const int32_t* tokens,
                            const uint8_t* mask, int64_t T, int64_t d, int64_t V, float* logp, float* entropy,
                            float* lse) {
  if (!c) return RL_ERR_INVALID_ARG;
  rl_status s = check_hw(H, ldH, W, ldW, T, d, V);
  if (s != RL_OK) return s;
  if (T == 0) return RL_OK;
  if (!tokens || !logp) return RL_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(c, T, d, V, false);
  if ((s = check_ws(c, L)) != RL_OK) return s;
  char* ws = static_cast<char*>(c->ws);
  cudaMemsetAsync(logp, 0, (size_t)T * 4, c->stream);
  if (entropy) cudaMemsetAsync(entropy, 0, (size_t)T * 4, c->stream);
  if (lse) cudaMemsetAsync(lse, 0, (size_t)T * 4, c->stream);
  GemmShape fwd_shape;
  if ((s = run_forward(c, L, H, ldH, W, ldW, tokens, mask, T, d, V, &fwd_shape)) != RL_OK) return s;
  LossParams p;
  memset(&p, 0, sizeof(p));
  p.partials = reinterpret_cast<const float4*>(ws + L.partials);
  p.part_stride = L.Tpad;
  p.fwd_shape = fwd_shape;
  p.fwd_cg = c->cta_group;
  p.fwd_workers = c->grid[c->cta_group] / c->cta_group;
  p.row_map = reinterpret_cast<const int*>(ws + L.row_map);
  p.with_loss = 0;
  p.lse_c = reinterpret_cast<float*>(ws + L.lse_c);
  p.ent_c = reinterpret_cast<float*>(ws + L.ent_c);
  p.logp_out = logp;
  p.ent_out = entropy;
  p.lse_out = lse;
  int blocks = (int)((T + kLossThreads - 1) / kLossThreads);
  if (blocks > 1024) blocks = 1024;
  combine_loss_kernel<<<blocks, kLossThreads, 0, c->stream>>>(p, c->dstatus);
  c->launches++;
  return cuda_ok();
}

// Body of rl_policy_loss_fwd_bwd_ex (shard == NULL) and of rl_policy_loss_shard_bwd.
static rl_status loss_fwd_bwd_impl(rl_ctx* c, const void* H, int64_t ldH, const void* W, int64_t ldW,
                                   const int32_t* tokens, const float* old_logp, const float* ref_logp,
                                   const float* adv, const uint8_t* mask, int64_t T, int64_t d, int64_t V,
                                   float eps_low, float eps_high, float beta, float* loss, void* dH, float* dW,
                                   const rl_loss_opts* opts, const ShardArgs* shard) {
  if (!c) return RL_ERR_INVALID_ARG;
  rl_status s = check_hw(H, ldH, W, ldW, T, d, V);
  if (s != RL_OK) return s;
  if (!(eps_low >= 0.f && eps_low < 1.f) || !(eps_high >= 0.f) || !(beta >= 0.f)) return RL_ERR_INVALID_ARG;
  if (!loss || !dW || !W) return RL_ERR_INVALID_ARG;
  if (T > 0 && (!tokens || !old_logp || !adv || !dH)) return RL_ERR_INVALID_ARG;
  rl_loss_opts o;
  memset(&o, 0, sizeof(o));
  if (opts) {
    if (opts->struct_size < sizeof(size_t) + sizeof(float) || opts->struct_size > sizeof(rl_loss_opts))
      return RL_ERR_INVALID_ARG;
    memcpy(&o, opts, opts->struct_size);
  }
  if (!(o.ent_coef >= 0.f)) return RL_ERR_INVALID_ARG;
  if (beta != 0.f && T > 0 && !ref_logp && !o.kl_full) return RL_ERR_INVALID_ARG;
  if (o.agg_mode < 0 || o.agg_mode > 2 || (o.dH_dtype != 0 && o.dH_dtype != 1)) return RL_ERR_INVALID_ARG;
  if ((o.sequence_level || (o.agg_mode != 0 && !o.token_weight)) && T > 0 &&
      (!o.seq_offsets || o.n_seq <= 0 || o.n_seq > T))
    return RL_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(dH) & 15) || (reinterpret_cast<uintptr_t>(dW) & 15)) return RL_ERR_ALIGNMENT;
  const bool seq_path = o.sequence_level || (o.agg_mode != 0 && !o.token_weight);
  KlRef klref;
  memset(&klref, 0, sizeof(klref));
  if (shard) {
    if (o.kl_full) return RL_ERR_INVALID_ARG;
    if (shard->vocab_off < 0 || shard->V_total < shard->vocab_off + V || shard->V_total >= (int64_t(1) << 30))
      return RL_ERR_SHAPE;
    if (T > 0 && (!shard->logp || !shard->entropy || !shard->lse)) return RL_ERR_INVALID_ARG;
  }
  if (o.kl_full) {
    if (seq_path) return RL_ERR_INVALID_ARG;
    if (!o.W_ref || (T > 0 && !o.H_ref) || o.d_ref <= 0) return RL_ERR_INVALID_ARG;
    if (o.d_ref % 64 != 0 || o.ldH_ref < o.d_ref || o.ldW_ref < o.d_ref || o.ldH_ref % 8 != 0 || o.ldW_ref % 8 != 0)
      return RL_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(o.H_ref) & 15) || (reinterpret_cast<uintptr_t>(o.W_ref) & 15))
      return RL_ERR_ALIGNMENT;
    klref.H_ref = o.H_ref; klref.ldH_ref = o.ldH_ref;
    klref.W_ref = o.W_ref; klref.ldW_ref = o.ldW_ref;
    klref.d_ref = o.d_ref;
  }
  const WsLayout L = ws_layout(c, T, d, V, false, o.kl_full ? o.d_ref : 0);
  if ((s = check_ws(c, L)) != RL_OK) return s;
  char* ws = static_cast<char*>(c->ws);
  cudaStream_t st = c->stream;

  if (T == 0) {
    cudaMemsetAsync(loss, 0, 4, st);
    if (!o.accumulate_dW) cudaMemsetAsync(dW, 0, (size_t)V * d * 4, st);
    if (o.metrics_out) cudaMemsetAsync(o.metrics_out, 0, 32, st);
    return cuda_ok();
  }
  cudaMemsetAsync(dH, 0, (size_t)T * d * (o.dH_dtype ? 4 : 2), st);
  if (o.logp_out) cudaMemsetAsync(o.logp_out, 0, (size_t)T * 4, st);
  if (o.entropy_out) cudaMemsetAsync(o.entropy_out, 0, (size_t)T * 4, st);

  // ---- forward: statistics per (row, vocabulary range)
  GemmShape fwd_shape;
  FwdPlan plan;
  if (shard) {
    // the statistics of the whole vocabulary are given: only the row compaction is needed
    plan.stats = false;
    plan.vocab_off = shard->vocab_off;
    plan.V_total = shard->V_total;
  }
  if ((s = run_forward(c, L, H, ldH, W, ldW, tokens, mask, T, d, V, &fwd_shape, o.kl_full ? &klref : nullptr, plan)) !=
      RL_OK)
    return s;

  // ---- merge + per-token loss, coefficients of the backward pass
  LossParams p;
  memset(&p, 0, sizeof(p));
  p.partials = reinterpret_cast<const float4*>(ws + L.partials);
  p.part_stride = L.Tpad;
  p.fwd_shape = fwd_shape;
  p.fwd_cg = c->cta_group;
  p.fwd_workers = c->grid[c->cta_group] / c->cta_group;
  p.row_map = reinterpret_cast<const int*>(ws + L.row_map);
  p.old_logp = old_logp;
  p.ref_logp = ref_logp;
  p.adv = adv;
  p.token_weight = o.token_weight;
  p.eps_low = eps_low;
  p.eps_high = eps_high;
  p.beta = beta;
  p.ent_coef = o.ent_coef;
  p.token_count = reinterpret_cast<const long long*>(o.token_count);
  p.with_loss = 1;
  p.lse_c = reinterpret_cast<float*>(ws + L.lse_c);
  p.ent_c = reinterpret_cast<float*>(ws + L.ent_c);
  p.cp_c = reinterpret_cast<float*>(ws + L.cp_c);
  p.ce_c = reinterpret_cast<float*>(ws + L.ce_c);
  p.logp_out = o.logp_out;
  p.ent_out = o.entropy_out;
  p.block_sums = reinterpret_cast<double*>(ws + L.block_sums);
  if (shard) {
    p.ext_logp = shard->logp;
    p.ext_ent = shard->entropy;
    p.ext_lse = shard->lse;
  }
  if (o.kl_full) {
    p.kl_full = 1;
    p.partials2 = reinterpret_cast<const float4*>(ws + L.partials2);
    p.lse_ref_c = reinterpret_cast<float*>(ws + L.lse_ref_c);
    p.kl_c = reinterpret_cast<float*>(ws + L.kl_c);
    p.cb_c = reinterpret_cast<float*>(ws + L.cb_c);
    p.kl_out = o.kl_out;
    if (o.kl_out) cudaMemsetAsync(o.kl_out, 0, (size_t)T * 4, st);
  }
  int blocks = (int)((T + kLossThreads - 1) / kLossThreads);
  if (blocks > 1024) blocks = 1024;
  const int pr_loss = prof_begin(c, 6);
  if (!seq_path) {
    combine_loss_kernel<<<blocks, kLossThreads, 0, st>>>(p, c->dstatus);
    c->launches++;
  } else {
    // merge the statistics first, then one warp per response forms weights, ratios and the loss
    p.with_loss = 0;
    p.logp_c = reinterpret_cast<float*>(ws + L.logp_c);
    combine_loss_kernel<<<blocks, kLossThreads, 0, st>>>(p, c->dstatus);
    SeqParams q;
    memset(&q, 0, sizeof(q));
    q.seq_offsets = o.seq_offsets;
    q.n_seq = (int)o.n_seq;
    q.agg_mode = o.token_weight ? 0 : o.agg_mode;
    q.sequence_level = o.sequence_level ? 1 : 0;
    q.row_map = p.row_map;
    q.logp_c = p.logp_c;
    q.ent_c = p.ent_c;
    q.old_logp = old_logp;
    q.ref_logp = ref_logp;
    q.adv = adv;
    q.token_weight = o.token_weight;
    q.eps_low = eps_low; q.eps_high = eps_high; q.beta = beta; q.ent_coef = o.ent_coef;
    q.l_max = reinterpret_cast<int*>(reinterpret_cast<char*>(c->dstatus) + 96);
    q.cp_c = p.cp_c;
    q.ce_c = p.ce_c;
    q.block_sums = p.block_sums;
    // valid rows that lie outside every response range take no part: their coefficients stay 0
    cudaMemsetAsync(q.cp_c, 0, (size_t)L.Tpad * 4, st);
    cudaMemsetAsync(q.ce_c, 0, (size_t)L.Tpad * 4, st);
    seq_lmax_kernel<<<1, 1024, 0, st>>>(o.seq_offsets, (int)o.n_seq, q.l_max);
    blocks = (int)((o.n_seq + kLossThreads / 32 - 1) / (kLossThreads / 32));
    if (blocks > 1024) blocks = 1024;
    seq_loss_kernel<<<blocks, kLossThreads, 0, st>>>(q, c->dstatus);
    c->launches += 3;
  }
  finalize_loss_kernel<<<1, 32 * kLossSums, 0, st>>>(p.block_sums, blocks, loss, o.metrics_out, c->dstatus);
  prof_end(c, pr_loss, 6);
  c->launches++;

  // ---- backward, one (row slab x vocabulary slab) at a time
  __nv_bfloat16* Hc = reinterpret_cast<__nv_bfloat16*>(ws + L.Hc);
  __nv_bfloat16* G = reinterpret_cast<__nv_bfloat16*>(ws + L.G);
  float* dH_acc = reinterpret_cast<float*>(ws + L.dH_acc);
  const int* row_map = reinterpret_cast<const int*>(ws + L.row_map);
  const int* n_valid = &c->dstatus->n_valid;

  CUtensorMap tmHc_k, tmW_k, tmG_k, tmW_mn, tmG_mn, tmHc_mn, tm_dH, tm_dW, tm_G_out, tmHr_k, tmWr_k;
  if (o.kl_full) {
    if (!map_kmajor(c, &tmHr_k, ws + L.Hc_ref, (uint64_t)L.Tpad, (uint64_t)o.d_ref, (uint64_t)o.d_ref, BM) ||
        !map_kmajor(c, &tmWr_k, o.W_ref, (uint64_t)V, (uint64_t)o.d_ref, (uint64_t)o.ldW_ref, b_box_rows(c)))
      return RL_ERR_CUDA;
  }
  bool ok = map_kmajor(c, &tmHc_k, Hc, (uint64_t)L.Tpad, (uint64_t)d, (uint64_t)d, BM) &&
            map_kmajor(c, &tmW_k, W, (uint64_t)V, (uint64_t)d, (uint64_t)ldW, b_box_rows(c)) &&
            map_kmajor(c, &tmG_k, G, (uint64_t)L.Ts, (uint64_t)L.Vs, (uint64_t)L.Vs, BM) &&
            map_mnmajor(c, &tmW_mn, W, (uint64_t)V, (uint64_t)d, (uint64_t)ldW, b_box_panels(c)) &&
            map_mnmajor(c, &tmG_mn, G, (uint64_t)L.Ts, (uint64_t)L.Vs, (uint64_t)L.Vs, BM / 64) &&
            map_mnmajor(c, &tmHc_mn, Hc, (uint64_t)L.Tpad, (uint64_t)d, (uint64_t)d, b_box_panels(c)) &&
            map_out_bf16(c, &tm_G_out, G, (uint64_t)L.Ts, (uint64_t)L.Vs, (uint64_t)L.Vs) &&
            map_out_f32(c, &tm_dH, dH_acc, (uint64_t)L.Ts, (uint64_t)d, (uint64_t)d, (uint64_t)dh_buffers(c), (uint64_t)L.Ts) &&
            map_out_f32(c, &tm_dW, dW, (uint64_t)V, (uint64_t)d, (uint64_t)d, 1, (uint64_t)V);
  if (!ok) return RL_ERR_CUDA;

  const int n_row_slabs = (L.Tpad + L.Ts - 1) / L.Ts;
  const int n_col_slabs = (int)((V + L.Vs - 1) / L.Vs);
  const int d_tiles = (int)((d + BN - 1) / BN);
  for (int r = 0; r < n_row_slabs; ++r) {
    GemmShape dh_shape;
    memset(&dh_shape, 0, sizeof(dh_shape));
    const int rows_cap = L.Ts;   // the valid rows are cut into equal slabs of at most Ts rows on the device
    // stream-K parts that finish a tile are added to the second accumulator buffer: it starts at zero
    if (dh_uses_stream_k(c)) cudaMemsetAsync(dH_acc + (size_t)L.Ts * d, 0, (size_t)L.Ts * d * 4, st);
    for (int cs = 0; cs < n_col_slabs; ++cs) {
      const int vocab_base = cs * L.Vs;
      const int cols = (int)((V - vocab_base) < L.Vs ? (V - vocab_base) : L.Vs);
      // (1) recompute the logits of the slab, write G = dloss/dlogits as bf16
      {
        GemmShape sh;
        memset(&sh, 0, sizeof(sh));
        sh.n_valid = n_valid;
        sh.m_rows_cap = rows_cap; sh.m_dyn = 1; sh.slab_cap = L.Ts; sh.slab_index = r;
        sh.k_cap = (int)d;
        sh.n_tiles = (cols + BN - 1) / BN;
        sh.n_range = 0; sh.n_range_lo = 1; sh.n_range_hi = kFwdRange; sh.n_range_always = 1;   // chosen on the device
        sh.a_mn_slab = 1;
        sh.b_mn_off = vocab_base;
        sh.m_group = row_group_tiles(c, d + (o.kl_full ? o.d_ref : 0));
        if (!o.kl_full) {
          EpiGrad::Params ep;
          ep.tokens_c = reinterpret_cast<const int*>(ws + L.tokens_c);
          ep.lse = p.lse_c; ep.ent = p.ent_c; ep.cp = p.cp_c; ep.ce = p.ce_c;
          ep.V = (int)V; ep.vocab_base = vocab_base;
          launch_gemm<EpiGrad, 0, 0>(c, 1, tmHc_k, tmW_k, tm_G_out, sh, ep);
        } else {
          EpiGradKL::Params ep;
          ep.tokens_c = reinterpret_cast<const int*>(ws + L.tokens_c);
          ep.lse = p.lse_c; ep.lse_ref = p.lse_ref_c; ep.ent = p.ent_c; ep.kl = p.kl_c;
          ep.cp = p.cp_c; ep.cb = p.cb_c; ep.ce = p.ce_c;
          ep.V = (int)V; ep.vocab_base = vocab_base;
          launch_dual<EpiGradKL>(c, 1, tmHc_k, tmW_k, tmHr_k, tmWr_k, tm_G_out, sh, (int)o.d_ref, ep);
        }
      }
      // (2) dH_slab (+)= G * W_slab        [rows x d], K = vocabulary columns of the slab
      {
        GemmShape sh;
        memset(&sh, 0, sizeof(sh));
        sh.n_valid = n_valid;
        sh.m_rows_cap = rows_cap; sh.m_dyn = 1; sh.slab_cap = L.Ts; sh.slab_index = r;
        sh.k_cap = cols;
        sh.n_tiles = d_tiles;
        sh.n_range = 1;
        sh.b_k_off = vocab_base;
        sh.n_fastest = 1;   // the CTAs that share a panel of G rows run together
        sh.k_split_max = c->dh_k_slices;
        sh.stream_k = dh_uses_stream_k(c) ? 1 : 0;
        dh_shape = sh;      // the slice count depends only on rows, d tiles and grid: same for every slab
        EpiAcc::Params ep;
        ep.n_cols = (int)d; ep.accumulate = cs > 0; ep.row_base = 0; ep.slice_add = sh.stream_k;
        if (use_wide(c)) {
          sh.n_tiles = (int)((d + 2 * BN - 1) / (2 * BN));
          dh_shape = sh;
          launch_wide<EpiAcc, 0, 1>(c, 2, tmG_k, tmW_mn, tm_dH, sh, ep);
        } else {
          launch_gemm<EpiAcc, 0, 1>(c, 2, tmG_k, tmW_mn, tm_dH, sh, ep);
        }
      }
      // (3) dW_slab (+)= G^T * H_slab      [vocabulary rows x d], K = valid rows of the slab
      {
        GemmShape sh;
        memset(&sh, 0, sizeof(sh));
        sh.n_valid = n_valid;
        sh.m_rows_cap = cols;
        sh.k_cap = rows_cap; sh.k_dyn = 1; sh.slab_cap = L.Ts; sh.slab_index = r;
        sh.n_tiles = d_tiles;
        sh.n_range = 1;
        sh.skip_if_k0 = (r > 0 || o.accumulate_dW) ? 1 : 0;
        sh.b_k_slab = 1;
        sh.n_fastest = 1;
        EpiAcc::Params ep;
        ep.n_cols = (int)d; ep.accumulate = (r > 0 || o.accumulate_dW) ? 1 : 0;
        ep.row_base = vocab_base; ep.slice_add = 0;
        if (use_wide(c)) {
          sh.n_tiles = (int)((d + 2 * BN - 1) / (2 * BN));
          launch_wide<EpiAcc, 1, 1>(c, 3, tmG_mn, tmHc_mn, tm_dW, sh, ep);
        } else {
          launch_gemm<EpiAcc, 1, 1>(c, 3, tmG_mn, tmHc_mn, tm_dW, sh, ep);
        }
        // rows [vocab_base, vocab_base + cols) of dW are complete once the last row slab has added to them
        if (c->dw_hook && r == n_row_slabs - 1) c->dw_hook(c->dw_hook_user, cs, vocab_base, (int64_t)vocab_base + cols);
      }
    }
    const int pr_sc = prof_begin(c, 7);
    if (o.dH_dtype)
      scatter_dH_f32_kernel<<<c->n_sm * 4, 256, 0, st>>>(dH_acc, (int)d, dh_shape, c->cta_group,
                                                         c->grid[c->cta_group] / c->cta_group, (long long)L.Ts * d, row_map,
                                                         static_cast<float*>(dH), c->dstatus);
    else
      scatter_dH_kernel<<<c->n_sm * 4, 256, 0, st>>>(dH_acc, (int)d, dh_shape, c->cta_group,
                                                     c->grid[c->cta_group] / c->cta_group, (long long)L.Ts * d, row_map,
                                                     static_cast<__nv_bfloat16*>(dH), c->dstatus);
    prof_end(c, pr_sc, 7);
    c->launches++;
  }
  return cuda_ok();
}

rl_status rl_policy_loss_fwd_bwd_ex(rl_ctx* c, const void* H, int64_t ldH, const void* W, int64_t ldW,
                                    const int32_t* tokens, const float* old_logp, const float* ref_logp,
                                    const float* adv, const uint8_t* mask, int64_t T, int64_t d, int64_t V,
                                    float eps_low, float eps_high, float beta, float* loss, void* dH, float* dW,
                                    const rl_loss_opts* opts) {
  return loss_fwd_bwd_impl(c, H, ldH, W, ldW, tokens, old_logp, ref_logp, adv, mask, T, d, V, eps_low, eps_high, beta,
                           loss, dH, dW, opts, nullptr);
}

rl_status rl_policy_loss_shard_bwd(rl_ctx* c, const void* H, int64_t ldH, const void* W_shard, int64_t ldW,
                                   const int32_t* tokens, const float* old_logp, const float* ref_logp,
                                   const float* adv, const uint8_t* mask, int64_t T, int64_t d, int64_t V_shard,
                                   int64_t vocab_offset, int64_t V_total, const float* logp, const float* entropy,
                                   const float* lse, float eps_low, float eps_high, float beta, float* loss,
                                   void* dH_partial, float* dW_shard, const rl_loss_opts* opts) {
  ShardArgs sh;
  sh.vocab_off = vocab_offset;
  sh.V_total = V_total;
  sh.logp = logp;
  sh.entropy = entropy;
  sh.lse = lse;
  return loss_fwd_bwd_impl(c, H, ldH, W_shard, ldW, tokens, old_logp, ref_logp, adv, mask, T, d, V_shard, eps_low,
                           eps_high, beta, loss, dH_partial, dW_shard, opts, &sh);
}

rl_status rl_shard_logit_stats(rl_ctx* c, const void* H, int64_t ldH, const void* W_shard, int64_t ldW,
                               const int32_t* tokens, const uint8_t* mask, int64_t T, int64_t d, int64_t V_shard,
                               int64_t vocab_offset, int64_t V_total, float* stats) {
  if (!c) return RL_ERR_INVALID_ARG;
  rl_status s = check_hw(H, ldH, W_shard, ldW, T, d, V_shard);
  if (s != RL_OK) return s;
  if (vocab_offset < 0 || V_total < vocab_offset + V_shard || V_total >= (int64_t(1) << 30)) return RL_ERR_SHAPE;
  if (T == 0) return RL_OK;
  if (!tokens || !stats) return RL_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(stats) & 15) return RL_ERR_ALIGNMENT;
  const WsLayout L = ws_layout(c, T, d, V_shard, false);
  if ((s = check_ws(c, L)) != RL_OK) return s;
  char* ws = static_cast<char*>(c->ws);
  cudaMemsetAsync(stats, 0, (size_t)T * 16, c->stream);
  GemmShape fwd_shape;
  FwdPlan plan;
  plan.vocab_off = vocab_offset;
  plan.V_total = V_total;
  if ((s = run_forward(c, L, H, ldH, W_shard, ldW, tokens, mask, T, d, V_shard, &fwd_shape, nullptr, plan)) != RL_OK)
    return s;
  LossParams p;
  memset(&p, 0, sizeof(p));
  p.partials = reinterpret_cast<const float4*>(ws + L.partials);
  p.part_stride = L.Tpad;
  p.fwd_shape = fwd_shape;
  p.fwd_cg = c->cta_group;
  p.fwd_workers = c->grid[c->cta_group] / c->cta_group;
  p.row_map = reinterpret_cast<const int*>(ws + L.row_map);
  p.stats_out = reinterpret_cast<float4*>(stats);
  int blocks = (int)((T + kLossThreads - 1) / kLossThreads);
  if (blocks > 1024) blocks = 1024;
  const int pr = prof_begin(c, 6);
  combine_loss_kernel<<<blocks, kLossThreads, 0, c->stream>>>(p, c->dstatus);
  prof_end(c, pr, 6);
  c->launches++;
  return cuda_ok();
}

rl_status rl_merge_logit_stats(rl_ctx* c, const float* stats, int n_shards, const uint8_t* mask, int64_t T,
                               float* logp, float* entropy, float* lse) {
  if (!c || T < 0 || n_shards < 1 || n_shards > 4096) return RL_ERR_INVALID_ARG;
  if (T == 0) return RL_OK;
  if (!stats || !logp) return RL_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(stats) & 15) return RL_ERR_ALIGNMENT;
  int blocks = (int)((T + 255) / 256);
  if (blocks > 4096) blocks = 4096;
  const int pr = prof_begin(c, 6);
  merge_shard_stats_kernel<<<blocks, 256, 0, c->stream>>>(reinterpret_cast<const float4*>(stats), n_shards,
                                                          (long long)T, mask, logp, entropy, lse);
  prof_end(c, pr, 6);
  c->launches++;
  return cuda_ok();
}

rl_status rl_token_logprobs_multi(rl_ctx* c, int n_models, const void* const* H, const int64_t* ldH,
                                  const void* const* W, const int64_t* ldW, const int64_t* d,
                                  const int32_t* tokens, const uint8_t* mask, int64_t T, int64_t V,
                                  float* const* logp, float* const* entropy) {
  if (!c || n_models < 1 || n_models > 16 || !H || !ldH || !W || !ldW || !d || !logp) return RL_ERR_INVALID_ARG;
  int64_t d_max = 0;
  for (int i = 0; i < n_models; ++i) {
    rl_status s = check_hw(H[i], ldH[i], W[i], ldW[i], T, d[i], V);
    if (s != RL_OK) return s;
    if (T > 0 && !logp[i]) return RL_ERR_INVALID_ARG;
    d_max = d[i] > d_max ? d[i] : d_max;
  }
  if (T == 0) return RL_OK;
  if (!tokens) return RL_ERR_INVALID_ARG;
  // one layout for all models: the compacted rows of the widest model fix the offsets
  const WsLayout L = ws_layout(c, T, d_max, V, false);
  rl_status s = check_ws(c, L);
  if (s != RL_OK) return s;
  char* ws = static_cast<char*>(c->ws);
  for (int i = 0; i < n_models; ++i) {
    cudaMemsetAsync(logp[i], 0, (size_t)T * 4, c->stream);
    if (entropy && entropy[i]) cudaMemsetAsync(entropy[i], 0, (size_t)T * 4, c->stream);
    GemmShape fwd_shape;
    FwdPlan plan;
    plan.scan = i == 0;   // the mask is scanned once; every model reuses the row map
    if ((s = run_forward(c, L, H[i], ldH[i], W[i], ldW[i], tokens, mask, T, d[i], V, &fwd_shape, nullptr, plan)) != RL_OK)
      return s;
    LossParams p;
    memset(&p, 0, sizeof(p));
    p.partials = reinterpret_cast<const float4*>(ws + L.partials);
    p.part_stride = L.Tpad;
    p.fwd_shape = fwd_shape;
    p.fwd_cg = c->cta_group;
    p.fwd_workers = c->grid[c->cta_group] / c->cta_group;
    p.row_map = reinterpret_cast<const int*>(ws + L.row_map);
    p.lse_c = reinterpret_cast<float*>(ws + L.lse_c);
    p.ent_c = reinterpret_cast<float*>(ws + L.ent_c);
    p.logp_out = logp[i];
    p.ent_out = entropy ? entropy[i] : nullptr;
    int blocks = (int)((T + kLossThreads - 1) / kLossThreads);
    if (blocks > 1024) blocks = 1024;
    combine_loss_kernel<<<blocks, kLossThreads, 0, c->stream>>>(p, c->dstatus);
    c->launches++;
  }
  return cuda_ok();
}

rl_status rl_policy_loss_fwd_bwd(rl_ctx* c, const void* H, int64_t ldH, const void* W, int64_t ldW,
                                 const int32_t* tokens, const float* old_logp, const float* ref_logp,
                                 const float* adv, const uint8_t* mask, int64_t T, int64_t d, int64_t V,
                                 float eps_low, float eps_high, float beta, float* loss, void* dH, float* dW) {
  return rl_policy_loss_fwd_bwd_ex(c, H, ldH, W, ldW, tokens, old_logp, ref_logp, adv, mask, T, d, V, eps_low,
                                   eps_high, beta, loss, dH, dW, nullptr);
}

// Arguments of one host-buffer step (all per-step inputs are host pointers).
struct HostStepArgs {
  const void* H_host;
  int64_t ldH;
  const void* W;
  int64_t ldW;
  const int32_t* tokens_host;
  const float *old_host, *ref_host, *adv_host, *rewards_host;
  int64_t n_seq;
  int group_size;
  const int32_t* seq_offsets_host;
  const uint8_t* mask_host;
  int64_t T, d, V;
  float eps_low, eps_high, beta, ent_coef;
  void* dH;
  float* dW;
};

static rl_status host_step_check(const rl_ctx* c, const HostStepArgs& a) {
  if (!c) return RL_ERR_INVALID_ARG;
  if (a.T < 0 || a.d <= 0 || a.V <= 0) return RL_ERR_INVALID_ARG;
  if (a.T > 0 && (!a.H_host || !a.tokens_host || !a.old_host)) return RL_ERR_INVALID_ARG;
  if (a.T > 0 && !a.adv_host && (!a.rewards_host || !a.seq_offsets_host || a.n_seq <= 0 || a.n_seq > a.T))
    return RL_ERR_INVALID_ARG;
  if (a.ldH != a.d) return RL_ERR_SHAPE;  // host rows are copied as one block
  // everything the advantage and loss calls would refuse is refused here, before a copy is enqueued
  if (a.d % 64 != 0 || a.ldW < a.d || a.T >= (int64_t(1) << 30) || a.V >= (int64_t(1) << 30)) return RL_ERR_SHAPE;
  if (a.ldW % 8 != 0 || (reinterpret_cast<uintptr_t>(a.W) & 15) || (reinterpret_cast<uintptr_t>(a.dH) & 15) ||
      (reinterpret_cast<uintptr_t>(a.dW) & 15))
    return RL_ERR_ALIGNMENT;
  if (!a.W || !a.dW || (a.T > 0 && !a.dH)) return RL_ERR_INVALID_ARG;
  if (!(a.eps_low >= 0.f && a.eps_low < 1.f) || !(a.eps_high >= 0.f) || !(a.beta >= 0.f) || !(a.ent_coef >= 0.f))
    return RL_ERR_INVALID_ARG;
  if (a.beta != 0.f && a.T > 0 && !a.ref_host) return RL_ERR_INVALID_ARG;
  if (a.T > 0 && !a.adv_host && (a.group_size < 2 || a.n_seq % a.group_size != 0)) return RL_ERR_SHAPE;
  return RL_OK;
}

// Copies the step's inputs into the stage on `copy` (the context's stream itself, or the copy stream, in
// which case the context's stream waits for copy_done) and enqueues advantages + loss forward/backward on
// the context's stream; the result words end up in hs.out.
static rl_status host_step_enqueue(rl_ctx* c, const HostStage& hs, cudaStream_t copy, cudaEvent_t copy_done,
                                   const HostStepArgs& a) {
  const int64_t T = a.T;
  if (T > 0) {
    cudaMemcpyAsync(hs.H, a.H_host, (size_t)T * a.d * 2, cudaMemcpyHostToDevice, copy);
    cudaMemcpyAsync(hs.tok, a.tokens_host, (size_t)T * 4, cudaMemcpyHostToDevice, copy);
    cudaMemcpyAsync(hs.old_lp, a.old_host, (size_t)T * 4, cudaMemcpyHostToDevice, copy);
    if (a.ref_host) cudaMemcpyAsync(hs.ref_lp, a.ref_host, (size_t)T * 4, cudaMemcpyHostToDevice, copy);
    if (a.adv_host) {
      cudaMemcpyAsync(hs.adv, a.adv_host, (size_t)T * 4, cudaMemcpyHostToDevice, copy);
    } else {
      cudaMemcpyAsync(hs.rew, a.rewards_host, (size_t)a.n_seq * 4, cudaMemcpyHostToDevice, copy);
      cudaMemcpyAsync(hs.off, a.seq_offsets_host, (size_t)(a.n_seq + 1) * 4, cudaMemcpyHostToDevice, copy);
    }
    if (a.mask_host) cudaMemcpyAsync(hs.mask, a.mask_host, (size_t)T, cudaMemcpyHostToDevice, copy);
  }
  if (copy != c->stream) {
    if (cudaEventRecord(copy_done, copy) != cudaSuccess || cudaStreamWaitEvent(c->stream, copy_done, 0) != cudaSuccess)
      return RL_ERR_CUDA;
  }
  if (T > 0 && !a.adv_host) {
    rl_status sa = rl_grpo_advantages_ex(c, hs.rew, a.n_seq, a.group_size, 1, 1e-6f, hs.off, T, hs.advseq, hs.adv);
    if (sa != RL_OK) return sa;
  }
  rl_loss_opts opts;
  memset(&opts, 0, sizeof(opts));
  opts.struct_size = sizeof(opts);
  opts.ent_coef = a.ent_coef;
  opts.metrics_out = hs.out + 8;
  return rl_policy_loss_fwd_bwd_ex(c, hs.H, a.d, a.W, a.ldW, hs.tok, hs.old_lp, a.ref_host ? hs.ref_lp : nullptr, hs.adv,
                                   a.mask_host ? hs.mask : nullptr, T, a.d, a.V, a.eps_low, a.eps_high, a.beta, hs.out,
                                   a.dH, a.dW, &opts);
}

rl_status rl_policy_loss_fwd_bwd_host(rl_ctx* c, const void* H_host, int64_t ldH, const void* W, int64_t ldW,
                                      const int32_t* tokens_host, const float* old_host, const float* ref_host,
                                      const float* adv_host, const float* rewards_host, int64_t n_seq,
                                      int group_size, const int32_t* seq_offsets_host,
                                      const uint8_t* mask_host, int64_t T, int64_t d,
                                      int64_t V, float eps_low, float eps_high, float beta, float ent_coef,
                                      float* loss_host, float* metrics_host, void* dH, float* dW) {
  if (!loss_host) return RL_ERR_INVALID_ARG;
  const HostStepArgs a = {H_host, ldH, W, ldW, tokens_host, old_host, ref_host, adv_host, rewards_host, n_seq, group_size,
                          seq_offsets_host, mask_host, T, d, V, eps_low, eps_high, beta, ent_coef, dH, dW};
  rl_status s = host_step_check(c, a);
  if (s != RL_OK) return s;
  const WsLayout L = ws_layout(c, T, d, V, 1);
  if ((s = check_ws(c, L)) != RL_OK) return s;
  HostStage hs;
  carve_stage(static_cast<char*>(c->ws) + L.staging, T, d, &hs);
  if ((s = host_step_enqueue(c, hs, c->stream, nullptr, a)) != RL_OK) return s;
  float h_out[16];
  if (cudaMemcpyAsync(h_out, hs.out, sizeof(h_out), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess) return RL_ERR_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return RL_ERR_CUDA;
  loss_host[0] = h_out[0];
  if (metrics_host) memcpy(metrics_host, h_out + 8, 32);
  return RL_OK;
}

rl_status rl_workspace_bytes_host_pipelined(rl_ctx* c, int64_t T, int64_t d, int64_t V, size_t* bytes) {
  if (!c || !bytes || T < 0 || d <= 0 || V <= 0) return RL_ERR_INVALID_ARG;
  *bytes = ws_layout(c, T, d, V, 2).total;
  return RL_OK;
}

rl_status rl_policy_loss_fwd_bwd_host_submit(rl_ctx* c, int slot, const void* H_host, int64_t ldH, const void* W,
                                             int64_t ldW, const int32_t* tokens_host, const float* old_host,
                                             const float* ref_host, const float* adv_host,
                                             const float* rewards_host, int64_t n_seq, int group_size,
                                             const int32_t* seq_offsets_host, const uint8_t* mask_host, int64_t T,
                                             int64_t d, int64_t V, float eps_low, float eps_high, float beta,
                                             float ent_coef, void* dH, float* dW) {
  const HostStepArgs a = {H_host, ldH, W, ldW, tokens_host, old_host, ref_host, adv_host, rewards_host, n_seq, group_size,
                          seq_offsets_host, mask_host, T, d, V, eps_low, eps_high, beta, ent_coef, dH, dW};
  rl_status s = host_step_check(c, a);
  if (s != RL_OK) return s;
  if (slot < 0 || slot > 1 || c->slot_busy[slot]) return RL_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(c, T, d, V, 2);
  if ((s = check_ws(c, L)) != RL_OK) return s;
  if (!c->copy_stream) {
    // first pipelined call on this context: the copy stream, two events and 64 pinned bytes per slot;
    // all of it or none of it, so that a later call never finds a half-made set
    cudaStream_t cs = nullptr;
    cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
    float* pin[2] = {nullptr, nullptr};
    bool ok = cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < 4 && ok; ++i) ok = cudaEventCreateWithFlags(&ev[i], cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
      ok = cudaHostAlloc(reinterpret_cast<void**>(&pin[i]), 64, cudaHostAllocDefault) == cudaSuccess;
    if (!ok) {
      for (int i = 0; i < 2; ++i) if (pin[i]) cudaFreeHost(pin[i]);
      for (int i = 0; i < 4; ++i) if (ev[i]) cudaEventDestroy(ev[i]);
      if (cs) cudaStreamDestroy(cs);
      cudaGetLastError();
      return RL_ERR_CUDA;
    }
    for (int i = 0; i < 2; ++i) { c->copy_done[i] = ev[2 * i]; c->step_done[i] = ev[2 * i + 1]; c->pinned_out[i] = pin[i]; }
    c->copy_stream = cs;
  }
  HostStage hs;
  const size_t stage = carve_stage(nullptr, T, d, nullptr);
  carve_stage(static_cast<char*>(c->ws) + L.staging + (size_t)slot * stage, T, d, &hs);
  // the stage of this slot is free: its previous step was waited for (slot_busy is clear)
  if ((s = host_step_enqueue(c, hs, c->copy_stream, c->copy_done[slot], a)) != RL_OK) return s;
  if (cudaMemcpyAsync(c->pinned_out[slot], hs.out, 64, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
      cudaEventRecord(c->step_done[slot], c->stream) != cudaSuccess)
    return RL_ERR_CUDA;
  c->slot_busy[slot] = 1;
  return RL_OK;
}

rl_status rl_policy_loss_fwd_bwd_host_wait(rl_ctx* c, int slot, float* loss_host, float* metrics_host) {
  if (!c || slot < 0 || slot > 1 || !loss_host || !c->slot_busy[slot]) return RL_ERR_INVALID_ARG;
  if (cudaEventSynchronize(c->step_done[slot]) != cudaSuccess) return RL_ERR_CUDA;
  c->slot_busy[slot] = 0;
  loss_host[0] = c->pinned_out[slot][0];
  if (metrics_host) memcpy(metrics_host, c->pinned_out[slot] + 8, 32);
  return RL_OK;
}

rl_status rl_debug_schedule(int64_t n_valid, int64_t rows_cap, int64_t k_len, int64_t n_tiles, int n_range,
                            int n_fastest, int m_group, int stream_k, int k_split_max, int cta_group,
                            int n_workers, int32_t* units, int64_t max_units, int64_t* n_units) {
  if (!n_units || n_valid < 0 || rows_cap <= 0 || k_len < 0 || n_tiles <= 0 || n_workers <= 0 || max_units < 0 ||
      (cta_group != 1 && cta_group != 2) || (max_units > 0 && !units))
    return RL_ERR_INVALID_ARG;
  const int nv = (int)n_valid;
  GemmShape sh;
  memset(&sh, 0, sizeof(sh));
  sh.n_valid = &nv;
  sh.m_rows_cap = (int)rows_cap;
  sh.m_dyn = 1;
  sh.k_cap = (int)k_len;
  sh.n_tiles = (int)n_tiles;
  if (n_range >= 0) {
    sh.n_range = n_range;
  } else if (n_range > -100) {   // as the gradient-of-the-logits pass: always chosen in [1, -n_range]
    sh.n_range_lo = 1; sh.n_range_hi = -n_range; sh.n_range_always = 1;
  } else {                       // as the forward pass: chosen in [8, -n_range - 100] when there is plenty of work
    sh.n_range_lo = kFwdRange; sh.n_range_hi = -n_range - 100;
  }
  sh.n_fastest = n_fastest;
  sh.m_group = m_group;
  sh.stream_k = stream_k;
  sh.k_split_max = k_split_max;
  const GemmExtents ex = gemm_extents(sh, nv, cta_group, n_workers);
  int64_t n = 0;
  for (int worker = 0; worker < n_workers; ++worker) {
    UnitWalk walk(sh, ex, worker, n_workers);
    int mu, nr, ks, kb0, kb1;
    while (walk.next(mu, nr, ks, kb0, kb1)) {
      if (n < max_units) {
        int32_t* o = units + n * 8;
        o[0] = worker; o[1] = mu; o[2] = nr * ex.n_range;
        o[3] = (nr + 1) * ex.n_range < sh.n_tiles ? (nr + 1) * ex.n_range : sh.n_tiles;
        o[4] = ks; o[5] = kb0; o[6] = kb1; o[7] = ex.k_blocks;
      }
      ++n;
    }
  }
  *n_units = n;
  return RL_OK;
}

rl_status rl_selftest_wait_timeout(rl_ctx* c, int limit_ms) {
  if (!c || limit_ms < 1 || limit_ms > 1000) return RL_ERR_INVALID_ARG;
  wait_timeout_probe_kernel<<<1, 32, 0, c->stream>>>((unsigned long long)limit_ms * 1000000ull, c->dstatus);
  c->launches++;
  return cuda_ok();
}

rl_status rl_selftest_cluster_exchange(rl_ctx* c, int mode, int cluster_size, int iters, int bytes, int partner_xor,
                                       float* ms_host, int* n_clusters_host) {
  if (!c || !ms_host || (mode != 0 && mode != 1) || iters < 1 || iters > (1 << 20)) return RL_ERR_INVALID_ARG;
  if (cluster_size != 2 && cluster_size != 4 && cluster_size != 8) return RL_ERR_INVALID_ARG;
  size_t smem = 1024;
  if (mode == 0) {
    smem += (size_t)kProbeTile * kProbeTile * 6;
  } else {
    if (bytes < 16 || bytes % 16 != 0 || bytes > 48 * 1024 || partner_xor < 1 || partner_xor >= cluster_size)
      return RL_ERR_INVALID_ARG;
    smem += 4 * (size_t)bytes;
  }
  if (cudaFuncSetAttribute(cluster_exchange_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return RL_ERR_CUDA;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(c->n_sm / cluster_size * cluster_size);
  cfg.blockDim = dim3(kProbeThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = cluster_size;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  int n_clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&n_clusters, cluster_exchange_kernel, &cfg) != cudaSuccess || n_clusters < 1) {
    cudaGetLastError();
    return RL_ERR_UNSUPPORTED_ARCH;
  }
  if (n_clusters * cluster_size < (int)cfg.gridDim.x) cfg.gridDim = dim3(n_clusters * cluster_size);
  if (n_clusters_host) *n_clusters_host = (int)cfg.gridDim.x / cluster_size;
  float* sink = reinterpret_cast<float*>(reinterpret_cast<char*>(c->dstatus) + 128);   // never written in practice
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
    if (e0) cudaEventDestroy(e0);
    return RL_ERR_CUDA;
  }
  rl_status rs = RL_OK;
  for (int pass = 0; pass < 2 && rs == RL_OK; ++pass) {   // one warm-up launch, one timed
    if (pass == 1) cudaEventRecord(e0, c->stream);
    if (cudaLaunchKernelEx(&cfg, cluster_exchange_kernel, mode, iters, bytes, partner_xor, sink, c->dstatus) != cudaSuccess)
      rs = RL_ERR_CUDA;
    c->launches++;
  }
  cudaEventRecord(e1, c->stream);
  if (rs == RL_OK && cudaEventSynchronize(e1) != cudaSuccess) rs = RL_ERR_CUDA;
  if (rs == RL_OK && cudaEventElapsedTime(ms_host, e0, e1) != cudaSuccess) rs = RL_ERR_CUDA;
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  return rs;
}

rl_status rl_selftest_gemm(rl_ctx* c, const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K,
                           int a_mn, int b_mn, int accumulate) {
  if (!c || !A || !B || !C || M <= 0 || N <= 0 || K <= 0) return RL_ERR_INVALID_ARG;
  if (M % 128 != 0 || N % 256 != 0 || K % 8 != 0) return RL_ERR_SHAPE;
  CUtensorMap ta, tb;
  bool ok = a_mn ? map_mnmajor(c, &ta, A, (uint64_t)K, (uint64_t)M, (uint64_t)M, BM / 64)
                 : map_kmajor(c, &ta, A, (uint64_t)M, (uint64_t)K, (uint64_t)K, BM);
  ok = ok && (b_mn ? map_mnmajor(c, &tb, B, (uint64_t)K, (uint64_t)N, (uint64_t)N, b_box_panels(c))
                   : map_kmajor(c, &tb, B, (uint64_t)N, (uint64_t)K, (uint64_t)K, b_box_rows(c)));
  if (!ok) return RL_ERR_CUDA;
  GemmShape sh;
  memset(&sh, 0, sizeof(sh));
  sh.m_rows_cap = (int)M;
  sh.k_cap = (int)K;
  sh.n_tiles = (int)(N / BN);
  sh.n_range = 1;
  sh.n_fastest = 1;   // walk the column tiles of one row panel first, as the gradient passes do
  CUtensorMap tc;
  if (!map_out_f32(c, &tc, C, (uint64_t)M, (uint64_t)N, (uint64_t)N, 1, (uint64_t)M)) return RL_ERR_CUDA;
  EpiAcc::Params ep;
  ep.n_cols = (int)N; ep.accumulate = accumulate; ep.row_base = 0; ep.slice_add = 0;
  if (use_wide(c)) {
    sh.n_tiles = (int)((N + 2 * BN - 1) / (2 * BN));
    if (!a_mn && !b_mn) launch_wide<EpiAcc, 0, 0>(c, -1, ta, tb, tc, sh, ep);
    else if (!a_mn && b_mn) launch_wide<EpiAcc, 0, 1>(c, -1, ta, tb, tc, sh, ep);
    else if (a_mn && !b_mn) launch_wide<EpiAcc, 1, 0>(c, -1, ta, tb, tc, sh, ep);
    else launch_wide<EpiAcc, 1, 1>(c, -1, ta, tb, tc, sh, ep);
  } else if (!a_mn && !b_mn) launch_gemm<EpiAcc, 0, 0>(c, -1, ta, tb, tc, sh, ep);
  else if (!a_mn && b_mn) launch_gemm<EpiAcc, 0, 1>(c, -1, ta, tb, tc, sh, ep);
  else if (a_mn && !b_mn) launch_gemm<EpiAcc, 1, 0>(c, -1, ta, tb, tc, sh, ep);
  else launch_gemm<EpiAcc, 1, 1>(c, -1, ta, tb, tc, sh, ep);
  return cuda_ok();
}

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of rl_token_logprobs.  Its scratch (compacted rows, row map, per-range
// softmax statistics, status word) lives in one file-scope device array instead of a caller
// workspace, so the call path contains no device allocation at all.
namespace {
constexpr size_t kStaticScratchBytes = size_t(16) << 20;   // 16 MiB per GPU that loads the library
constexpr size_t kStaticHeaderBytes = 256;                  // status word, then the workspace proper
constexpr int kStaticMaxDevices = 16;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
struct StaticSlot {
  bool ready;
  rl_ctx ctx;
};
StaticSlot g_static_slot[kStaticMaxDevices];
std::mutex g_static_mutex;
}  // namespace

rl_status rl_token_logprobs_static(void* cuda_stream, const void* H, int64_t ldH, const void* W, int64_t ldW,
                                   const int32_t* tokens, const uint8_t* mask, int64_t T, int64_t d, int64_t V,
                                   float* logp, float* entropy, float* lse, int32_t* dev_status) {
  rl_status s = check_hw(H, ldH, W, ldW, T, d, V);
  if (s != RL_OK) return s;
  if (T > 0 && (!tokens || !logp)) return RL_ERR_INVALID_ARG;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) return RL_ERR_CUDA;
  if (device < 0 || device >= kStaticMaxDevices) return RL_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  StaticSlot& slot = g_static_slot[device];
  if (!slot.ready) {
    // once per device, with that device current: the array's name is only a host-side handle;
    // the address kernels and memsets can use comes from cudaGetSymbolAddress
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return RL_ERR_CUDA;
    if (prop.major != 10) return RL_ERR_UNSUPPORTED_ARCH;
    unsigned char* base = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&base), g_static_scratch) != cudaSuccess || !base)
      return RL_ERR_CUDA;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
      return RL_ERR_CUDA;
    if (set_smem_attr<EpiStats, 0, 0>() != cudaSuccess) return RL_ERR_CUDA;
    rl_ctx& c = slot.ctx;
    memset(&c, 0, sizeof(c));
    c.device = device;
    c.n_sm = prop.multiProcessorCount;
    c.encode = reinterpret_cast<EncodeTiledFn>(fn);
    c.dstatus = reinterpret_cast<DevStatus*>(base);
    c.ws = base + kStaticHeaderBytes;
    c.ws_bytes = kStaticScratchBytes - kStaticHeaderBytes;
    c.slab_rows = kSlabRowsMax;
    c.slab_cols = kSlabColsMax;
    c.cta_group = 1;
    c.dh_k_slices = 1;
    c.dh_stream_k = 0;
    c.wide_tiles = 0;
    c.row_group_bytes = kRowGroupBytes;
    c.grid[1] = c.n_sm;
    slot.ready = true;
  }
  rl_ctx* c = &slot.ctx;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  if (T == 0) {
    // nothing to compute, but the caller's status words must not keep stale contents
    if (dev_status && cudaMemsetAsync(dev_status, 0, 2 * sizeof(int32_t), c->stream) != cudaSuccess) return RL_ERR_CUDA;
    return RL_OK;
  }
  // only the forward part of the workspace layout is needed: everything before the gradient slab
  const WsLayout L = ws_layout(c, T, d, V, false);
  if (L.G > c->ws_bytes) return RL_ERR_WORKSPACE;
  char* ws = static_cast<char*>(c->ws);
  // the array keeps the previous call's contents: the status word and the valid-row count start at zero
  if (cudaMemsetAsync(c->dstatus, 0, sizeof(DevStatus), c->stream) != cudaSuccess) return RL_ERR_CUDA;
  cudaMemsetAsync(logp, 0, (size_t)T * 4, c->stream);
  if (entropy) cudaMemsetAsync(entropy, 0, (size_t)T * 4, c->stream);
  if (lse) cudaMemsetAsync(lse, 0, (size_t)T * 4, c->stream);
  GemmShape fwd_shape;
  if ((s = run_forward(c, L, H, ldH, W, ldW, tokens, mask, T, d, V, &fwd_shape)) != RL_OK) return s;
  LossParams p;
  memset(&p, 0, sizeof(p));
  p.partials = reinterpret_cast<const float4*>(ws + L.partials);
  p.part_stride = L.Tpad;
  p.fwd_shape = fwd_shape;
  p.fwd_cg = c->cta_group;
  p.fwd_workers = c->grid[c->cta_group] / c->cta_group;
  p.row_map = reinterpret_cast<const int*>(ws + L.row_map);
  p.with_loss = 0;
  p.lse_c = reinterpret_cast<float*>(ws + L.lse_c);
  p.ent_c = reinterpret_cast<float*>(ws + L.ent_c);
  p.logp_out = logp;
  p.ent_out = entropy;
  p.lse_out = lse;
  int blocks = (int)((T + kLossThreads - 1) / kLossThreads);
  if (blocks > 1024) blocks = 1024;
  combine_loss_kernel<<<blocks, kLossThreads, 0, c->stream>>>(p, c->dstatus);
  if (dev_status &&
      cudaMemcpyAsync(dev_status, c->dstatus, 2 * sizeof(int32_t), cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess)
    return RL_ERR_CUDA;
  return cuda_ok();
}

}  // extern "C"
