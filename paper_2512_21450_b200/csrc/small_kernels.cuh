// O(T) and O(B) kernels around the tensor-core passes: mask scan / row compaction
// (padding-free execution), GRPO advantages, merge of the per-range softmax statistics,
// per-token loss arithmetic with a deterministic two-stage reduction, and the final
// conversion of dH.  All of them are bandwidth- or latency-bound; loads are coalesced and
// vectorised where a row is wide enough to matter.
#pragma once
#include "kl_epilogues.cuh"

namespace rlh {

// ------------------------------------------------------------------------------------------
// Mask scan in three launches: row_map[i] = index of the i-th row with mask != 0 (ascending),
// n_valid = their number.  Each block owns 4096 consecutive rows, each thread 16 of them (one
// 16-byte load when the mask is 16-byte aligned): (1) per-block counts, (2) one block turns the
// counts into exclusive offsets, (3) every block scans its rows again and writes its indices.
constexpr int kScanThreads = 256;
constexpr int kScanRowsPerThread = 16;
constexpr int kScanRowsPerBlock = kScanThreads * kScanRowsPerThread;

// Bit i of the result = (mask[base + i] != 0), rows past T read as 0; mask == NULL means all valid.
__device__ __forceinline__ unsigned scan_load_bits(const uint8_t* __restrict__ mask, long long base, int T) {
  if (base >= T) return 0u;
  const int n = (int)min((long long)kScanRowsPerThread, (long long)T - base);
  if (!mask) return n == 16 ? 0xFFFFu : ((1u << n) - 1u);
  unsigned bits = 0;
  if (n == 16 && ((reinterpret_cast<uintptr_t>(mask + base) & 15) == 0)) {
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(mask + base));
    const unsigned wds[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int w = 0; w < 4; ++w)
#pragma unroll
      for (int b = 0; b < 4; ++b) bits |= ((wds[w] >> (8 * b)) & 0xFFu) ? (1u << (4 * w + b)) : 0u;
  } else {
    for (int i = 0; i < n; ++i) bits |= __ldg(mask + base + i) ? (1u << i) : 0u;
  }
  return bits;
}

__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int u = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += u;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = lane < (int)(blockDim.x >> 5) ? warp_sums[lane] : 0;
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += u;
    }
    warp_sums[lane] = wi - w;
    if (lane == 31 && total) *total = wi;
  }
  __syncthreads();
  return warp_sums[warp] + incl - v;
}

__global__ void __launch_bounds__(kScanThreads) mask_count_kernel(const uint8_t* __restrict__ mask, int T,
                                                                  int* __restrict__ block_counts) {
  __shared__ int warp_sums[32];
  const long long base = ((long long)blockIdx.x * kScanThreads + threadIdx.x) * kScanRowsPerThread;
  int c = __popc(scan_load_bits(mask, base, T));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    int t = 0;
    for (int w = 0; w < kScanThreads / 32; ++w) t += warp_sums[w];
    block_counts[blockIdx.x] = t;
  }
}

// One block: block_counts[0..n) -> exclusive offsets in place, total -> st->n_valid.
__global__ void __launch_bounds__(1024) mask_offsets_kernel(int* __restrict__ block_counts, int n, DevStatus* st) {
  __shared__ int warp_sums[32];
  __shared__ int chunk_total;
  int carry = 0;
  for (int base = 0; base < n; base += 1024) {
    const int i = base + threadIdx.x;
    const int v = i < n ? block_counts[i] : 0;
    const int ex = block_exclusive_scan(v, warp_sums, &chunk_total);
    if (i < n) block_counts[i] = carry + ex;
    carry += chunk_total;
    __syncthreads();
  }
  if (threadIdx.x == 0) st->n_valid = carry;
}

__global__ void __launch_bounds__(kScanThreads) mask_write_kernel(const uint8_t* __restrict__ mask, int T,
                                                                  const int* __restrict__ block_offsets,
                                                                  int* __restrict__ row_map) {
  __shared__ int warp_sums[32];
  __shared__ int block_total;
  __shared__ int staged[kScanRowsPerBlock];   // the block's valid rows, in order
  const long long base = ((long long)blockIdx.x * kScanThreads + threadIdx.x) * kScanRowsPerThread;
  unsigned bits = scan_load_bits(mask, base, T);
  int pos = block_exclusive_scan(__popc(bits), warp_sums, &block_total);
  while (bits) {
    const int i = __ffs(bits) - 1;
    bits &= bits - 1;
    staged[pos++] = (int)base + i;
  }
  __syncthreads();
  // coalesced copy of the block's indices to their place in the map
  int* dst = row_map + block_offsets[blockIdx.x];
  for (int k = threadIdx.x; k < block_total; k += kScanThreads) dst[k] = staged[k];
}

// ------------------------------------------------------------------------------------------
// Row compaction: Hc[i,:] = H[row_map[i],:] for i < n_valid, zero rows up to the next multiple
// of 128 (so that tensor-core tiles never see stale data), compact token ids, and the
// token-range check.  One warp per row, 16-byte loads.  Token ids are checked against the whole
// vocabulary [0, V) and stored relative to vocab_off, the first id of the rows of W this call
// holds (0 unless the head is split by vocabulary): an id outside the held slice becomes a
// negative or too large column that no tile ever matches.
__global__ void __launch_bounds__(256) gather_rows_kernel(const __nv_bfloat16* __restrict__ H, long long ldH, int d,
                                                          const int* __restrict__ row_map,
                                                          const int* __restrict__ tokens, int V, int vocab_off,
                                                          __nv_bfloat16* __restrict__ Hc,
                                                          int* __restrict__ tokens_c, DevStatus* st) {
  const int n = st->n_valid;
  const int n_pad = (n + 127) / 128 * 128;
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  const int vec_per_row = d / 8;
  for (int i = blockIdx.x * warps_per_block + (threadIdx.x >> 5); i < n_pad; i += gridDim.x * warps_per_block) {
    uint4* dst = reinterpret_cast<uint4*>(Hc + (size_t)i * d);
    if (i < n) {
      const int r = row_map[i];
      const uint4* src = reinterpret_cast<const uint4*>(H + (size_t)r * ldH);
      for (int v = lane; v < vec_per_row; v += 32) dst[v] = __ldg(src + v);
      if (lane == 0) {
        const int y = tokens[r];
        const bool in_range = y >= 0 && y < V;
        tokens_c[i] = in_range ? y - vocab_off : -1;
        if (!in_range) latch_status(st, kStatusTokenRange, r);
      }
    } else {
      for (int v = lane; v < vec_per_row; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
      if (lane == 0) tokens_c[i] = -1;
    }
  }
}

// Row compaction of a second hidden-state matrix (the reference model's) with the same row map.
__global__ void __launch_bounds__(256) gather_plain_kernel(const __nv_bfloat16* __restrict__ H, long long ldH, int d,
                                                           const int* __restrict__ row_map,
                                                           __nv_bfloat16* __restrict__ Hc, const DevStatus* st) {
  const int n = st->n_valid;
  const int n_pad = (n + 127) / 128 * 128;
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  const int vec_per_row = d / 8;
  for (int i = blockIdx.x * warps_per_block + (threadIdx.x >> 5); i < n_pad; i += gridDim.x * warps_per_block) {
    uint4* dst = reinterpret_cast<uint4*>(Hc + (size_t)i * d);
    if (i < n) {
      const uint4* src = reinterpret_cast<const uint4*>(H + (size_t)row_map[i] * ldH);
      for (int v = lane; v < vec_per_row; v += 32) dst[v] = __ldg(src + v);
    } else {
      for (int v = lane; v < vec_per_row; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
    }
  }
}

// ------------------------------------------------------------------------------------------
// GRPO advantages (section 4.2 group-based normalisation), warp-shuffle segmented: a warp is cut
// into segments of seg = (smallest power of two >= G, at most 32) lanes, one group of G consecutive
// rewards per segment (a group of more than 32 responses takes a whole warp and strides over it).
// Mean, centred sum of squares (both in double) and the all-equal test are butterfly reductions that
// stay inside the segment.  For power-of-two G a warp reads and writes 128 contiguous bytes.
__global__ void __launch_bounds__(256) grpo_adv_kernel(const float* __restrict__ rewards, int n_groups, int G,
                                                       int ddof, float eps_std, float* __restrict__ adv_seq) {
  int seg = 32;
  while (seg > 1 && (seg >> 1) >= G) seg >>= 1;
  const int groups_per_warp = 32 / seg;
  const int lane = threadIdx.x & 31;
  const int sub = lane & (seg - 1);
  const long long warp_global = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long g = warp_global * groups_per_warp + lane / seg;
  const bool live = g < n_groups;                 // lanes of groups past the end still take part in the shuffles
  const float* r = rewards + (size_t)(live ? g : 0) * G;
  // sums in double: a group whose rewards lie close together has a small sigma, and the rounding of
  // an fp32 mean divided by it would exceed the 1e-6 the advantages are held to
  double sum = 0.0;
  float mx = -CUDART_INF_F, mn = CUDART_INF_F;
  for (int i = sub; i < G && live; i += seg) {
    const float x = r[i];
    sum += (double)x;
    mx = fmaxf(mx, x);
    mn = fminf(mn, x);
  }
  for (int o = seg >> 1; o > 0; o >>= 1) {
    sum += __shfl_xor_sync(0xffffffffu, sum, o);
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
  }
  const double mu = sum / (double)G;
  double ss = 0.0;
  for (int i = sub; i < G && live; i += seg) {
    const double c = (double)r[i] - mu;
    ss = fma(c, c, ss);
  }
  for (int o = seg >> 1; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const double sigma = sqrt(ss / (double)(G - ddof));
  const double inv = (mx == mn) ? 0.0 : 1.0 / (sigma + (double)eps_std);
  for (int i = sub; i < G && live; i += seg)
    adv_seq[(size_t)g * G + i] = (mx == mn) ? 0.f : (float)(((double)r[i] - mu) * inv);
}

// The same arithmetic with one THREAD per group, for batches of many groups whose size is a multiple of four
// (G = 4 * G4 <= 32): a thread reads its group as G4 16-byte words (a warp reads 32 * G * 4 contiguous bytes), keeps
// it in registers and needs no shuffles, so the double-precision mean / variance / square root / reciprocal are
// paid once per group instead of once per lane of a segment.  At 2^20 groups of 8 this is what lets the kernel
// run at memory speed; the shuffle kernel above serves small batches (one warp instruction covers 32 / seg groups,
// which keeps the launch short when there are only a few groups) and every other group size.
template <int G4>
__global__ void __launch_bounds__(256) grpo_adv_rows_kernel(const float4* __restrict__ rewards, int n_groups, int ddof,
                                                            float eps_std, float4* __restrict__ adv_seq) {
  constexpr int G = 4 * G4;
  const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= n_groups) return;
  float x[G];
#pragma unroll
  for (int j = 0; j < G4; ++j) {
    const float4 v = rewards[g * G4 + j];
    x[4 * j] = v.x; x[4 * j + 1] = v.y; x[4 * j + 2] = v.z; x[4 * j + 3] = v.w;
  }
  double sum = 0.0;
  float mx = -CUDART_INF_F, mn = CUDART_INF_F;
#pragma unroll
  for (int i = 0; i < G; ++i) {
    sum += (double)x[i];
    mx = fmaxf(mx, x[i]);
    mn = fminf(mn, x[i]);
  }
  const double mu = sum / (double)G;
  double ss = 0.0;
#pragma unroll
  for (int i = 0; i < G; ++i) {
    const double c = (double)x[i] - mu;
    ss = fma(c, c, ss);
  }
  const double sigma = sqrt(ss / (double)(G - ddof));
  const double inv = (mx == mn) ? 0.0 : 1.0 / (sigma + (double)eps_std);
#pragma unroll
  for (int j = 0; j < G4; ++j) {
    float4 o;
    o.x = (mx == mn) ? 0.f : (float)(((double)x[4 * j] - mu) * inv);
    o.y = (mx == mn) ? 0.f : (float)(((double)x[4 * j + 1] - mu) * inv);
    o.z = (mx == mn) ? 0.f : (float)(((double)x[4 * j + 2] - mu) * inv);
    o.w = (mx == mn) ? 0.f : (float)(((double)x[4 * j + 3] - mu) * inv);
    adv_seq[g * G4 + j] = o;
  }
}

// Other critic-free estimators named in section 4.2 (no formula printed there; readings):
//   est 1 RLOO: A_i = r_i - mean of the other responses of the group
//   est 2 OPO : A_i = r_i - sum_j(len_j r_j) / sum_j(len_j)          (length-weighted baseline)
//   est 3     : c_i = r_i - group mean (first stage of REINFORCE++; batch normalisation follows)
// One warp per group, shuffle reductions.
__global__ void __launch_bounds__(256) group_baseline_kernel(const float* __restrict__ rewards,
                                                             const int* __restrict__ lengths, int n_groups, int G,
                                                             int est, float* __restrict__ adv_seq) {
  const int lane = threadIdx.x & 31;
  const int g = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (g >= n_groups) return;
  const float* r = rewards + (size_t)g * G;
  float sr = 0.f, sl = 0.f, slr = 0.f;
  for (int i = lane; i < G; i += 32) {
    const float x = r[i];
    const float l = (est == 2) ? (float)lengths[(size_t)g * G + i] : 1.f;
    sr += x;
    sl += l;
    slr = fmaf(l, x, slr);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    sr += __shfl_xor_sync(0xffffffffu, sr, o);
    sl += __shfl_xor_sync(0xffffffffu, sl, o);
    slr += __shfl_xor_sync(0xffffffffu, slr, o);
  }
  for (int i = lane; i < G; i += 32) {
    const float x = r[i];
    float a;
    if (est == 1) a = x - (sr - x) / (float)(G - 1);
    else if (est == 2) a = x - (sl > 0.f ? slr / sl : 0.f);
    else a = x - sr / (float)G;
    adv_seq[(size_t)g * G + i] = a;
  }
}

// Batch statistics of c[n] in double, fixed order (one block): stats[0] = mean, stats[1] = population std.
__global__ void __launch_bounds__(1024) batch_stats_kernel(const float* __restrict__ c, long long n,
                                                           double* __restrict__ stats) {
  __shared__ double red[32];
  __shared__ double mean_s;
  double acc = 0.0;
  for (long long i = threadIdx.x; i < n; i += blockDim.x) acc += (double)c[i];
  for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      double t = 0.0;
      for (int w = 0; w < 32; ++w) t += red[w];
      if (pass == 0) { mean_s = t / (double)n; stats[0] = mean_s; }
      else stats[1] = sqrt(t / (double)n);
    }
    __syncthreads();
    if (pass == 0) {
      const double mu = mean_s;
      acc = 0.0;
      for (long long i = threadIdx.x; i < n; i += blockDim.x) { const double dlt = (double)c[i] - mu; acc += dlt * dlt; }
    }
  }
}

__global__ void __launch_bounds__(256) batch_normalise_kernel(float* __restrict__ c, long long n,
                                                              const double* __restrict__ stats, float eps_std) {
  const double mu = stats[0];
  const double inv = 1.0 / (stats[1] + (double)eps_std);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    c[i] = (float)(((double)c[i] - mu) * inv);
}

// Broadcast of the per-response advantage to the rows of the response (outcome supervision).
// The row ranges [seq_offsets[s], seq_offsets[s+1]) are ascending and adjacent, so they partition
// [seq_offsets[0], seq_offsets[n_seq]); rows outside that span get 0.  A block owns
// kBroadcastSweeps * 1024 consecutive rows and walks them in sweeps of 1024; a thread owns four
// consecutive rows per sweep (one 16-byte store when the output is aligned).  It finds the response
// of its first row by binary search in its first sweep and from then on by a galloping search that starts
// at the response it ended the previous sweep in, so the cost per row does not depend on how long
// the responses are and almost all offset reads after the first sweep hit lines the block just used.
constexpr int kBroadcastSweeps = 8;

// Largest s in [s_from, n_seq) with seq_offsets[s] <= t, given seq_offsets[s_from] <= t < seq_offsets[n_seq].
__device__ __forceinline__ int seq_of_row(const int* __restrict__ seq_offsets, int n_seq, int s_from, long long t) {
  int lo = s_from, step = 1;
  while (lo + step < n_seq && seq_offsets[lo + step] <= t) { lo += step; step <<= 1; }
  int hi = min(lo + step, n_seq);        // seq_offsets[lo] <= t < seq_offsets[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (seq_offsets[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

__global__ void __launch_bounds__(256) broadcast_adv_kernel(const float* __restrict__ adv_seq,
                                                            const int* __restrict__ seq_offsets, int n_seq,
                                                            long long T, float* __restrict__ adv_tok) {
  const int first = seq_offsets[0], last = seq_offsets[n_seq];
  const bool vec_ok = (reinterpret_cast<uintptr_t>(adv_tok) & 15) == 0;
  const long long rows_per_block = (long long)kBroadcastSweeps * blockDim.x * 4;
  for (long long b0 = (long long)blockIdx.x * rows_per_block; b0 < T; b0 += (long long)gridDim.x * rows_per_block) {
    int s = -1;                           // response this thread was in last, -1: not searched yet
    for (int sweep = 0; sweep < kBroadcastSweeps; ++sweep) {
      const long long t0 = b0 + ((long long)sweep * blockDim.x + threadIdx.x) * 4;
      if (t0 >= T) break;
      float v[4] = {0.f, 0.f, 0.f, 0.f};
      if (t0 + 3 >= first && t0 < last) {
        const long long t_in = t0 < first ? first : t0;
        if (s < 0) {
          int lo = 0, hi = n_seq;         // seq_offsets[lo] <= t_in < seq_offsets[hi]
          while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (seq_offsets[mid] <= t_in) lo = mid; else hi = mid;
          }
          s = lo;
        } else {
          s = seq_of_row(seq_offsets, n_seq, s, t_in);
        }
        int end = seq_offsets[s + 1];
        float a = adv_seq[s];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const long long t = t0 + i;
          if (t < first || t >= last) continue;
          while (t >= end) { ++s; end = seq_offsets[s + 1]; a = adv_seq[s]; }   // empty ranges are skipped
          v[i] = a;
        }
      }
      if (vec_ok && t0 + 3 < T) {
        *reinterpret_cast<float4*>(adv_tok + t0) = make_float4(v[0], v[1], v[2], v[3]);
      } else {
        for (int i = 0; i < 4 && t0 + i < T; ++i) adv_tok[t0 + i] = v[i];
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Token-level KL reward shaping (section 2.2 "Regularization": the KL-to-reference term applied as
// per-token rewards; the paper prints no formula, reading): every valid token t of a response gets
// the shaped reward r_t = -beta kl_t, its last valid token additionally the response's scalar
// seq_value, and the per-token value is the return-to-go ret_t = r_t + gamma ret_(next valid token).
// kl_t is the signed log-ratio logp - ref (kind 0), exp(delta) - delta - 1 with delta = ref - logp
// (kind 1), or a value handed in (kind 2).  Masked rows get 0 and are not a discount step.
// One warp per response: it walks the response's rows from the end in 32-row chunks aligned to
// 128 bytes, loads kShapeChunks chunks at a time and runs a suffix scan of the linear maps
// x -> v + g x (valid row: g = gamma, v = r_t; masked row: the identity) with shuffles, carrying the
// return of the first valid token of the chunks already done.  Per-token terms in fp32, sums in double.
constexpr int kShapeChunks = 4;

__global__ void __launch_bounds__(256) kl_shaped_returns_kernel(const float* __restrict__ seq_value,
                                                                const float* __restrict__ logp,
                                                                const float* __restrict__ ref_logp,
                                                                const float* __restrict__ kl_tok,
                                                                const uint8_t* __restrict__ mask,
                                                                const int* __restrict__ seq_offsets, int n_seq,
                                                                float beta, float gamma, int kind,
                                                                float* __restrict__ shaped, float* __restrict__ ret) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int sq = blockIdx.x * warps_per_block + (threadIdx.x >> 5); sq < n_seq; sq += gridDim.x * warps_per_block) {
    const int lo = seq_offsets[sq], hi = seq_offsets[sq + 1];
    if (hi <= lo) continue;
    const double R = (double)seq_value[sq];
    double carry = 0.0;            // return-to-go of the first valid token after the chunks done so far
    bool terminal_done = false;    // the last valid token of the response has been found
    const int c_first = lo >> 5;
    for (int c_hi = (hi - 1) >> 5; c_hi >= c_first; c_hi -= kShapeChunks) {
      double r[kShapeChunks];
      bool inside[kShapeChunks], valid[kShapeChunks];
#pragma unroll
      for (int j = 0; j < kShapeChunks; ++j) {
        const int t = (c_hi - j) * 32 + lane;
        inside[j] = (c_hi - j) >= c_first && t >= lo && t < hi;
        valid[j] = inside[j] && (!mask || mask[t] != 0);
        double kl = 0.0;
        if (valid[j]) {
          if (kind == 2) {
            kl = (double)kl_tok[t];
          } else {
            // the difference of two fp32 values is exact in double; the exponential itself is taken in fp32
            // (expm1f keeps small log-ratios accurate to an ulp), the sums below run in double
            const double delta = (double)ref_logp[t] - (double)logp[t];
            const float df = (float)delta;
            kl = kind == 0 ? -delta : (double)expm1f(df) - delta;
          }
        }
        r[j] = -(double)beta * kl;
      }
#pragma unroll
      for (int j = 0; j < kShapeChunks; ++j) {
        const unsigned live = __ballot_sync(0xffffffffu, valid[j]);
        if (!terminal_done && live) {
          if (lane == 31 - __clz(live)) r[j] += R;
          terminal_done = true;
        }
        double g = valid[j] ? (double)gamma : 1.0, v = valid[j] ? r[j] : 0.0;
        if (gamma == 1.f) {
          // no discount: a plain suffix sum
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const double v2 = __shfl_down_sync(0xffffffffu, v, o);
            if (lane + o < 32) v += v2;
          }
        } else {
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const double g2 = __shfl_down_sync(0xffffffffu, g, o);
            const double v2 = __shfl_down_sync(0xffffffffu, v, o);
            if (lane + o < 32) { v = fma(g, v2, v); g *= g2; }
          }
        }
        const double out = fma(g, carry, v);
        carry = __shfl_sync(0xffffffffu, out, 0);
        if (inside[j]) {
          const int t = (c_hi - j) * 32 + lane;
          ret[t] = valid[j] ? (float)out : 0.f;
          if (shaped) shaped[t] = valid[j] ? (float)r[j] : 0.f;
        }
      }
    }
  }
}

// Rows that lie outside every response range, [0, seq_offsets[0]) and [seq_offsets[n_seq], T), get 0.
__global__ void __launch_bounds__(256) zero_outside_ranges_kernel(const int* __restrict__ seq_offsets, int n_seq,
                                                                  long long T, float* __restrict__ a,
                                                                  float* __restrict__ b) {
  const long long first = seq_offsets[0], last = seq_offsets[n_seq];
  const long long n_out = first + (T > last ? T - last : 0);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_out; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i < first ? i : last + (i - first);
    a[t] = 0.f;
    if (b) b[t] = 0.f;
  }
}

// ------------------------------------------------------------------------------------------
// Merge of the per-range statistics and the per-token loss arithmetic (Eq. 6 with the clipped
// surrogate of section 3.1 and the k3 KL-to-reference term).
struct LossParams {
  // inputs
  const float4* partials;
  int part_stride;
  GemmShape fwd_shape;  // shape of the forward pass: together with its grid it fixes the vocabulary split
  int fwd_cg;           // CTAs per row tile of the forward pass
  int fwd_workers;      // grid of the forward pass / fwd_cg
  const int* row_map;
  const float* old_logp;   // [T] original rows; NULL in log-prob-only mode
  const float* ref_logp;   // [T] or NULL
  const float* adv;        // [T]
  const float* token_weight;  // [T] or NULL
  const long long* token_count;   // device scalar or NULL: divisor of the token mean (data-parallel global count)
  float eps_low, eps_high, beta, ent_coef;
  int with_loss;
  // full-distribution KL to the reference policy (two-product forward): second partial per
  // (range, row) = {D, Mr, Sr, 0}; outputs lse_ref, KL_t and the coefficient cb_t = w_t beta
  const float4* partials2;
  int kl_full;
  float* lse_ref_c;
  float* kl_c;
  float* cb_c;
  // compact outputs
  float* lse_c;
  float* ent_c;
  float* logp_c;   // compact log-probabilities, or NULL
  float* cp_c;
  float* ce_c;
  // scattered outputs (original rows), any may be NULL
  float* logp_out;
  float* ent_out;
  float* lse_out;
  float* kl_out;
  // reduction scratch: [gridDim.x][kLossSums] doubles
  double* block_sums;
  // vocabulary-parallel head: stats_out != NULL -> only merge the ranges of this call's slice and
  // write (M, S, A, z_y) per original row; ext_lse != NULL -> the statistics of the whole
  // vocabulary come from the caller ([T], original rows) instead of the partials
  float4* stats_out;
  const float* ext_logp;
  const float* ext_ent;
  const float* ext_lse;
};
constexpr int kLossSums = 8;  // loss, pg, kl, ent, clip, ratio, ratio_max, unused
constexpr int kLossThreads = 256;

// Fixed-order sum of column k of the block partials by one warp: lane l adds blocks l, l + 32, ... in order, then a
// butterfly over the lanes; the order depends on n_blocks alone, so the result is reproducible.
__device__ __forceinline__ double reduce_block_sums(const double* __restrict__ block_sums, int n_blocks, int k) {
  const int lane = threadIdx.x & 31;
  double v = 0.0;
  for (int b = lane; b < n_blocks; b += 32) {
    const double u = block_sums[(size_t)b * kLossSums + k];
    v = (k == 6) ? fmax(v, u) : v + u;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const double u = __shfl_xor_sync(0xffffffffu, v, o);
    v = (k == 6) ? fmax(v, u) : v + u;
  }
  return v;
}


__global__ void __launch_bounds__(kLossThreads) combine_loss_kernel(const LossParams p, DevStatus* st) {
  const int n = st->n_valid;
  const int n_ranges = p.ext_lse ? 0 : gemm_extents(p.fwd_shape, n, p.fwd_cg, p.fwd_workers).n_ranges;
  double acc[kLossSums];
#pragma unroll
  for (int k = 0; k < kLossSums; ++k) acc[k] = 0.0;
  const long long n_mean = p.token_count ? *p.token_count : (long long)n;
  const float w_mean = n_mean > 0 ? (float)(1.0 / (double)n_mean) : 0.f;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    float lse, logp, ent;
    float M = -CUDART_INF_F, S = 0.f, A = 0.f;
    if (p.ext_lse) {
      const int row = p.row_map[i];
      lse = p.ext_lse[row];
      logp = p.ext_logp[row];
      ent = p.ext_ent[row];
    } else {
      for (int r = 0; r < n_ranges; ++r) M = fmaxf(M, p.partials[(size_t)r * p.part_stride + i].x);
      float zy = 0.f;
      for (int r = 0; r < n_ranges; ++r) {
        const float4 q = p.partials[(size_t)r * p.part_stride + i];
        const float sc = exp2f((q.x - M) * kLog2e);
        S = fmaf(q.y, sc, S);
        A = fmaf(q.z, sc, A);
        zy += q.w;
      }
      if (p.stats_out) {
        p.stats_out[p.row_map[i]] = make_float4(M, S, A, zy);
        continue;
      }
      lse = M + logf(S);
      logp = zy - lse;
      ent = lse - A / S;
    }
    float kl = 0.f;
    if (p.kl_full) {
      float Mr = -CUDART_INF_F;
      for (int r = 0; r < n_ranges; ++r) Mr = fmaxf(Mr, p.partials2[(size_t)r * p.part_stride + i].y);
      float D = 0.f, Sr = 0.f;
      for (int r = 0; r < n_ranges; ++r) {
        const float4 q2 = p.partials2[(size_t)r * p.part_stride + i];
        D = fmaf(q2.x, exp2f((p.partials[(size_t)r * p.part_stride + i].x - M) * kLog2e), D);
        Sr = fmaf(q2.z, exp2f((q2.y - Mr) * kLog2e), Sr);
      }
      const float lse_ref = Mr + logf(Sr);
      kl = (A - D) / S - lse + lse_ref;      // sum_j p_j (z_j - zr_j) - lse + lse_ref
      p.lse_ref_c[i] = lse_ref;
      p.kl_c[i] = kl;
    }
    const int row = p.row_map[i];
    if (p.kl_out) p.kl_out[row] = kl;
    p.lse_c[i] = lse;
    p.ent_c[i] = ent;
    if (p.logp_c) p.logp_c[i] = logp;
    if (p.logp_out) p.logp_out[row] = logp;
    if (p.ent_out) p.ent_out[row] = ent;
    if (p.lse_out) p.lse_out[row] = lse;
    if (p.with_loss) {
      const float w = p.token_weight ? p.token_weight[row] : w_mean;
      const float A_t = p.adv[row];
      const float rho = expf(logp - p.old_logp[row]);
      const float clipped = fminf(fmaxf(rho, 1.f - p.eps_low), 1.f + p.eps_high);
      const float su = rho * A_t, sc = clipped * A_t;
      const bool active = su <= sc;          // unclipped branch is the minimum (ties: unclipped)
      const float s = active ? su : sc;
      float k3 = 0.f, dk3 = 0.f;
      if (p.kl_full) {
        k3 = kl;                              // its gradient is applied per vocabulary entry (cb)
        p.cb_c[i] = w * p.beta;
      } else if (p.beta != 0.f) {
        const float delta = p.ref_logp[row] - logp;
        const float ed = expf(delta);
        k3 = ed - delta - 1.f;
        dk3 = 1.f - ed;
      }
      const float dlogp = -(active ? A_t * rho : 0.f) + p.beta * dk3;
      p.cp_c[i] = -w * dlogp;
      p.ce_c[i] = w * p.ent_coef;
      acc[0] += (double)w * (double)(-s + p.beta * k3 - p.ent_coef * ent);
      acc[1] += (double)w * (double)(-s);
      acc[2] += (double)w * (double)k3;
      acc[3] += (double)w * (double)ent;
      acc[4] += active ? 0.0 : (double)w;
      acc[5] += (double)w * (double)rho;
      acc[6] = fmax(acc[6], (double)rho);
    }
  }
  if (!p.with_loss) return;
  __shared__ double red[kLossThreads / 32][kLossSums];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int k = 0; k < kLossSums; ++k) {
    double v = acc[k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double u = __shfl_xor_sync(0xffffffffu, v, o);
      v = (k == 6) ? fmax(v, u) : v + u;
    }
    if (lane == 0) red[warp][k] = v;
  }
  __syncthreads();
  if (threadIdx.x < kLossSums) {
    const int k = threadIdx.x;
    double v = red[0][k];
    for (int w = 1; w < kLossThreads / 32; ++w) v = (k == 6) ? fmax(v, red[w][k]) : v + red[w][k];
    p.block_sums[(size_t)blockIdx.x * kLossSums + k] = v;
  }
}

// ------------------------------------------------------------------------------------------
// The per-token loss arithmetic on its own (Eq. 6 with the clipped surrogate of section 3.1 and the k3
// estimate of the KL term), for a caller that already holds the log-probability and entropy of every
// token: works on the original rows, four consecutive rows per thread (16-byte loads and stores when
// every array is 16-byte aligned), masked rows give zero derivatives.  Same arithmetic, in the same
// order, as combine_loss_kernel applies to the statistics it has merged.
__global__ void __launch_bounds__(256) count_valid_kernel(const uint8_t* __restrict__ mask, long long T,
                                                          unsigned long long* __restrict__ count) {
  unsigned int n = 0;
  const bool vec = (reinterpret_cast<uintptr_t>(mask) & 15) == 0;
  const long long n16 = vec ? T / 16 : 0;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (long long)gridDim.x * blockDim.x) {
    const uint4 m = reinterpret_cast<const uint4*>(mask)[i];
    const unsigned int w[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
      for (int b = 0; b < 4; ++b) n += ((w[k] >> (8 * b)) & 0xffu) != 0u;
  }
  for (long long t = n16 * 16 + (long long)blockIdx.x * blockDim.x + threadIdx.x; t < T;
       t += (long long)gridDim.x * blockDim.x)
    n += mask[t] != 0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
  __shared__ unsigned int red[8];
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = n;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long tot = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += red[w];
    if (tot) atomicAdd(count, tot);   // integer sum: the order of the blocks does not change it
  }
}

struct TokenLossParams {
  const float* logp;
  const float* entropy;       // or NULL: taken as 0
  const float* old_logp;
  const float* ref_logp;      // or NULL (beta == 0)
  const float* adv;
  const uint8_t* mask;        // or NULL: every row valid
  const float* token_weight;  // or NULL: token mean
  const unsigned long long* count;   // divisor of the token mean (valid rows, or the caller's global count) ...
  unsigned long long n_known;        // ... or, when count is NULL, the divisor itself
  long long T;
  float eps_low, eps_high, beta, ent_coef;
  float* dlogp;               // or NULL
  float* dentropy;            // or NULL
  double* block_sums;         // [gridDim.x][kLossSums]
};

template <bool VEC>
__global__ void __launch_bounds__(kLossThreads, 4) token_loss_kernel(const TokenLossParams p) {
  double acc[kLossSums];
#pragma unroll
  for (int k = 0; k < kLossSums; ++k) acc[k] = 0.0;
  const unsigned long long n_mean = p.count ? *p.count : p.n_known;
  const float w_mean = n_mean > 0 ? (float)(1.0 / (double)n_mean) : 0.f;
  const long long n4 = (p.T + 3) / 4;
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n4; q += (long long)gridDim.x * blockDim.x) {
    const long long t0 = q * 4;
    const int nrow = (int)(p.T - t0 < 4 ? p.T - t0 : 4);
    float lp[4], en[4], ol[4], rf[4], av[4], tw[4];
    unsigned int mk[4];
    if (VEC && nrow == 4) {
      const float4 a = *reinterpret_cast<const float4*>(p.logp + t0);
      const float4 b = *reinterpret_cast<const float4*>(p.old_logp + t0);
      const float4 c = *reinterpret_cast<const float4*>(p.adv + t0);
      lp[0] = a.x; lp[1] = a.y; lp[2] = a.z; lp[3] = a.w;
      ol[0] = b.x; ol[1] = b.y; ol[2] = b.z; ol[3] = b.w;
      av[0] = c.x; av[1] = c.y; av[2] = c.z; av[3] = c.w;
      const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
      const float4 e = p.entropy ? *reinterpret_cast<const float4*>(p.entropy + t0) : z;
      const float4 r = p.ref_logp ? *reinterpret_cast<const float4*>(p.ref_logp + t0) : z;
      const float4 w = p.token_weight ? *reinterpret_cast<const float4*>(p.token_weight + t0) : z;
      en[0] = e.x; en[1] = e.y; en[2] = e.z; en[3] = e.w;
      rf[0] = r.x; rf[1] = r.y; rf[2] = r.z; rf[3] = r.w;
      tw[0] = w.x; tw[1] = w.y; tw[2] = w.z; tw[3] = w.w;
      const unsigned int m4 = p.mask ? *reinterpret_cast<const unsigned int*>(p.mask + t0) : 0x01010101u;
#pragma unroll
      for (int i = 0; i < 4; ++i) mk[i] = (m4 >> (8 * i)) & 0xffu;
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const bool in = i < nrow;
        lp[i] = in ? p.logp[t0 + i] : 0.f;
        ol[i] = in ? p.old_logp[t0 + i] : 0.f;
        av[i] = in ? p.adv[t0 + i] : 0.f;
        en[i] = (in && p.entropy) ? p.entropy[t0 + i] : 0.f;
        rf[i] = (in && p.ref_logp) ? p.ref_logp[t0 + i] : 0.f;
        tw[i] = (in && p.token_weight) ? p.token_weight[t0 + i] : 0.f;
        mk[i] = in ? (p.mask ? p.mask[t0 + i] : 1u) : 0u;
      }
    }
    float dl[4], de[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      dl[i] = 0.f;
      de[i] = 0.f;
      if (!mk[i]) continue;
      const float w = p.token_weight ? tw[i] : w_mean;
      const float rho = expf(lp[i] - ol[i]);
      const float clipped = fminf(fmaxf(rho, 1.f - p.eps_low), 1.f + p.eps_high);
      const float su = rho * av[i], sc = clipped * av[i];
      const bool active = su <= sc;          // unclipped branch is the minimum (ties: unclipped)
      const float s = active ? su : sc;
      float k3 = 0.f, dk3 = 0.f;
      if (p.beta != 0.f) {
        const float delta = rf[i] - lp[i];
        const float ed = expf(delta);
        k3 = ed - delta - 1.f;
        dk3 = 1.f - ed;
      }
      const float dlogp = -(active ? av[i] * rho : 0.f) + p.beta * dk3;
      dl[i] = w * dlogp;
      de[i] = -(w * p.ent_coef);
      acc[0] += (double)w * (double)(-s + p.beta * k3 - p.ent_coef * en[i]);
      acc[1] += (double)w * (double)(-s);
      acc[2] += (double)w * (double)k3;
      acc[3] += (double)w * (double)en[i];
      acc[4] += active ? 0.0 : (double)w;
      acc[5] += (double)w * (double)rho;
      acc[6] = fmax(acc[6], (double)rho);
    }
    if (VEC && nrow == 4) {
      if (p.dlogp) *reinterpret_cast<float4*>(p.dlogp + t0) = make_float4(dl[0], dl[1], dl[2], dl[3]);
      if (p.dentropy) *reinterpret_cast<float4*>(p.dentropy + t0) = make_float4(de[0], de[1], de[2], de[3]);
    } else {
      for (int i = 0; i < nrow; ++i) {
        if (p.dlogp) p.dlogp[t0 + i] = dl[i];
        if (p.dentropy) p.dentropy[t0 + i] = de[i];
      }
    }
  }
  __shared__ double red[kLossThreads / 32][kLossSums];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int k = 0; k < kLossSums; ++k) {
    double v = acc[k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double u = __shfl_xor_sync(0xffffffffu, v, o);
      v = (k == 6) ? fmax(v, u) : v + u;
    }
    if (lane == 0) red[warp][k] = v;
  }
  __syncthreads();
  if (threadIdx.x < kLossSums) {
    const int k = threadIdx.x;
    double v = red[0][k];
    for (int w = 1; w < kLossThreads / 32; ++w) v = (k == 6) ? fmax(v, red[w][k]) : v + red[w][k];
    p.block_sums[(size_t)blockIdx.x * kLossSums + k] = v;
  }
}

// Fixed-order sum of the block partials of token_loss_kernel -> loss[1], metrics[8].  One warp per sum.
__global__ void __launch_bounds__(32 * kLossSums) finalize_token_loss_kernel(const double* __restrict__ block_sums,
                                                                             int n_blocks, float* __restrict__ loss,
                                                                             float* __restrict__ metrics,
                                                                             const unsigned long long* __restrict__ count,
                                                                             unsigned long long n_rows_valid_known) {
  const int k = threadIdx.x >> 5;
  const double v = reduce_block_sums(block_sums, n_blocks, k);
  if ((threadIdx.x & 31) != 0) return;
  if (k == 0) loss[0] = (float)v;
  if (metrics) {
    if (k >= 1 && k <= 6) metrics[k - 1] = (float)v;
    if (k == 7) { metrics[6] = (float)(count ? *count : n_rows_valid_known); metrics[7] = 0.f; }
  }
}

// ------------------------------------------------------------------------------------------
// Sequence-aware loss path: aggregation weights that depend on each response's valid length
// (the length normalisation by token weights of section 2.2) and the sequence-level importance
// ratio (the GSPO variant named in section 4.2; reading: rho_i = exp of the mean
// token log-ratio over the valid tokens of response i, used by every token of the response).
// One warp per response; its valid tokens are the compact rows [lo, hi) found by binary search
// in the ascending row map.
struct SeqParams {
  const int* seq_offsets;   // [n_seq + 1] row range of each response
  int n_seq;
  int agg_mode;             // 0 token mean, 1 mean of per-response token means, 2 token sum / (B * L_max)
  int sequence_level;       // 1: sequence-level ratio
  const int* row_map;
  const float* logp_c;
  const float* ent_c;
  const float* old_logp;
  const float* ref_logp;
  const float* adv;
  const float* token_weight;  // overrides agg_mode when not NULL
  float eps_low, eps_high, beta, ent_coef;
  int* l_max;               // device scalar: longest row range
  float* cp_c;
  float* ce_c;
  double* block_sums;       // [gridDim.x][kLossSums]
};

__global__ void __launch_bounds__(1024) seq_lmax_kernel(const int* __restrict__ seq_offsets, int n_seq, int* l_max) {
  __shared__ int red[32];
  int m = 0;
  for (int i = threadIdx.x; i < n_seq; i += blockDim.x) m = max(m, seq_offsets[i + 1] - seq_offsets[i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 32; ++w) m = max(m, red[w]);
    *l_max = m;
  }
}

__device__ __forceinline__ int lower_bound_rows(const int* __restrict__ row_map, int n, int key) {
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (row_map[mid] < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__global__ void __launch_bounds__(kLossThreads) seq_loss_kernel(const SeqParams p, DevStatus* st) {
  const int n = st->n_valid;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int warps_per_block = kLossThreads / 32;
  double acc[kLossSums];
#pragma unroll
  for (int k = 0; k < kLossSums; ++k) acc[k] = 0.0;
  // token mean (agg_mode 0): over the valid rows that lie inside a response range, the ones that take part
  const int n_part = p.agg_mode == 0 ? lower_bound_rows(p.row_map, n, p.seq_offsets[p.n_seq]) -
                                           lower_bound_rows(p.row_map, n, p.seq_offsets[0])
                                     : 0;
  for (int sq = blockIdx.x * warps_per_block + warp; sq < p.n_seq; sq += gridDim.x * warps_per_block) {
    const int lo = lower_bound_rows(p.row_map, n, p.seq_offsets[sq]);
    const int hi = lower_bound_rows(p.row_map, n, p.seq_offsets[sq + 1]);
    const int len = hi - lo;
    if (len <= 0) continue;
    float w_seq = 0.f;
    if (p.agg_mode == 0) w_seq = 1.f / (float)n_part;
    else if (p.agg_mode == 1) w_seq = 1.f / ((float)p.n_seq * (float)len);
    else w_seq = 1.f / ((float)p.n_seq * (float)max(*p.l_max, 1));
    float rho_seq = 1.f, seq_sum = 0.f;
    if (p.sequence_level) {
      float lr = 0.f;
      for (int k = lo + lane; k < hi; k += 32) lr += p.logp_c[k] - p.old_logp[p.row_map[k]];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) lr += __shfl_xor_sync(0xffffffffu, lr, o);
      rho_seq = expf(lr / (float)len);
      const float clipped = fminf(fmaxf(rho_seq, 1.f - p.eps_low), 1.f + p.eps_high);
      for (int k = lo + lane; k < hi; k += 32) {
        const int row = p.row_map[k];
        const float w = p.token_weight ? p.token_weight[row] : w_seq;
        const float A_t = p.adv[row];
        const bool active = rho_seq * A_t <= clipped * A_t;
        seq_sum += active ? w * A_t : 0.f;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) seq_sum += __shfl_xor_sync(0xffffffffu, seq_sum, o);
    }
    for (int k = lo + lane; k < hi; k += 32) {
      const int row = p.row_map[k];
      const float w = p.token_weight ? p.token_weight[row] : w_seq;
      const float A_t = p.adv[row];
      const float logp = p.logp_c[k];
      const float ent = p.ent_c[k];
      const float rho = p.sequence_level ? rho_seq : expf(logp - p.old_logp[row]);
      const float clipped = fminf(fmaxf(rho, 1.f - p.eps_low), 1.f + p.eps_high);
      const float su = rho * A_t, sc = clipped * A_t;
      const bool active = su <= sc;
      const float s = active ? su : sc;
      float k3 = 0.f, dk3 = 0.f;
      if (p.beta != 0.f) {
        const float delta = p.ref_logp[row] - logp;
        const float ed = expf(delta);
        k3 = ed - delta - 1.f;
        dk3 = 1.f - ed;
      }
      // weighted d loss / d logp_t
      const float wdlogp = (p.sequence_level ? -(rho_seq / (float)len) * seq_sum : -(active ? w * A_t * rho : 0.f)) +
                           w * p.beta * dk3;
      p.cp_c[k] = -wdlogp;
      p.ce_c[k] = w * p.ent_coef;
      acc[0] += (double)w * (double)(-s + p.beta * k3 - p.ent_coef * ent);
      acc[1] += (double)w * (double)(-s);
      acc[2] += (double)w * (double)k3;
      acc[3] += (double)w * (double)ent;
      acc[4] += active ? 0.0 : (double)w;
      acc[5] += (double)w * (double)rho;
      acc[6] = fmax(acc[6], (double)rho);
    }
  }
  __shared__ double red[kLossThreads / 32][kLossSums];
#pragma unroll
  for (int k = 0; k < kLossSums; ++k) {
    double v = acc[k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double u = __shfl_xor_sync(0xffffffffu, v, o);
      v = (k == 6) ? fmax(v, u) : v + u;
    }
    if (lane == 0) red[warp][k] = v;
  }
  __syncthreads();
  if (threadIdx.x < kLossSums) {
    const int k = threadIdx.x;
    double v = red[0][k];
    for (int w = 1; w < kLossThreads / 32; ++w) v = (k == 6) ? fmax(v, red[w][k]) : v + red[w][k];
    p.block_sums[(size_t)blockIdx.x * kLossSums + k] = v;
  }
}

// Second stage: fixed-order sum of the block partials -> loss[1] and metrics[8].  One warp per sum.
__global__ void __launch_bounds__(32 * kLossSums) finalize_loss_kernel(const double* __restrict__ block_sums, int n_blocks,
                                                                       float* __restrict__ loss, float* __restrict__ metrics,
                                                                       const DevStatus* st) {
  const int k = threadIdx.x >> 5;
  const double v = reduce_block_sums(block_sums, n_blocks, k);
  if ((threadIdx.x & 31) != 0) return;
  if (k == 0) loss[0] = (float)v;
  if (metrics) {
    if (k >= 1 && k <= 6) metrics[k - 1] = (float)v;
    if (k == 7) { metrics[6] = (float)st->n_valid; metrics[7] = 0.f; }
  }
}

// ------------------------------------------------------------------------------------------
// Vocabulary-parallel head: merge of the per-row statistics (M, S, A, z_y) of the n_shards slices
// of a partition of the vocabulary (stats[s][t], original rows) into the log-probability of the
// sampled token, the entropy and the log-sum-exp over the whole vocabulary.  Rows with mask 0
// get 0.  One thread per row; the slices are visited in order, so the result is reproducible.
__global__ void __launch_bounds__(256) merge_shard_stats_kernel(const float4* __restrict__ stats, int n_shards,
                                                                long long T, const uint8_t* __restrict__ mask,
                                                                float* __restrict__ logp, float* __restrict__ ent,
                                                                float* __restrict__ lse) {
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < T; t += (long long)gridDim.x * blockDim.x) {
    float o_logp = 0.f, o_ent = 0.f, o_lse = 0.f;
    if (!mask || mask[t]) {
      float M = -CUDART_INF_F;
      for (int s = 0; s < n_shards; ++s) M = fmaxf(M, __ldg(&stats[(size_t)s * T + t]).x);
      float S = 0.f, A = 0.f, zy = 0.f;
      for (int s = 0; s < n_shards; ++s) {
        const float4 q = __ldg(&stats[(size_t)s * T + t]);
        const float sc = exp2f((q.x - M) * kLog2e);
        S = fmaf(q.y, sc, S);
        A = fmaf(q.z, sc, A);
        zy += q.w;
      }
      o_lse = M + logf(S);
      o_logp = zy - o_lse;
      o_ent = o_lse - A / S;
    }
    logp[t] = o_logp;
    if (ent) ent[t] = o_ent;
    if (lse) lse[t] = o_lse;
  }
}

// ------------------------------------------------------------------------------------------
// dH of one row slab: fp32 accumulator rows -> bf16 rows of the caller's dH at their original
// positions.  One warp per row.
// The dH pass may have cut K into slices that accumulate in separate buffers, split_stride
// elements apart (same slice count as gemm_extents chose for the pass): summed here in slice order.
__device__ __forceinline__ float4 sum_k_slices(const float4* p, int n_slices, long long split_stride) {
  float4 x = __ldcs(p);
  if (n_slices == 1) return x;
  for (int s = 1; s < n_slices; ++s) {
    const float4 y = __ldcs(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p) + s * split_stride));
    x.x += y.x; x.y += y.y; x.z += y.z; x.w += y.w;
  }
  return x;
}

// Same with an fp32 destination.
__global__ void __launch_bounds__(256) scatter_dH_f32_kernel(const float* __restrict__ acc, int d, const GemmShape dh_shape,
                                                             int dh_cg, int dh_workers, long long split_stride,
                                                             const int* __restrict__ row_map,
                                                             float* __restrict__ dH, const DevStatus* st) {
  int slab_base, rows;
  slab_extent(st->n_valid, dh_shape.slab_cap, dh_shape.slab_index, slab_base, rows);
  // stream-K launches always keep two buffers (the second holds the parts that finished a tile)
  const int n_slices = dh_shape.stream_k ? 2 : gemm_extents(dh_shape, st->n_valid, dh_cg, dh_workers).k_split;
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int i = blockIdx.x * warps_per_block + (threadIdx.x >> 5); i < rows; i += gridDim.x * warps_per_block) {
    const float4* src = reinterpret_cast<const float4*>(acc + (size_t)i * d);
    float4* dst = reinterpret_cast<float4*>(dH + (size_t)row_map[slab_base + i] * d);
    for (int v = lane; v < d / 4; v += 32) dst[v] = sum_k_slices(src + v, n_slices, split_stride);
  }
}

__global__ void __launch_bounds__(256) scatter_dH_kernel(const float* __restrict__ acc, int d, const GemmShape dh_shape,
                                                         int dh_cg, int dh_workers, long long split_stride,
                                                         const int* __restrict__ row_map,
                                                         __nv_bfloat16* __restrict__ dH, const DevStatus* st) {
  int slab_base, rows;
  slab_extent(st->n_valid, dh_shape.slab_cap, dh_shape.slab_index, slab_base, rows);
  // stream-K launches always keep two buffers (the second holds the parts that finished a tile)
  const int n_slices = dh_shape.stream_k ? 2 : gemm_extents(dh_shape, st->n_valid, dh_cg, dh_workers).k_split;
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int i = blockIdx.x * warps_per_block + (threadIdx.x >> 5); i < rows; i += gridDim.x * warps_per_block) {
    // eight elements per lane: two 16-byte loads, one 16-byte store (d is a multiple of 64)
    const float4* src = reinterpret_cast<const float4*>(acc + (size_t)i * d);
    uint4* dst = reinterpret_cast<uint4*>(dH + (size_t)row_map[slab_base + i] * d);
    for (int v = lane; v < d / 8; v += 32) {
      const float4 x = sum_k_slices(src + 2 * v, n_slices, split_stride);
      const float4 y = sum_k_slices(src + 2 * v + 1, n_slices, split_stride);
      __nv_bfloat162 b0 = __floats2bfloat162_rn(x.x, x.y), b1 = __floats2bfloat162_rn(x.z, x.w);
      __nv_bfloat162 b2 = __floats2bfloat162_rn(y.x, y.y), b3 = __floats2bfloat162_rn(y.z, y.w);
      uint4 o;
      o.x = *reinterpret_cast<uint32_t*>(&b0);
      o.y = *reinterpret_cast<uint32_t*>(&b1);
      o.z = *reinterpret_cast<uint32_t*>(&b2);
      o.w = *reinterpret_cast<uint32_t*>(&b3);
      __stcs(dst + v, o);
    }
  }
}

// ------------------------------------------------------------------------------------------
// Exercises the bounded wait: one warp waits on an mbarrier that nothing ever arrives on, with a
// short limit, and must come back with the timeout latched instead of spinning forever.
__global__ void __launch_bounds__(32) wait_timeout_probe_kernel(unsigned long long limit_ns, DevStatus* st) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncwarp();
  volatile int* abort_p = &abort_flag;
  if (threadIdx.x == 0) {
    if (!mbar_wait_bounded(smem_u32(&bar), 0, abort_p, limit_ns)) latch_status(st, kStatusTimeout, 0x70000000);
  }
  __syncwarp();
}

}  // namespace rlh
