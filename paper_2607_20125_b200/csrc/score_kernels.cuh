// Scoring half of the one-time classification (Sec. 4.2): the merges of the attention kernel's partial results
// compute, row by row and in registers, the token-wise cosine similarities between the proxy outputs and the reference
// output (Eq. 3), the squared error of the Spatial proxy and the attention masses (from log-sum-exp differences);
// then per head the means, the 5th percentile, the score of Eq. 4 and the label of Eq. 5.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "attn_kernel.cuh"

namespace hc {

constexpr int TOK_COS_SINK = 0, TOK_COS_DUMMY = 1, TOK_COS_SPATIAL = 2, TOK_SQERR = 3, TOK_MASS_FIRST = 4,
              TOK_MASS_LAST = 5, TOK_MASS_SPATIAL = 6, TOK_MASS_REST = 7, TOK_N = 8;

// Sum over the CHUNKS consecutive lanes that share one query row (CHUNKS = 8 or 16 divides the warp).
template <int CHUNKS>
__device__ __forceinline__ float row_sum(float v) {
#pragma unroll
  for (int o = CHUNKS / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ float cosine(float dot, float na, float nb) { return dot / fmaxf(sqrtf(na) * sqrtf(nb), 1e-12f); }

// Classification, first half: the reference attention (Eq. 2) and the Sink / Dummy proxies from ONE sweep over the keys.
// The sweep is cut into key ranges tagged first block / middle blocks / newest block, every range leaves an unnormalised
// partial result, and this kernel merges them three ways per query row - all ranges -> reference output, first block
// only -> Sink proxy, newest block only -> Dummy proxy - and scores the row while the three outputs are in registers:
// the cosines of Eq. 3 for the two proxies and the masses of the first and newest block.  Only the reference output
// and its log-sum-exp go back to memory (the Spatial proxy's merge needs them).
// parts[first_part .. first_part + n_parts) of a group list (partial slot, tag); a group is one 256-row query pair.
struct ClsPart {
  int32_t slot, tag;  // tag: 0 first block, 1 middle, 2 newest block
};
struct ClsGroup {
  int32_t head, q_start, q_count[2], first_part, n_parts;
};

template <int D>
__global__ void __launch_bounds__(COMBINE_ROWS * (D / 8))
cls_combine_kernel(const ClsGroup* groups, const ClsPart* parts, const float* part_o, const float2* part_ml, float* o_ref,
                   float* lse_ref, float* tok, int n_heads, int block_tokens) {
  constexpr int CHUNKS = D / 8;
  constexpr int BLOCKS_PER_TILE = 128 / COMBINE_ROWS;
  const ClsGroup g = groups[blockIdx.x / (2 * BLOCKS_PER_TILE)];
  const int sub = (blockIdx.x / BLOCKS_PER_TILE) & 1;
  const int r = (blockIdx.x % BLOCKS_PER_TILE) * COMBINE_ROWS + threadIdx.x / CHUNKS;
  const int c = threadIdx.x % CHUNKS;
  const bool valid = r < g.q_count[sub];  // rows past the block's end do the arithmetic on zeros and write nothing
  const ClsPart* pp = parts + g.first_part;
  const int n_parts = valid ? g.n_parts : 0;
  float m[3] = {-INFINITY, -INFINITY, -INFINITY};  // all, first, newest
  for (int i = 0; i < n_parts; ++i) {
    const float mi = part_ml[static_cast<size_t>(pp[i].slot) * 256 + sub * 128 + r].x;
    m[0] = fmaxf(m[0], mi);
    if (pp[i].tag == 0) m[1] = fmaxf(m[1], mi);
    if (pp[i].tag == 2) m[2] = fmaxf(m[2], mi);
  }
  float acc[3][8], l[3] = {0.f, 0.f, 0.f};
#pragma unroll
  for (int k = 0; k < 3; ++k)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[k][j] = 0.f;
  for (int i = 0; i < n_parts; ++i) {
    const size_t row = static_cast<size_t>(pp[i].slot) * 256 + sub * 128 + r;
    const float2 ml = part_ml[row];
    if (ml.x == -INFINITY) continue;
    const float4* src = reinterpret_cast<const float4*>(part_o + row * D + c * 8);
    const float4 a = src[0], b = src[1];
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      const bool in_set = (k == 0) || (k == 1 && pp[i].tag == 0) || (k == 2 && pp[i].tag == 2);
      if (!in_set) continue;
      const float wgt = ex2_approx(ml.x - m[k]);
      l[k] += wgt * ml.y;
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[k][j] += wgt * v[j];
    }
  }
  float dot[2] = {0.f, 0.f}, nrm[3] = {0.f, 0.f, 0.f};
#pragma unroll
  for (int k = 0; k < 3; ++k) {
    const float inv = l[k] > 0.f ? 1.f / l[k] : 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      acc[k][j] *= inv;
      nrm[k] += acc[k][j] * acc[k][j];
      if (k > 0) dot[k - 1] += acc[k][j] * acc[0][j];
    }
  }
#pragma unroll
  for (int k = 0; k < 3; ++k) nrm[k] = row_sum<CHUNKS>(nrm[k]);
  dot[0] = row_sum<CHUNKS>(dot[0]);
  dot[1] = row_sum<CHUNKS>(dot[1]);
  if (!valid) return;
  const int token = g.q_start + sub * 128 + r;
  const size_t idx = static_cast<size_t>(token) * n_heads + g.head;
  float4* dst = reinterpret_cast<float4*>(o_ref + idx * D + c * 8);
  dst[0] = make_float4(acc[0][0], acc[0][1], acc[0][2], acc[0][3]);
  dst[1] = make_float4(acc[0][4], acc[0][5], acc[0][6], acc[0][7]);
  if (c == 0) {
    const float ln2 = 0.6931471805599453f;
    float lse[3];
#pragma unroll
    for (int k = 0; k < 3; ++k) lse[k] = (l[k] > 0.f) ? m[k] * ln2 + __logf(l[k]) : -INFINITY;
    lse_ref[idx] = lse[0];
    const size_t hl = static_cast<size_t>(n_heads) * block_tokens, at = static_cast<size_t>(g.head) * block_tokens + token;
    tok[TOK_COS_SINK * hl + at] = cosine(dot[0], nrm[1], nrm[0]);
    tok[TOK_COS_DUMMY * hl + at] = cosine(dot[1], nrm[2], nrm[0]);
    tok[TOK_MASS_FIRST * hl + at] = __expf(lse[1] - lse[0]);
    tok[TOK_MASS_LAST * hl + at] = __expf(lse[2] - lse[0]);
  }
}

// Classification, second half: the Spatial proxy's band of one query pair is cut into pieces along its key range like
// any other item; this merges the pieces and scores the row against the reference output written by cls_combine_kernel:
// token-wise cosine and squared error (Eq. 3, Eq. 4), the mass inside the neighbourhood and the mass of the rest
// (middle blocks, outside the neighbourhood).  The proxy output itself is never written.
template <int D>
__global__ void __launch_bounds__(COMBINE_ROWS * (D / 8))
proxy_combine_kernel(const ClsGroup* groups, const ClsPart* parts, const float* part_o, const float2* part_ml,
                     const float* part_mid, const float* o_ref, const float* lse_ref, float* tok, int n_heads,
                     int block_tokens) {
  constexpr int CHUNKS = D / 8;
  constexpr int BLOCKS_PER_TILE = 128 / COMBINE_ROWS;
  const ClsGroup g = groups[blockIdx.x / (2 * BLOCKS_PER_TILE)];
  const int sub = (blockIdx.x / BLOCKS_PER_TILE) & 1;
  const int r = (blockIdx.x % BLOCKS_PER_TILE) * COMBINE_ROWS + threadIdx.x / CHUNKS;
  const int c = threadIdx.x % CHUNKS;
  const bool valid = r < g.q_count[sub];
  const ClsPart* pp = parts + g.first_part;
  const int n_parts = valid ? g.n_parts : 0;
  float m = -INFINITY;
  for (int i = 0; i < n_parts; ++i) m = fmaxf(m, part_ml[static_cast<size_t>(pp[i].slot) * 256 + sub * 128 + r].x);
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, l = 0.f, l_mid = 0.f;
  for (int i = 0; i < n_parts; ++i) {
    const size_t row = static_cast<size_t>(pp[i].slot) * 256 + sub * 128 + r;
    const float2 ml = part_ml[row];
    if (ml.x == -INFINITY) continue;
    const float wgt = ex2_approx(ml.x - m);
    l += wgt * ml.y;
    l_mid += wgt * part_mid[row];
    const float4* src = reinterpret_cast<const float4*>(part_o + row * D + c * 8);
    const float4 a = src[0], b = src[1];
    acc[0] += wgt * a.x; acc[1] += wgt * a.y; acc[2] += wgt * a.z; acc[3] += wgt * a.w;
    acc[4] += wgt * b.x; acc[5] += wgt * b.y; acc[6] += wgt * b.z; acc[7] += wgt * b.w;
  }
  const int token = g.q_start + sub * 128 + r;
  const size_t idx = static_cast<size_t>(valid ? token : 0) * n_heads + g.head;
  float ref[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  if (valid) {
    const float4* src = reinterpret_cast<const float4*>(o_ref + idx * D + c * 8);
    const float4 a = src[0], b = src[1];
    ref[0] = a.x; ref[1] = a.y; ref[2] = a.z; ref[3] = a.w; ref[4] = b.x; ref[5] = b.y; ref[6] = b.z; ref[7] = b.w;
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  float dot = 0.f, n_sp = 0.f, n_ref = 0.f, sq = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float x = acc[j] * inv;
    dot += x * ref[j];
    n_sp += x * x;
    n_ref += ref[j] * ref[j];
    sq += (x - ref[j]) * (x - ref[j]);
  }
  dot = row_sum<CHUNKS>(dot);
  n_sp = row_sum<CHUNKS>(n_sp);
  n_ref = row_sum<CHUNKS>(n_ref);
  sq = row_sum<CHUNKS>(sq);
  if (!valid || c != 0) return;
  const float ln2 = 0.6931471805599453f;
  const float l_ref = lse_ref[idx];
  const float lse_sp = (l > 0.f) ? m * ln2 + __logf(l) : -INFINITY;
  const float lse_mid = (l_mid > 0.f) ? m * ln2 + __logf(l_mid) : -INFINITY;
  const size_t hl = static_cast<size_t>(n_heads) * block_tokens, at = static_cast<size_t>(g.head) * block_tokens + token;
  tok[TOK_COS_SPATIAL * hl + at] = cosine(dot, n_sp, n_ref);
  tok[TOK_SQERR * hl + at] = sq;
  tok[TOK_MASS_SPATIAL * hl + at] = __expf(lse_sp - l_ref);
  tok[TOK_MASS_REST * hl + at] =
      fmaxf(0.f, 1.f - tok[TOK_MASS_FIRST * hl + at] - tok[TOK_MASS_LAST * hl + at] - __expf(lse_mid - l_ref));
}

__device__ __forceinline__ uint32_t float_order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float float_from_key(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// k-th smallest (0-based) of v[0..n) by a 4-pass, 8-bit-digit radix select.  Block-wide; result broadcast.
// *n_le receives how many values are <= the result (so the caller can tell whether rank k + 1 holds the same value).
__device__ float block_select(const float* v, int n, int k, uint32_t* hist /* [256] shared */, uint32_t* bcast /* [3] */,
                              uint32_t* n_le) {
  uint32_t prefix = 0, mask = 0, below_total = 0;
  int remaining = k;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      const uint32_t key = float_order_key(v[i]);
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (threadIdx.x < 256) {
      // the digit whose bin holds rank `remaining`: thread d adds up the bins below d (all threads read the same bin
      // at the same time: a broadcast), exactly one thread finds the rank inside its own bin
      uint32_t below = 0;
      for (int d = 0; d < static_cast<int>(threadIdx.x); ++d) below += hist[d];
      const uint32_t rank = static_cast<uint32_t>(remaining);
      if (below <= rank && rank < below + hist[threadIdx.x]) {
        bcast[0] = threadIdx.x;
        bcast[1] = rank - below;
        bcast[2] = below + (shift == 0 ? hist[threadIdx.x] : 0u);  // values of this prefix that sort below (last pass: up to) the digit
      }
    }
    __syncthreads();
    prefix |= bcast[0] << shift;
    mask |= 255u << shift;
    remaining = static_cast<int>(bcast[1]);
    below_total += bcast[2];
    __syncthreads();
  }
  *n_le = below_total;
  return float_from_key(prefix);
}

// Smallest value of v[0..n) that is greater than x (+inf if none).  Block-wide; result broadcast through *slot.
__device__ float block_min_above(const float* v, int n, float x, uint32_t* slot) {
  if (threadIdx.x == 0) *slot = 0xffffffffu;
  __syncthreads();
  uint32_t best = 0xffffffffu;
  const uint32_t kx = float_order_key(x);
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const uint32_t key = float_order_key(v[i]);
    if (key > kx) best = min(best, key);
  }
  for (int off = 16; off > 0; off >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, off));
  if ((threadIdx.x & 31) == 0 && best != 0xffffffffu) atomicMin(slot, best);
  __syncthreads();
  const uint32_t r = *slot;
  __syncthreads();
  return r == 0xffffffffu ? INFINITY : float_from_key(r);
}

struct DecideParams {
  const float* tok;  // [TOK_N][H][L]
  float* scores;     // [H][10]
  int32_t* labels;   // [H]
  int32_t L, H, D;
  int32_t rank_lo;   // floor(0.05 * (L - 1))
  float rank_frac;
  float theta_sink, theta_dummy, theta_spatial, theta_score, gamma;
  int32_t rule;      // 0: cosine rule of Eq. 5; 1: the same cascade on the mean attention masses
  float mass_tau;
};

// One block per head: fixed-order sums (deterministic), percentile by selection, Eq. 4 and Eq. 5.
__global__ void __launch_bounds__(1024) head_decide_kernel(const DecideParams p) {
  __shared__ double red[TOK_N][32];
  __shared__ uint32_t hist[256];
  __shared__ uint32_t bcast[3];
  __shared__ double sums[TOK_N];
  const int h = blockIdx.x;
  const size_t hl = static_cast<size_t>(p.H) * p.L;
  {
    // all per-token quantities in one pass; the order of every sum is fixed by the thread layout alone
    double acc[TOK_N];
#pragma unroll
    for (int q = 0; q < TOK_N; ++q) acc[q] = 0.0;
    const float* v = p.tok + static_cast<size_t>(h) * p.L;
    for (int i = threadIdx.x; i < p.L; i += blockDim.x) {
#pragma unroll
      for (int q = 0; q < TOK_N; ++q) acc[q] += static_cast<double>(v[q * hl + i]);
    }
#pragma unroll
    for (int q = 0; q < TOK_N; ++q) {
      double x = acc[q];
      for (int off = 16; off > 0; off >>= 1) x += __shfl_down_sync(0xffffffffu, x, off);
      if ((threadIdx.x & 31) == 0) red[q][threadIdx.x >> 5] = x;
    }
    __syncthreads();
    if (threadIdx.x < TOK_N) {
      double x = 0.0;
      for (int wp = 0; wp < static_cast<int>(blockDim.x >> 5); ++wp) x += red[threadIdx.x][wp];
      sums[threadIdx.x] = x;
    }
    __syncthreads();
  }
  const float* cos_sp = p.tok + TOK_COS_SPATIAL * hl + static_cast<size_t>(h) * p.L;
  // order statistics rank_lo and rank_lo + 1: one selection, then either the same value again (ties) or the smallest
  // value above it
  uint32_t n_le = 0;
  const float lo = block_select(cos_sp, p.L, p.rank_lo, hist, bcast, &n_le);
  const float above = block_min_above(cos_sp, p.L, lo, bcast);
  const float hi = (p.rank_lo + 1 >= p.L || static_cast<int>(n_le) > p.rank_lo + 1) ? lo : above;
  if (threadIdx.x == 0) {
    const float inv_l = 1.f / static_cast<float>(p.L);
    const float cs = static_cast<float>(sums[TOK_COS_SINK]) * inv_l;
    const float cd = static_cast<float>(sums[TOK_COS_DUMMY]) * inv_l;
    const float csp = static_cast<float>(sums[TOK_COS_SPATIAL]) * inv_l;
    const float p5 = lo + p.rank_frac * (hi - lo);
    const float mse = static_cast<float>(sums[TOK_SQERR] / (static_cast<double>(p.L) * p.D));
    const float score = p5 - p.gamma * mse;
    const float m_first = static_cast<float>(sums[TOK_MASS_FIRST]) * inv_l;
    const float m_last = static_cast<float>(sums[TOK_MASS_LAST]) * inv_l;
    const float m_near = static_cast<float>(sums[TOK_MASS_SPATIAL]) * inv_l;
    int label = 3;
    if (p.rule == 1) {  // mass rule: same order of tests, same >=, a NaN fails every comparison
      if (m_first >= p.mass_tau) label = 0;
      else if (m_last >= p.mass_tau) label = 1;
      else if (m_near >= p.mass_tau) label = 2;
    } else {
      if (cs >= p.theta_sink) label = 0;
      else if (cd >= p.theta_dummy) label = 1;
      else if (csp >= p.theta_spatial && score >= p.theta_score) label = 2;
    }
    p.labels[h] = label;
    float* s = p.scores + h * 10;
    s[0] = cs; s[1] = cd; s[2] = csp; s[3] = p5; s[4] = mse; s[5] = score;
    s[6] = m_first;
    s[7] = m_last;
    s[8] = m_near;
    s[9] = static_cast<float>(sums[TOK_MASS_REST]) * inv_l;
  }
}

}  // namespace hc
