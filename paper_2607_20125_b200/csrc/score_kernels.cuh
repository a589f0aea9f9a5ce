// Scoring half of the one-time classification (Sec. 4.2): per-token cosine similarities between the
// proxy outputs and the reference output (Eq. 3), the squared error of the Spatial proxy, attention
// masses from log-sum-exp differences, then per head the means, the 5th percentile, the score of Eq. 4
// and the label of Eq. 5.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace hc {

constexpr int TOK_COS_SINK = 0, TOK_COS_DUMMY = 1, TOK_COS_SPATIAL = 2, TOK_SQERR = 3, TOK_MASS_FIRST = 4,
              TOK_MASS_LAST = 5, TOK_MASS_SPATIAL = 6, TOK_MASS_REST = 7, TOK_N = 8;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One warp per (token, head).  o: [4][L][H][D] fp32 (reference, Sink, Dummy, Spatial proxy outputs),
// lse: [5][L][H] (same four, then the Spatial proxy restricted to the middle blocks).
// tok: [TOK_N][H][L] per-token quantities.
template <int D>
__global__ void __launch_bounds__(256) token_scores_kernel(const float* __restrict__ o, const float* __restrict__ lse,
                                                           float* __restrict__ tok, int L, int H) {
  const int lane = threadIdx.x & 31;
  const long long warp_id = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const long long n_rows = static_cast<long long>(L) * H;
  if (warp_id >= n_rows) return;
  const size_t pass = static_cast<size_t>(n_rows) * D;
  const float* base = o + static_cast<size_t>(warp_id) * D;
  constexpr int PER = D / 32;
  float ref[PER], dot[3] = {0, 0, 0}, nrm[3] = {0, 0, 0}, nref = 0.f, sq = 0.f;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    ref[i] = base[i * 32 + lane];
    nref += ref[i] * ref[i];
  }
#pragma unroll
  for (int m = 0; m < 3; ++m) {
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const float x = base[(m + 1) * pass + i * 32 + lane];
      dot[m] += x * ref[i];
      nrm[m] += x * x;
      if (m == 2) sq += (x - ref[i]) * (x - ref[i]);
    }
  }
  nref = warp_sum(nref);
  sq = warp_sum(sq);
#pragma unroll
  for (int m = 0; m < 3; ++m) {
    dot[m] = warp_sum(dot[m]);
    nrm[m] = warp_sum(nrm[m]);
  }
  if (lane == 0) {
    const int t = static_cast<int>(warp_id / H), h = static_cast<int>(warp_id - static_cast<long long>(t) * H);
    const size_t hl = static_cast<size_t>(H) * L, at = static_cast<size_t>(h) * L + t;
#pragma unroll
    for (int m = 0; m < 3; ++m) tok[m * hl + at] = dot[m] / fmaxf(sqrtf(nrm[m]) * sqrtf(nref), 1e-12f);
    tok[TOK_SQERR * hl + at] = sq;
    const float l_ref = lse[warp_id];
    const float m_first = __expf(lse[n_rows + warp_id] - l_ref);
    const float m_last = __expf(lse[2 * n_rows + warp_id] - l_ref);
    const float m_near = __expf(lse[3 * n_rows + warp_id] - l_ref);
    const float m_near_mid = __expf(lse[4 * n_rows + warp_id] - l_ref);
    tok[TOK_MASS_FIRST * hl + at] = m_first;
    tok[TOK_MASS_LAST * hl + at] = m_last;
    tok[TOK_MASS_SPATIAL * hl + at] = m_near;
    tok[TOK_MASS_REST * hl + at] = fmaxf(0.f, 1.f - m_first - m_last - m_near_mid);
  }
}

__device__ __forceinline__ uint32_t float_order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float float_from_key(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// k-th smallest (0-based) of v[0..n) by a 4-pass, 8-bit-digit radix select.  Block-wide; result broadcast.
__device__ float block_select(const float* v, int n, int k, uint32_t* hist /* [256] shared */, uint32_t* bcast /* [2] */) {
  uint32_t prefix = 0, mask = 0;
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
      }
    }
    __syncthreads();
    prefix |= bcast[0] << shift;
    mask |= 255u << shift;
    remaining = static_cast<int>(bcast[1]);
    __syncthreads();
  }
  return float_from_key(prefix);
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
__global__ void __launch_bounds__(512) head_decide_kernel(const DecideParams p) {
  __shared__ double red[TOK_N][16];
  __shared__ uint32_t hist[256];
  __shared__ uint32_t bcast[2];
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
  const float lo = block_select(cos_sp, p.L, p.rank_lo, hist, bcast);
  const float hi = block_select(cos_sp, p.L, min(p.rank_lo + 1, p.L - 1), hist, bcast);
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
