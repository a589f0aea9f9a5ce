// Byte-exact cache movement: append of one block into the monolithic ring and/or the per-archetype
// buffers, the split of the monolithic cache (one launch per cached block), and the export of one
// head's logical content.  All copies move 16-byte chunks; a thread handles a few chunks of K and of V
// so that enough loads are in flight to cover HBM latency.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace hc {

enum : int32_t { CLS_SINK = 0, CLS_DUMMY = 1, CLS_SPATIAL = 2, CLS_GLOBAL = 3, CLS_NONE = -1 };

constexpr int MAX_HEADS = 64;
constexpr int MAX_BLOCKS = 32;

struct RouteParams {
  // source block: [L][H][d] bf16, viewed as 16-byte chunks
  const uint4* src_k;
  const uint4* src_v;
  // destinations (any may be null)
  uint4* mono_k;
  uint4* mono_v;
  uint4* sd_k;  // [N_sink + N_dummy][L][d]
  uint4* sd_v;
  uint4* g_k;   // [N_global][n_blocks * L][d], block slots are a ring
  uint4* g_v;
  uint4* sp_k;  // [N_spatial][cell][slot][frame][token in cell][d]
  uint4* sp_v;
  const int32_t* sp_base;  // [T_f]: n_blocks * F_b * (tokens in earlier cells) + index of the token inside its cell
  const int32_t* sp_nc;    // [T_f]: tokens per frame in the token's cell
  int32_t L, H, chunks;    // chunks = d / 8
  int32_t tokens_per_frame, frames_per_block, n_blocks;
  int32_t slot;            // destination ring slot
  int32_t n_sink;
  int32_t copy_mono, copy_sink, copy_dummy, copy_window;
  int8_t cls[MAX_HEADS];   // archetype per original head (CLS_NONE before the split)
  int8_t idx[MAX_HEADS];   // index of the head inside its archetype group
};

__device__ __forceinline__ long long route_dst(const RouteParams& p, int t, int h, int c, uint4** k, uint4** v) {
  const int cls = p.cls[h], idx = p.idx[h];
  if (cls == CLS_SINK) {
    if (!p.copy_sink) return -1;
    *k = p.sd_k; *v = p.sd_v;
    return (static_cast<long long>(idx) * p.L + t) * p.chunks + c;
  }
  if (cls == CLS_DUMMY) {
    if (!p.copy_dummy) return -1;
    *k = p.sd_k; *v = p.sd_v;
    return (static_cast<long long>(p.n_sink + idx) * p.L + t) * p.chunks + c;
  }
  if (!p.copy_window) return -1;
  if (cls == CLS_GLOBAL) {
    *k = p.g_k; *v = p.g_v;
    return ((static_cast<long long>(idx) * p.n_blocks + p.slot) * p.L + t) * p.chunks + c;
  }
  if (cls == CLS_SPATIAL) {
    *k = p.sp_k; *v = p.sp_v;
    const int f = t / p.tokens_per_frame, pos = t - f * p.tokens_per_frame;
    const long long row = static_cast<long long>(idx) * p.n_blocks * p.L + p.sp_base[pos] +
                          static_cast<long long>(p.slot * p.frames_per_block + f) * p.sp_nc[pos];
    return row * p.chunks + c;
  }
  return -1;
}

constexpr int ROUTE_UNROLL = 4;

__global__ void __launch_bounds__(256) route_block_kernel(const RouteParams p) {
  const long long per_token = static_cast<long long>(p.H) * p.chunks;
  const long long total = per_token * p.L;
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  for (long long g0 = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; g0 < total;
       g0 += stride * ROUTE_UNROLL) {
    uint4 kv[ROUTE_UNROLL], vv[ROUTE_UNROLL];
#pragma unroll
    for (int u = 0; u < ROUTE_UNROLL; ++u) {
      const long long g = g0 + u * stride;
      if (g < total) {
        kv[u] = __ldcs(p.src_k + g);
        vv[u] = __ldcs(p.src_v + g);
      }
    }
#pragma unroll
    for (int u = 0; u < ROUTE_UNROLL; ++u) {
      const long long g = g0 + u * stride;
      if (g >= total) continue;
      const int t = static_cast<int>(g / per_token);
      const int rem = static_cast<int>(g - t * per_token);
      const int h = rem / p.chunks, c = rem - h * p.chunks;
      if (p.copy_mono) {
        const long long m = static_cast<long long>(p.slot) * total + g;
        p.mono_k[m] = kv[u];
        p.mono_v[m] = vv[u];
      }
      uint4 *dk = nullptr, *dv = nullptr;
      const long long d = route_dst(p, t, h, c, &dk, &dv);
      if (d >= 0) {
        dk[d] = kv[u];
        dv[d] = vv[u];
      }
    }
  }
}

struct ExportParams {
  const uint4* src_k;  // buffer of the head's archetype (or the monolithic cache)
  const uint4* src_v;
  uint4* dst_k;        // [n_logical * L][d]
  uint4* dst_v;
  const int32_t* sp_base;
  const int32_t* sp_nc;
  int32_t L, H, chunks, tokens_per_frame, frames_per_block, n_blocks;
  int32_t layout;      // 0: monolithic [slot][L][H][d]; 1: [head][slot][L][d]; 2: Spatial cell-major; 3: [head][L][d]
  int32_t head;        // original head (layout 0) or index inside the group (others)
  int32_t n_logical;
  int32_t slots[MAX_BLOCKS];  // physical slot of each logical block
};

__global__ void __launch_bounds__(256) export_head_kernel(const ExportParams p) {
  const long long total = static_cast<long long>(p.n_logical) * p.L * p.chunks;
  for (long long g = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; g < total;
       g += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int c = static_cast<int>(g % p.chunks);
    const long long row = g / p.chunks;
    const int b = static_cast<int>(row / p.L), t = static_cast<int>(row - static_cast<long long>(b) * p.L);
    const int slot = p.slots[b];
    long long s;
    if (p.layout == 0) {
      s = ((static_cast<long long>(slot) * p.L + t) * p.H + p.head) * p.chunks + c;
    } else if (p.layout == 1) {
      s = ((static_cast<long long>(p.head) * p.n_blocks + slot) * p.L + t) * p.chunks + c;
    } else if (p.layout == 2) {
      const int f = t / p.tokens_per_frame, pos = t - f * p.tokens_per_frame;
      s = (static_cast<long long>(p.head) * p.n_blocks * p.L + p.sp_base[pos] +
           static_cast<long long>(slot * p.frames_per_block + f) * p.sp_nc[pos]) * p.chunks + c;
    } else {
      s = (static_cast<long long>(p.head) * p.L + t) * p.chunks + c;
    }
    if (p.dst_k) p.dst_k[g] = p.src_k[s];
    if (p.dst_v) p.dst_v[g] = p.src_v[s];
  }
}

}  // namespace hc
