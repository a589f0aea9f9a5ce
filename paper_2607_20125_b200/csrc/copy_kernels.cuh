// Byte-exact cache movement: append of one block into the monolithic ring and/or the per-archetype
// buffers, the split of the monolithic cache (one launch, one grid row per cached block), and the export of one
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
  uint4* sd_k;  // [N_sink + N_dummy][sd_slots][L][d]
  uint4* sd_v;
  uint4* g_k;   // [N_global][n_blocks * L][d], block slots are a ring
  uint4* g_v;
  uint4* sp_k;  // [N_spatial][cell][slot][frame][token in cell][d]
  uint4* sp_v;
  const int32_t* sp_base;  // [T_f]: n_blocks * F_b * (tokens in earlier cells) + index of the token inside its cell
  const int32_t* sp_nc;    // [T_f]: tokens per frame in the token's cell
  int32_t L, H, chunks;    // chunks = d / 8
  int32_t tokens_per_frame, frames_per_block, n_blocks;
  int32_t n_sink;
  int32_t copy_mono, copy_window;
  // blockIdx.y selects the source block: it is read at src + src_stride * slots[y] (stride 0: the caller's block)
  // and lands in ring slot slots[y]; sd_slot_sink[y] / sd_slot_dummy[y] name the block slot of the Sink-Dummy
  // buffer that source feeds for Sink / Dummy heads (-1: none)
  long long src_stride;    // in 16-byte chunks
  int32_t sd_slots;        // blocks per head in the Sink-Dummy buffer (1, or 2 with the anchor + current variant)
  int8_t sd_slot_sink[MAX_BLOCKS], sd_slot_dummy[MAX_BLOCKS];
  int8_t slots[MAX_BLOCKS];
  // threads are laid over the heads somebody keeps: kept[k] lists them for source rows of kind k
  // (0: feeds the Sink heads too, 1: the Dummy heads too, 2: both, 3: neither), n_kept[k] counts them
  int8_t kind[MAX_BLOCKS];
  int8_t n_kept[4];
  int8_t kept[4][MAX_HEADS];
  int8_t cls[MAX_HEADS];   // archetype per original head (CLS_NONE before the split)
  int8_t idx[MAX_HEADS];   // index of the head inside its archetype group
};

constexpr int ROUTE_UNROLL = 4;

// Threads of a block are laid over (token, kept head, 16-byte chunk) of consecutive source tokens, so a thread's
// head - and with it where its chunks go - is fixed for the whole launch and only the token advances; heads whose
// chunks nobody keeps (Sink / Dummy heads of the other blocks) get no threads and are never loaded.
__global__ void __launch_bounds__(1024) route_block_kernel(const RouteParams p) {
  const int per_token = p.H * p.chunks;
  const int src = blockIdx.y, slot = p.slots[src];
  const int kind = p.kind[src];
  const int kept_chunks = p.n_kept[kind] * p.chunks;
  if (kept_chunks == 0) return;
  const int tokens_per_iter = blockDim.x / kept_chunks;
  const int tl = threadIdx.x / kept_chunks, kc = threadIdx.x - tl * kept_chunks;
  if (tl >= tokens_per_iter) return;
  const int h = p.kept[kind][kc / p.chunks], c = kc % p.chunks;
  const int hc = h * p.chunks + c;
  const long long total = static_cast<long long>(per_token) * p.L;
  const uint4* src_k = p.src_k + p.src_stride * slot;
  const uint4* src_v = p.src_v + p.src_stride * slot;
  const int cls = p.cls[h], idx = p.idx[h];
  // destination of this thread's chunks: base + t * chunks for the row-major buffers
  uint4 *dk = nullptr, *dv = nullptr;
  long long base = 0;
  bool spatial = false;
  if (cls == CLS_SINK && p.sd_slot_sink[src] >= 0) {
    dk = p.sd_k; dv = p.sd_v;
    base = (static_cast<long long>(idx) * p.sd_slots + p.sd_slot_sink[src]) * p.L * p.chunks + c;
  } else if (cls == CLS_DUMMY && p.sd_slot_dummy[src] >= 0) {
    dk = p.sd_k; dv = p.sd_v;
    base = (static_cast<long long>(p.n_sink + idx) * p.sd_slots + p.sd_slot_dummy[src]) * p.L * p.chunks + c;
  } else if (cls == CLS_GLOBAL && p.copy_window) {
    dk = p.g_k; dv = p.g_v;
    base = (static_cast<long long>(idx) * p.n_blocks + slot) * p.L * p.chunks + c;
  } else if (cls == CLS_SPATIAL && p.copy_window) {
    dk = p.sp_k; dv = p.sp_v;
    base = static_cast<long long>(idx) * p.n_blocks * p.L;  // in rows; the rest depends on the token
    spatial = true;
  }
  const int t_stride = gridDim.x * tokens_per_iter;
  for (int t0 = blockIdx.x * tokens_per_iter + tl; t0 < p.L; t0 += t_stride * ROUTE_UNROLL) {
    uint4 kv[ROUTE_UNROLL], vv[ROUTE_UNROLL];
    int sb[ROUTE_UNROLL], sn[ROUTE_UNROLL];
#pragma unroll
    for (int u = 0; u < ROUTE_UNROLL; ++u) {
      const int t = t0 + u * t_stride;
      if (t < p.L) {
        const long long g = static_cast<long long>(t) * per_token + hc;
        kv[u] = __ldcs(src_k + g);
        vv[u] = __ldcs(src_v + g);
        if (spatial) {
          const int pos = t % p.tokens_per_frame;
          sb[u] = p.sp_base[pos];
          sn[u] = p.sp_nc[pos];
        }
      }
    }
#pragma unroll
    for (int u = 0; u < ROUTE_UNROLL; ++u) {
      const int t = t0 + u * t_stride;
      if (t >= p.L) continue;
      if (p.copy_mono) {
        const long long m = static_cast<long long>(slot) * total + static_cast<long long>(t) * per_token + hc;
        p.mono_k[m] = kv[u];
        p.mono_v[m] = vv[u];
      }
      if (dk) {
        long long d;
        if (spatial) {
          const int f = t / p.tokens_per_frame;
          d = (base + sb[u] + static_cast<long long>(slot * p.frames_per_block + f) * sn[u]) * p.chunks + c;
        } else {
          d = base + static_cast<long long>(t) * p.chunks;
        }
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
  int32_t layout;      // 0: monolithic [slot][L][H][d]; 1: [head][slot][L][d]; 2: Spatial cell-major; 3: Sink-Dummy [head][sd_slots][L][d]
  int32_t sd_slots;
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
      s = ((static_cast<long long>(p.head) * p.sd_slots + slot) * p.L + t) * p.chunks + c;
    }
    if (p.dst_k) p.dst_k[g] = p.src_k[s];
    if (p.dst_v) p.dst_v[g] = p.src_v[s];
  }
}

}  // namespace hc
