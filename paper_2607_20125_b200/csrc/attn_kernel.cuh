// Flash-style attention for every HeadCast pathway on sm_100a tensor cores.
//
// One persistent CTA per SM walks a host-built list of work items.  A work item is up to two
// 128-row query tiles of one head that share one key/value stream:
//   - S = Q K^T and O += P V run on tcgen05.mma (M = 128, N = 128 / head_dim, bf16 in, fp32 accumulate)
//     with S, P and O living in tensor memory (P overlays S as packed bf16 and is fed to the second
//     product straight from tensor memory);
//   - K/V tiles (128 keys) arrive through TMA into one 4-slot shared-memory ring (128-byte swizzle), in the
//     order they are consumed (K0 V0 K1 V1 ...), so loads run two tiles ahead of the products;
//   - sixteen softmax warps, eight per query tile, two threads per query row (online softmax in the
//     exp2 domain, a quarter of the exponentials evaluated as a cubic on the FMA pipe to relieve the
//     special-function unit, rescaling of O only when the running maximum grew by more than 2^8);
//   - warp 0 is the TMA producer, warp 1 issues every MMA.
// Which keys a query tile sees is entirely a property of the work item: a row range of one of the
// cache buffers (whole window, one block, one Spatial cell) or, for the classification's Spatial
// proxy, a per-frame band of tokens plus an element-wise neighbourhood test.
//
// Every wait is bounded (see mbar_wait); on expiry the CTA drains, frees its tensor memory and leaves,
// and the host reports HC_ERR_TIMEOUT.
#pragma once
#include "tc05.cuh"

namespace hc {

struct CellGeom {
  int32_t y0, x0, ch, cw;  // top-left grid position and extent of a deployed Spatial cell
};

enum : int32_t { OUT_BF16 = 0, OUT_PARTIAL = 1 };

struct WorkItem {
  int32_t head;           // original head index: addresses Q and the output
  int32_t cell;           // < 0: query rows are consecutive tokens; else index into AttnParams::cells
  int32_t q_start[2];     // first token (cell < 0) or first packed index within the cell's queries
  int32_t q_count[2];     // valid rows of each 128-row query tile (0: tile unused)
  int32_t kv_map;         // K map = maps[2 * kv_map], V map = maps[2 * kv_map + 1]
  int32_t kv_x0;          // element column of this head inside a buffer row
  int32_t kv_row0;        // buffer row of the first key of segment 0
  int32_t seg_stride;     // rows between the starts of consecutive segments
  int32_t seg_len;        // keys per segment
  int32_t tiles_per_seg;  // ceil(seg_len / 128)
  int32_t tile_begin;     // this item covers tiles [tile_begin, tile_end) of the segment-major enumeration
  int32_t tile_end;
  int32_t out_mode;       // OUT_*
  int32_t out_slot;       // OUT_PARTIAL: partial slot
};

struct AttnParams {
  const WorkItem* items;
  const int32_t* cta_first;  // [gridDim.x + 1]: CTA b owns items [cta_first[b], cta_first[b + 1])
  const CellGeom* cells;
  const __nv_bfloat16* q;  // [L][H][d]
  __nv_bfloat16* out;      // [L][H][d]
  float* part_o;           // [slot][256][d] unnormalised partial outputs
  float2* part_ml;         // [slot][256] (running max in the log2 domain, row sum)
  float* part_mid;         // [slot][256] Spatial proxy only: the part of the row sum that came from the middle blocks
  int32_t n_heads, tokens_per_frame, grid_w, block_tokens;
  float scale_log2e;       // softmax scale * log2(e)
  int32_t* status;
  // dynamic tail: when a CTA has finished its own list it draws items [dyn_first, dyn_end) of `items` from a shared
  // queue; dyn_counter[0] is the next queue position, dyn_counter[1] counts CTAs that are done (the last clears both)
  int32_t dyn_first, dyn_end;
  int32_t* dyn_counter;
  unsigned long long* trace;  // optional [2 * n_items]: globaltimer (ns) when query tile 0's warpgroup starts / ends an item
  // Spatial proxy only
  int32_t radius;
  int32_t mid_seg_lo, mid_seg_hi, last_seg_lo, last_seg_hi;  // segments (cached frames) of the middle / newest blocks
  // K map = maps[2 * kv_map], V map = maps[2 * kv_map + 1].  The descriptors travel in the kernel's parameter space
  // (the kernel takes its parameters as __grid_constant__), so a launch always reads the descriptors it was given:
  // no copy to global memory, nothing another launch can overwrite, no tensor-map proxy fence to forget.
  alignas(64) CUtensorMap maps[8];
};

constexpr int ATTN_THREADS = 576;  // warp 0: TMA, warp 1: MMA, warps 2-9 / 10-17: softmax for query tile 0 / 1 (112 registers each)
constexpr int SOFTMAX_WARPS = 8;    // per query tile: two threads per row, each owning 64 of the tile's 128 keys
constexpr int KV_SLOTS = 4;  // one shared-memory ring for K and V tiles, filled and drained in the order K0 V0 K1 V1 ...
#ifndef HC_POLY_MASK
#define HC_POLY_MASK 3  // pairs whose index has all these bits set take the polynomial exponential (3: every 4th)
#endif
#ifndef HC_L2_HINT
#define HC_L2_HINT 2  // 1: Spatial cells' K/V are loaded evict-first; 2: the other K/V also evict-last
#endif
#ifndef HC_RESCALE_THRESHOLD
#define HC_RESCALE_THRESHOLD 8.0f
#endif
constexpr float RESCALE_THRESHOLD = HC_RESCALE_THRESHOLD;  // log2 units

template <int D>
struct AttnSmem {
  static constexpr int BLOCK_BYTES = 128 * 128;      // [128 rows][64 bf16], 128-byte swizzle
  static constexpr int TILE_BYTES = (D / 64) * BLOCK_BYTES;
  static constexpr int Q_OFF = 0;
  static constexpr int KV_OFF = 2 * TILE_BYTES;
  static constexpr int TOTAL = KV_OFF + KV_SLOTS * TILE_BYTES;
  static constexpr int DYN_BYTES = TOTAL + 1024;  // slack for manual 1024-byte alignment
};

// Token index of packed query `p` of a cell (frame-major, then cell row, then cell column).
__device__ __forceinline__ int cell_query_token(const CellGeom& g, int p, int tokens_per_frame, int grid_w) {
  const int nc = g.ch * g.cw;
  const int f = p / nc, i = p - f * nc;
  const int dy = i / g.cw, dx = i - dy * g.cw;
  return f * tokens_per_frame + (g.y0 + dy) * grid_w + g.x0 + dx;
}

// Which of 32 consecutive keys a query row may see, as a bit mask: columns >= n_valid (ragged tail of a segment) are
// never seen; for the Spatial proxy neither are keys outside the (2r+1)^2 neighbourhood of the query's grid position
// (qy, qx).  tok0 is the in-frame token index of column 0.  The neighbourhood is at most 2r+1 runs of consecutive
// tokens (one per grid row), so the mask costs a few integer operations per row of the neighbourhood, not per key.
template <bool PROXY>
__device__ __forceinline__ uint32_t visible_keys(int n_valid, int tok0, int qy, int qx, int radius, int grid_w) {
  uint32_t tail = (n_valid >= 32) ? 0xffffffffu : (n_valid <= 0 ? 0u : (0xffffffffu >> (32 - n_valid)));
  if (!PROXY) return tail;
  uint32_t allow = 0;
  const int lo_x = max(qx - radius, 0), hi_x = min(qx + radius, grid_w - 1);
#pragma unroll 1
  for (int ky = max(qy - radius, 0); ky <= qy + radius; ++ky) {
    const int a = max(ky * grid_w + lo_x - tok0, 0), b = min(ky * grid_w + hi_x - tok0, 31);  // inclusive column range
    if (a <= b) allow |= (0xffffffffu >> (31 - b + a)) << a;
  }
  return allow & tail;
}

// Sets the logits of the keys a row must not see to -inf.  Outside the proxy only the ragged tail of a segment is
// hidden, which is the same for all rows: a comparison per column, skipped for full chunks.
template <bool PROXY>
__device__ __forceinline__ void apply_visible(uint32_t (&sv)[32], uint32_t visible, int n_valid) {
  if (PROXY) {
#pragma unroll
    for (int i = 0; i < 32; ++i)
      if (!((visible >> i) & 1u)) sv[i] = 0xff800000u;
  } else if (n_valid < 32) {
#pragma unroll
    for (int i = 0; i < 32; ++i)
      if (i >= n_valid) sv[i] = 0xff800000u;
  }
}

template <int D, bool PROXY>
__global__ void __launch_bounds__(ATTN_THREADS, 1) attn_kernel(const __grid_constant__ AttnParams p) {
  using SM = AttnSmem<D>;
  constexpr int NB = D / 64;          // 64-column blocks per tile
  constexpr int QK_STEPS = D / 16;    // k-steps of S = Q K^T
    constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t S_COL = 0, O_COL = 256;  // S_t at t*128, O_t at 256 + t*128; P_t overlays S_t

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t bar_q_full[2], bar_s_full[2], bar_p_full[2], bar_o_full[2], bar_pair[2];
  __shared__ float pair_val[2][2][2][128];  // [query tile][parity][column half][row]: values the two threads of a row swap
  __shared__ uint64_t bar_kv_full[KV_SLOTS], bar_kv_free[KV_SLOTS];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ uint64_t bar_dyn[4];
  __shared__ int32_t dyn_item[4];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int t = 0; t < 2; ++t) {
      // softmax warps arrive once per warp (lane 0, after __syncwarp): 256 arrivals on one mbarrier would be
      // 256 serialised shared-memory atomics per tile
      mbar_init(&bar_q_full[t], SOFTMAX_WARPS);
      mbar_init(&bar_s_full[t], 1);
      mbar_init(&bar_p_full[t], SOFTMAX_WARPS);
      mbar_init(&bar_o_full[t], 1);
      mbar_init(&bar_pair[t], SOFTMAX_WARPS);
    }
    for (int s = 0; s < KV_SLOTS; ++s) {
      mbar_init(&bar_kv_full[s], 1);
      mbar_init(&bar_kv_free[s], 1);
    }
    for (int s = 0; s < 4; ++s) mbar_init(&bar_dyn[s], 1);
    // A context whose earlier kernel gave up on a wait keeps its status word set until the host has read it; the
    // shared queue's counters may then be half drawn, so until then a launch does nothing at all (every thread sees
    // the same answer: one thread reads the word, the others read its copy after the barrier below)
    abort_flag = (*reinterpret_cast<volatile int32_t*>(p.status) != 0) ? 1 : 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_slot, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  volatile int* abortp = &abort_flag;

  const bool dead_on_arrival = abort_flag != 0;  // read before any wait of this launch can raise the flag
  const int item_lo = p.cta_first[blockIdx.x], item_hi = p.cta_first[blockIdx.x + 1];
  const bool has_queue = p.dyn_end > p.dyn_first;
  // Items come from the CTA's own list first, then from the shared queue.  The producer thread draws the queue
  // position and publishes it through a ring of four shared-memory slots; it runs at most two key tiles (less than
  // one item) ahead of the other roles, so a slot is read long before its fourth successor is written.
  struct ItemCursor { int it; bool in_queue; uint32_t k; };
  // issuer and softmax warps: advance to the next item (false: no more)
  auto next_item = [&](ItemCursor& cur) -> bool {
    if (!cur.in_queue) {
      if (cur.it + 1 < item_hi) { ++cur.it; return true; }
      cur.in_queue = true;
    }
    if (!has_queue) return false;
    if (!mbar_wait(&bar_dyn[cur.k & 3], (cur.k >> 2) & 1, abortp, p.status, 51)) return false;
    cur.it = dyn_item[cur.k & 3];
    ++cur.k;
    return cur.it >= 0;
  };
  // producer thread: the same, but it is the one that draws from the queue and tells the others
  auto next_item_producer = [&](ItemCursor& cur) -> bool {
    if (!cur.in_queue) {
      if (cur.it + 1 < item_hi) { ++cur.it; return true; }
      cur.in_queue = true;
    }
    if (!has_queue) return false;
    const int pos = atomicAdd(&p.dyn_counter[0], 1);
    const int v = (pos < p.dyn_end - p.dyn_first) ? p.dyn_first + pos : -1;
    dyn_item[cur.k & 3] = v;
    mbar_arrive(&bar_dyn[cur.k & 3]);  // release: the slot is written before the arrival is seen
    ++cur.k;
    cur.it = v;
    if (v < 0 && atomicAdd(&p.dyn_counter[1], 1) == static_cast<int>(gridDim.x) - 1) {
      p.dyn_counter[0] = 0;  // every CTA has drawn its end marker: the queue is ready for the next launch
      p.dyn_counter[1] = 0;
    }
    return v >= 0;
  };

  if (dead_on_arrival) {
    // nothing: straight to the teardown
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t kt = 0;
      bool ok = true;
      // L2 policy per item: a Spatial cell's keys are read by one item only (its queries fill at most one tile pair),
      // so they stream through L2 without pushing out the long K/V streams that every query tile of a head re-reads
      const uint64_t pol_stream = l2_policy_evict_first();
#if HC_L2_HINT == 2
      const uint64_t pol_keep = l2_policy_evict_last();
#else
      const uint64_t pol_keep = l2_policy_evict_normal();
#endif
      ItemCursor cur = {item_lo - 1, false, 0u};
      while (ok && next_item_producer(cur)) {
        const int it = cur.it;
        const WorkItem w = p.items[it];
        const CUtensorMap* kmap = &p.maps[2 * w.kv_map];
        const CUtensorMap* vmap = kmap + 1;
        const uint64_t policy = (HC_L2_HINT && w.cell >= 0) ? pol_stream : pol_keep;
        for (int tile = w.tile_begin; tile < w.tile_end; ++tile, ++kt) {
          const int seg = tile / w.tiles_per_seg, c = tile - seg * w.tiles_per_seg;
          const int row = w.kv_row0 + seg * w.seg_stride + c * 128;
          // ring position g = 2 * kt holds K of this tile, g + 1 its V
          for (int kv = 0; kv < 2; ++kv) {
            const uint32_t g = 2 * kt + kv, st = g % KV_SLOTS, ph = (g / KV_SLOTS) & 1;
            if (!(ok = mbar_wait(&bar_kv_free[st], ph ^ 1, abortp, p.status, 11 + kv))) break;
            mbar_arrive_expect_tx(&bar_kv_full[st], SM::TILE_BYTES);
            for (int b = 0; b < NB; ++b)
              tma_load_2d_hint(smem + SM::KV_OFF + st * SM::TILE_BYTES + b * SM::BLOCK_BYTES, kv ? vmap : kmap,
                               w.kv_x0 + 64 * b, row, &bar_kv_full[st], policy);
          }
          if (!ok) break;
        }
      }
      if (!ok) {
        // after an expired wait elsewhere: let the copies already in flight land before the CTA leaves
        for (uint32_t back = 1; back <= KV_SLOTS && back <= 2 * kt; ++back) {
          const uint32_t g = 2 * kt - back, st = g % KV_SLOTS, ph = (g / KV_SLOTS) & 1;
          int local_abort = 0;
          mbar_wait(&bar_kv_full[st], ph, &local_abort, p.status, 13);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0);
      const uint32_t idesc_o = idesc_bf16_f32(128, D, 0, 1);
      const uint32_t q_addr = smem_u32(smem + SM::Q_OFF), kv_addr = smem_u32(smem + SM::KV_OFF);
      uint32_t kt = 0, q_cnt[2] = {0, 0}, p_cnt[2] = {0, 0};
      bool ok = true;
      const uint64_t q_desc = smem_desc_sw128(q_addr, 16, 1024), k_desc = smem_desc_sw128(kv_addr, 16, 1024);
      const uint64_t v_desc = smem_desc_sw128(kv_addr, SM::BLOCK_BYTES, 1024);
      auto issue_qk = [&](int t, uint32_t st) {
        mma_block_ss<QK_STEPS>(tmem + S_COL + t * 128, q_desc + ((t * SM::TILE_BYTES) >> 4),
                               k_desc + ((st * SM::TILE_BYTES) >> 4), idesc_s, SM::BLOCK_BYTES >> 4, SM::BLOCK_BYTES >> 4);
      };
      auto issue_pv = [&](int t, uint32_t st, bool accumulate) {
        mma_block_ts8(tmem + O_COL + t * 128, tmem + S_COL + t * 128, v_desc + ((st * SM::TILE_BYTES) >> 4), idesc_o,
                      accumulate ? 1u : 0u);
      };
      ItemCursor cur = {item_lo - 1, false, 0u};
      while (ok && next_item(cur)) {
        const int it = cur.it;
        const WorkItem w = p.items[it];
        const int nt = w.tile_end - w.tile_begin;
        const int n_q = w.q_count[1] > 0 ? 2 : 1;
        {
          const uint32_t st = (2 * kt) % KV_SLOTS, ph = ((2 * kt) / KV_SLOTS) & 1;
          if (!(ok = mbar_wait(&bar_kv_full[st], ph, abortp, p.status, 21))) break;
          for (int t = 0; t < n_q && ok; ++t) {
            if (!(ok = mbar_wait(&bar_q_full[t], q_cnt[t] & 1, abortp, p.status, 22))) break;
            ++q_cnt[t];
            tc_fence_after_sync();
            issue_qk(t, st);
            mma_commit(&bar_s_full[t]);
          }
          if (!ok) break;
          mma_commit(&bar_kv_free[st]);
        }
        for (int j = 0; j < nt && ok; ++j) {
          const uint32_t gv = 2 * (kt + j) + 1, gk = gv + 1;  // ring positions of V_j and K_{j+1}
          const uint32_t st = gv % KV_SLOTS, ph = (gv / KV_SLOTS) & 1;
          const uint32_t st1 = gk % KV_SLOTS, ph1 = (gk / KV_SLOTS) & 1;
          if (!(ok = mbar_wait(&bar_kv_full[st], ph, abortp, p.status, 23))) break;
          for (int t = 0; t < n_q && ok; ++t) {
            if (!(ok = mbar_wait(&bar_p_full[t], p_cnt[t] & 1, abortp, p.status, 24))) break;
            ++p_cnt[t];
            tc_fence_after_sync();
            issue_pv(t, st, j > 0);
            if (j + 1 < nt) {
              if (t == 0 && !(ok = mbar_wait(&bar_kv_full[st1], ph1, abortp, p.status, 25))) break;
              tc_fence_after_sync();
              issue_qk(t, st1);
              mma_commit(&bar_s_full[t]);
              if (t == n_q - 1) mma_commit(&bar_kv_free[st1]);
            } else {
              mma_commit(&bar_o_full[t]);
            }
          }
          if (!ok) break;
          mma_commit(&bar_kv_free[st]);
        }
        kt += nt;
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue warps
    // Eight warps per query tile.  A warp may only touch the 32 TMEM lanes (rows) of its warp-id quarter, and a
    // lone warp cannot issue fast enough to keep up with the tensor pipe, so every row is shared by two threads
    // of two warps on the same scheduler: each owns 64 of the tile's 128 keys (and half of the output columns)
    // and they swap their row maxima through shared memory once per tile.
    const int t = (warp - 2) >> 3;                  // query tile
    const int half = ((warp - 2) >> 2) & 1;         // which 64 keys / which half of the output columns
    const int r = ((warp & 3) << 5) | lane;         // row inside the tile == TMEM lane
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) << 5) << 16;
    const uint32_t s_addr = tmem + lane_off + S_COL + t * 128 + half * 64;   // this thread's logits
    const uint32_t p_addr = s_addr;  // its share of P (packed bf16) goes over the first 32 columns of its own logits
    constexpr int OC = D / 2;                                                // output columns per thread
    const uint32_t o_addr = tmem + lane_off + O_COL + t * 128 + half * OC;
    uint8_t* sq = smem + SM::Q_OFF + t * SM::TILE_BYTES;
    uint32_t s_cnt = 0, o_cnt = 0, x_cnt = 0;
    bool ok = true;
    // swaps one float with the other thread of the row (bounded wait like every other wait here)
    auto swap_with_partner = [&](float mine, float& theirs) -> bool {
      const int par = x_cnt & 1;
      pair_val[t][par][half][r] = mine;
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar_pair[t]);
      if (!mbar_wait(&bar_pair[t], par, abortp, p.status, 34)) return false;
      ++x_cnt;
      theirs = pair_val[t][par][half ^ 1][r];
      return true;
    };
    ItemCursor cur = {item_lo - 1, false, 0u};
    while (ok && next_item(cur)) {
      const int it = cur.it;
      const WorkItem w = p.items[it];
      if (w.q_count[t] == 0) continue;
      if (p.trace && t == 0 && r == 0 && half == 0) p.trace[2 * it] = global_timer_ns();
      const bool row_valid = r < w.q_count[t];
      int token = 0;
      if (row_valid) {
        token = w.q_start[t] + r;
        if (w.cell >= 0) token = cell_query_token(p.cells[w.cell], token, p.tokens_per_frame, p.grid_w);
      }
      // ---- stage this warp's 32 query rows (its half of the columns) into shared memory (swizzled); invalid rows are
      // zero.  The lanes share the rows: CH consecutive lanes fetch the CH 16-byte chunks of one row, so a load
      // instruction touches 32 / CH rows (4 lines of 128 bytes at d = 128) instead of 32 - with one row per lane the
      // 16 warps needed 4096 line visits per item and the load/store unit, not the latency, set the time (2.5 us).
      {
        constexpr int CH = D / 16;  // 16-byte chunks of a half row
        uint4 v[CH];
#pragma unroll
        for (int k = 0; k < CH; ++k) {
          const int idx = k * 32 + lane, row = idx / CH, c = half * CH + idx % CH;
          const int tok = __shfl_sync(0xffffffffu, token, row);
          const bool valid = __shfl_sync(0xffffffffu, row_valid ? 1 : 0, row) != 0;
          v[k] = make_uint4(0, 0, 0, 0);
          if (valid) v[k] = __ldg(reinterpret_cast<const uint4*>(p.q + (static_cast<size_t>(tok) * p.n_heads + w.head) * D) + c);
        }
#pragma unroll
        for (int k = 0; k < CH; ++k) {
          const int idx = k * 32 + lane, row = idx / CH, c = half * CH + idx % CH;
          *reinterpret_cast<uint4*>(sq + (c / 8) * SM::BLOCK_BYTES + sw128_offset((r & ~31) + row, c % 8)) = v[k];
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();  // orders this thread's TMEM reads of the previous item before the arrive
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar_q_full[t]);
      }
      int qy = 0, qx = 0;
      if (PROXY) {
        const int pos = token % p.tokens_per_frame;
        qy = pos / p.grid_w;
        qx = pos - qy * p.grid_w;
      }
      float m_ref = -INFINITY, l_sum = 0.f, l_mid = 0.f;  // l_* cover this thread's 64 keys per tile only
      const int nt = w.tile_end - w.tile_begin;
      for (int j = 0; j < nt; ++j) {
        const int tile = w.tile_begin + j;
        const int seg = tile / w.tiles_per_seg, c = tile - seg * w.tiles_per_seg;
        const int n_valid = min(128, w.seg_len - c * 128) - half * 64;  // valid keys among this thread's 64
        const int tok0 = PROXY ? (w.kv_row0 + c * 128 + half * 64) : 0;  // in-frame token of its first key
        if (!(ok = mbar_wait(&bar_s_full[t], s_cnt & 1, abortp, p.status, 31))) break;
        ++s_cnt;
        tc_fence_after_sync();
        // pass 1: maximum of this thread's 64 logits (32 columns at a time; they are read again in pass 2, which
        // keeps the live registers low enough for 576 threads per CTA).  Keys this row must not see count as -inf:
        // the ragged tail of a segment, and for the Spatial proxy every key outside the (2r+1)^2 neighbourhood.
        float mx;
        {
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            const uint32_t visible = PROXY ? visible_keys<PROXY>(n_valid - ch * 32, tok0 + ch * 32, qy, qx, p.radius, p.grid_w) : 0u;
            if (PROXY && __all_sync(0xffffffffu, visible == 0u)) continue;  // no row of this warp sees any of these keys
            uint32_t sv[32];
            tmem_ld32(s_addr + ch * 32, sv);
            tmem_wait_ld();
            apply_visible<PROXY>(sv, visible, n_valid - ch * 32);
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              mx4[0] = max3(mx4[0], __uint_as_float(sv[i]), __uint_as_float(sv[i + 1]));
              mx4[1] = max3(mx4[1], __uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3]));
              mx4[2] = max3(mx4[2], __uint_as_float(sv[i + 4]), __uint_as_float(sv[i + 5]));
              mx4[3] = max3(mx4[3], __uint_as_float(sv[i + 6]), __uint_as_float(sv[i + 7]));
            }
          }
          mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        }
        float mx_other;
        if (!(ok = swap_with_partner(mx, mx_other))) break;
        mx = fmaxf(mx, mx_other) * p.scale_log2e;  // row maximum; scale > 0, so the maximum commutes with it
        // running maximum: move the reference only when some row of the warp outgrew it by 2^8.  Both threads of
        // a row see the same maximum and sit in the same lane of their warps, so both warps decide alike.
        const bool grow = mx > m_ref + RESCALE_THRESHOLD || (m_ref == -INFINITY && mx > -INFINITY);
        if (__any_sync(0xffffffffu, grow)) {
          const float m_new = fmaxf(m_ref, mx);
          const float alpha = (m_new == -INFINITY) ? 1.f : ex2_approx(m_ref - m_new);
          l_sum *= alpha;
          l_mid *= alpha;
          m_ref = m_new;
          if (j > 0) {  // O_t holds the products of the earlier tiles: bring this thread's columns to the new reference
#pragma unroll 1
            for (int ch = 0; ch < OC / 32; ++ch) {
              uint32_t v[32];
              tmem_ld32(o_addr + ch * 32, v);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
              tmem_st32(o_addr + ch * 32, v);
            }
          }
        }
        const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
        // pass 2: p = 2^(s * c - m), bf16 pack over the first 32 columns of this thread's logits, row sum in fp32
        const uint64_t c2 = pack_f32x2(p.scale_log2e, p.scale_log2e), m2 = pack_f32x2(-m_use, -m_use);
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          const uint32_t visible = PROXY ? visible_keys<PROXY>(n_valid - ch * 32, tok0 + ch * 32, qy, qx, p.radius, p.grid_w) : 0u;
          uint32_t pk[16];
          if (PROXY && __all_sync(0xffffffffu, visible == 0u)) {
            // nothing to exponentiate: P = 0 for these keys (the product still reads them)
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = 0u;
            tmem_st16(p_addr + ch * 16, pk);
            continue;
          }
          uint32_t sv[32];
          tmem_ld32(s_addr + ch * 32, sv);
          tmem_wait_ld();
          apply_visible<PROXY>(sv, visible, n_valid - ch * 32);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint64_t x2 = fma_f32x2(pack_f32x2(__uint_as_float(sv[2 * i]), __uint_as_float(sv[2 * i + 1])), c2, m2);
            float x0, x1, e0, e1;
            unpack_f32x2(x2, x0, x1);
            if ((i & HC_POLY_MASK) == HC_POLY_MASK) {
              // every fourth pair takes the polynomial route on the FMA pipe: the special-function unit alone
              // cannot produce 128 x 128 exponentials in the time the tensor pipe needs for the tile
              ex2_poly_pair(pack_f32x2(fmaxf(x0, -126.f), fmaxf(x1, -126.f)), e0, e1);
            } else {
              e0 = ex2_approx(x0);
              e1 = ex2_approx(x1);
            }
            pk[i] = pack_bf16x2(e0, e1);
            // the row sum adds the ROUNDED values: out = sum(p v) / sum(p) is then an exact convex combination of
            // the values even when the reference lags behind the row maximum and the largest p is not exactly 1
            add_bf16x2_to_f32(pk[i], sum4[(i & 1) * 2], sum4[(i & 1) * 2 + 1]);
          }
          tmem_st16(p_addr + ch * 16, pk);
        }
        const float tile_sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        l_sum += tile_sum;
        if (PROXY && seg >= p.mid_seg_lo && seg < p.mid_seg_hi && !(seg >= p.last_seg_lo && seg < p.last_seg_hi))
          l_mid += tile_sum;
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar_p_full[t]);
      }
      if (!ok) break;
      // ---- epilogue: row sums of the two halves are added, each thread normalises and stores its output columns
      float other;
      if (!(ok = swap_with_partner(l_sum, other))) break;
      l_sum += other;
      if (PROXY) {
        if (!(ok = swap_with_partner(l_mid, other))) break;
        l_mid += other;
      }
      if (!(ok = mbar_wait(&bar_o_full[t], o_cnt & 1, abortp, p.status, 32))) break;
      ++o_cnt;
      tc_fence_after_sync();
      const float inv = (l_sum > 0.f) ? 1.f / l_sum : 0.f;
      const float mult = (w.out_mode == OUT_PARTIAL) ? 1.f : inv;
      if constexpr (D == 128) {
        // The thread holds its row's OC output columns, but one row per lane is the worst pattern for global stores
        // (32 lines per instruction: 4096 line visits per tile, 4-5 us per item).  So the warp turns its 32 x OC block
        // through shared memory - its 4 KB of this tile's query buffer, which the last S product has finished reading
        // (the O product committed to bar_o_full was issued after it) - and stores whole 128-byte lines: 8 lanes a row.
        uint8_t* stg = sq + (half * 4 + (warp & 3)) * 4096;
        const int row0 = r & ~31;  // first row of this warp inside the tile
        if (w.out_mode == OUT_BF16) {
          constexpr int U = OC / 8;  // 16-byte units of a row's half: 8 (d = 128) or 4 (d = 64)
  #pragma unroll 1
          for (int ch = 0; ch < OC / 32; ++ch) {
            uint32_t v[32];
            tmem_ld32(o_addr + ch * 32, v);
            tmem_wait_ld();
  #pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint4 o4;
              o4.x = pack_bf16x2(__uint_as_float(v[8 * i + 0]) * mult, __uint_as_float(v[8 * i + 1]) * mult);
              o4.y = pack_bf16x2(__uint_as_float(v[8 * i + 2]) * mult, __uint_as_float(v[8 * i + 3]) * mult);
              o4.z = pack_bf16x2(__uint_as_float(v[8 * i + 4]) * mult, __uint_as_float(v[8 * i + 5]) * mult);
              o4.w = pack_bf16x2(__uint_as_float(v[8 * i + 6]) * mult, __uint_as_float(v[8 * i + 7]) * mult);
              *reinterpret_cast<uint4*>(stg + lane * 128 + (((ch * 4 + i) ^ (lane & 7)) << 4)) = o4;
            }
          }
          __syncwarp();
  #pragma unroll
          for (int k = 0; k < U; ++k) {
            const int idx = k * 32 + lane, row = idx / U, u = idx % U;
            const uint4 val = *reinterpret_cast<const uint4*>(stg + row * 128 + ((u ^ (row & 7)) << 4));
            const int tok = __shfl_sync(0xffffffffu, token, row);
            const bool valid = __shfl_sync(0xffffffffu, row_valid ? 1 : 0, row) != 0;
            if (valid)
              *reinterpret_cast<uint4*>(p.out + (static_cast<size_t>(tok) * p.n_heads + w.head) * D + half * OC + u * 8) = val;
          }
          __syncwarp();
        } else {
          float* base = p.part_o + (static_cast<size_t>(w.out_slot) * 256 + t * 128 + row0) * D + half * OC;
  #pragma unroll 1
          for (int ch = 0; ch < OC / 32; ++ch) {
            uint32_t v[32];
            tmem_ld32(o_addr + ch * 32, v);
            tmem_wait_ld();
  #pragma unroll
            for (int i = 0; i < 8; ++i)
              *reinterpret_cast<float4*>(stg + lane * 128 + ((i ^ (lane & 7)) << 4)) =
                  make_float4(__uint_as_float(v[4 * i + 0]) * mult, __uint_as_float(v[4 * i + 1]) * mult,
                              __uint_as_float(v[4 * i + 2]) * mult, __uint_as_float(v[4 * i + 3]) * mult);
            __syncwarp();
  #pragma unroll
            for (int k = 0; k < 8; ++k) {
              const int idx = k * 32 + lane, row = idx >> 3, u = idx & 7;
              const float4 val = *reinterpret_cast<const float4*>(stg + row * 128 + ((u ^ (row & 7)) << 4));
              const bool valid = __shfl_sync(0xffffffffu, row_valid ? 1 : 0, row) != 0;
              if (valid) *reinterpret_cast<float4*>(base + static_cast<size_t>(row) * D + ch * 32 + u * 4) = val;
            }
            __syncwarp();
          }
        }
      } else
      {
        // head_dim 64: a tile's query buffer (16 KB) is too small to turn the fp32 block through; one row per lane
        const size_t row_elem = (static_cast<size_t>(token) * p.n_heads + w.head) * D + half * OC;
#pragma unroll 1
        for (int ch = 0; ch < OC / 32; ++ch) {
          uint32_t v[32];
          tmem_ld32(o_addr + ch * 32, v);
          tmem_wait_ld();
          if (!row_valid) continue;
          if (w.out_mode == OUT_BF16) {
            uint4* dst = reinterpret_cast<uint4*>(p.out + row_elem + ch * 32);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint4 o4;
              o4.x = pack_bf16x2(__uint_as_float(v[8 * i + 0]) * mult, __uint_as_float(v[8 * i + 1]) * mult);
              o4.y = pack_bf16x2(__uint_as_float(v[8 * i + 2]) * mult, __uint_as_float(v[8 * i + 3]) * mult);
              o4.z = pack_bf16x2(__uint_as_float(v[8 * i + 4]) * mult, __uint_as_float(v[8 * i + 5]) * mult);
              o4.w = pack_bf16x2(__uint_as_float(v[8 * i + 6]) * mult, __uint_as_float(v[8 * i + 7]) * mult);
              dst[i] = o4;
            }
          } else {
            float* base = p.part_o + (static_cast<size_t>(w.out_slot) * 256 + t * 128 + r) * D + half * OC;
            float4* dst = reinterpret_cast<float4*>(base + ch * 32);
#pragma unroll
            for (int i = 0; i < 8; ++i)
              dst[i] = make_float4(__uint_as_float(v[4 * i + 0]) * mult, __uint_as_float(v[4 * i + 1]) * mult,
                                   __uint_as_float(v[4 * i + 2]) * mult, __uint_as_float(v[4 * i + 3]) * mult);
          }
        }
      }
      if (row_valid && half == 0 && w.out_mode == OUT_PARTIAL) {
        p.part_ml[static_cast<size_t>(w.out_slot) * 256 + t * 128 + r] = make_float2(m_ref, l_sum);
        if (PROXY) p.part_mid[static_cast<size_t>(w.out_slot) * 256 + t * 128 + r] = l_mid;
      }
      if (p.trace && t == 0 && r == 0 && half == 0) p.trace[2 * it + 1] = global_timer_ns();
    }
  }
  // ------------------------------------------------------------------ teardown
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

// Merges the partial results of query tiles whose key range was cut into several work items:
// out = sum_i 2^(m_i - m) O_i / sum_i 2^(m_i - m) l_i.  One thread per (row, 8 output columns),
// COMBINE_ROWS rows per block.
struct CombineEntry {
  int32_t head, cell, q_start, q_count;  // one 128-row query tile
  int32_t first_slot, n_parts, sub;      // partial slots first_slot .. +n_parts-1, rows sub*128 .. of each slot
  int32_t pad;
};

constexpr int COMBINE_ROWS = 16;  // query rows per block of combine_kernel

// Streaming 16-byte load, as a volatile statement: the compiler keeps such loads in program order, so a batch written
// before its first use really is in flight together (left to itself it sinks each load to its use to save registers).
__device__ __forceinline__ float4 ld_stream_f4(const float4* p) {
  float4 v;
  asm volatile("ld.global.cs.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

template <int D>
__global__ void __launch_bounds__(COMBINE_ROWS * (D / 8))
combine_kernel(const CombineEntry* entries, const CellGeom* cells, const float* part_o, const float2* part_ml,
               __nv_bfloat16* out, int n_heads, int tokens_per_frame, int grid_w) {
  constexpr int CHUNKS = D / 8;
  const CombineEntry e = entries[blockIdx.x / (128 / COMBINE_ROWS)];
  const int r = (blockIdx.x % (128 / COMBINE_ROWS)) * COMBINE_ROWS + threadIdx.x / CHUNKS;
  const int c = threadIdx.x % CHUNKS;
  if (r >= e.q_count) return;
  // Rows of successive parts lie 256 rows apart.  The parts are taken four at a time with all loads of a batch issued
  // before the first use (a thread has only 32 bytes per part to fetch, so one part at a time leaves the kernel waiting
  // on one memory round trip after the other); the partial results are read once, hence the streaming loads.
  const size_t row0 = static_cast<size_t>(e.first_slot) * 256 + e.sub * 128 + r;
  const int n = e.n_parts;
  float m = -INFINITY;
  for (int i0 = 0; i0 < n; i0 += 4) {
    float mk[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      mk[k] = (i0 + k < n) ? __ldg(&part_ml[row0 + static_cast<size_t>(i0 + k) * 256]).x : -INFINITY;
    m = fmaxf(fmaxf(m, fmaxf(mk[0], mk[1])), fmaxf(mk[2], mk[3]));
  }
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, l = 0.f;
  for (int i0 = 0; i0 < n; i0 += 4) {
    float2 ml[4];
    float4 a[4], b[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const size_t row = row0 + static_cast<size_t>(min(i0 + k, n - 1)) * 256;  // past the end: a valid row, weight 0
      ml[k] = __ldg(&part_ml[row]);
      const float4* src = reinterpret_cast<const float4*>(part_o + row * D + c * 8);
      a[k] = ld_stream_f4(src);
      b[k] = ld_stream_f4(src + 1);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float wgt = (i0 + k >= n || ml[k].x == -INFINITY) ? 0.f : ex2_approx(ml[k].x - m);
      l += wgt * ml[k].y;
      acc[0] += wgt * a[k].x; acc[1] += wgt * a[k].y; acc[2] += wgt * a[k].z; acc[3] += wgt * a[k].w;
      acc[4] += wgt * b[k].x; acc[5] += wgt * b[k].y; acc[6] += wgt * b[k].z; acc[7] += wgt * b[k].w;
    }
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  int token = e.q_start + r;
  if (e.cell >= 0) token = cell_query_token(cells[e.cell], token, tokens_per_frame, grid_w);
  uint4 o4;
  o4.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
  o4.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
  o4.z = pack_bf16x2(acc[4] * inv, acc[5] * inv);
  o4.w = pack_bf16x2(acc[6] * inv, acc[7] * inv);
  *reinterpret_cast<uint4*>(out + (static_cast<size_t>(token) * n_heads + e.head) * D + c * 8) = o4;
}

// The same merge for query tiles that were cut into MANY pieces (the pieces of one pair in the shared queue of the
// dynamic tail can run to dozens): one block per ROW, the parts dealt over COMBINE_LANES groups of threads that each
// merge their share as above, then one group merges the groups' results through shared memory.  With one thread
// walking all parts of its row the launch ended with a few blocks each waiting on twenty memory round trips in turn.
constexpr int COMBINE_LANES = 16;
constexpr int COMBINE_LONG_PARTS = 16;  // entries with more parts than this go through combine_long_kernel

template <int D>
__global__ void __launch_bounds__(COMBINE_LANES * (D / 8))
combine_long_kernel(const CombineEntry* entries, const CellGeom* cells, const float* part_o, const float2* part_ml,
                    __nv_bfloat16* out, int n_heads, int tokens_per_frame, int grid_w) {
  constexpr int CHUNKS = D / 8;
  __shared__ float sh_m[COMBINE_LANES], sh_l[COMBINE_LANES];
  __shared__ float sh_acc[COMBINE_LANES][D];
  const CombineEntry e = entries[blockIdx.x / 128];
  const int r = blockIdx.x % 128;
  if (r >= e.q_count) return;  // the whole block leaves: no barrier is missed
  const int c = threadIdx.x % CHUNKS, lane = threadIdx.x / CHUNKS;
  const size_t row0 = static_cast<size_t>(e.first_slot) * 256 + e.sub * 128 + r;
  const int n = e.n_parts;
  float m = -INFINITY;
  for (int i = lane; i < n; i += COMBINE_LANES) m = fmaxf(m, __ldg(&part_ml[row0 + static_cast<size_t>(i) * 256]).x);
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, l = 0.f;
  for (int i = lane; i < n; i += COMBINE_LANES) {
    const size_t row = row0 + static_cast<size_t>(i) * 256;
    const float2 ml = __ldg(&part_ml[row]);
    const float4* src = reinterpret_cast<const float4*>(part_o + row * D + c * 8);
    const float4 a = ld_stream_f4(src), b = ld_stream_f4(src + 1);
    const float wgt = (ml.x == -INFINITY) ? 0.f : ex2_approx(ml.x - m);
    l += wgt * ml.y;
    acc[0] += wgt * a.x; acc[1] += wgt * a.y; acc[2] += wgt * a.z; acc[3] += wgt * a.w;
    acc[4] += wgt * b.x; acc[5] += wgt * b.y; acc[6] += wgt * b.z; acc[7] += wgt * b.w;
  }
  if (c == 0) {
    sh_m[lane] = m;
    sh_l[lane] = l;
  }
#pragma unroll
  for (int k = 0; k < 8; ++k) sh_acc[lane][c * 8 + k] = acc[k];
  __syncthreads();
  if (lane != 0) return;
  float m_all = -INFINITY;
#pragma unroll
  for (int g = 0; g < COMBINE_LANES; ++g) m_all = fmaxf(m_all, sh_m[g]);
  float l_all = 0.f;
#pragma unroll
  for (int k = 0; k < 8; ++k) acc[k] = 0.f;
  for (int g = 0; g < COMBINE_LANES; ++g) {
    const float wgt = (sh_m[g] == -INFINITY) ? 0.f : ex2_approx(sh_m[g] - m_all);
    l_all += wgt * sh_l[g];
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] += wgt * sh_acc[g][c * 8 + k];
  }
  const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
  int token = e.q_start + r;
  if (e.cell >= 0) token = cell_query_token(cells[e.cell], token, tokens_per_frame, grid_w);
  uint4 o4;
  o4.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
  o4.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
  o4.z = pack_bf16x2(acc[4] * inv, acc[5] * inv);
  o4.w = pack_bf16x2(acc[6] * inv, acc[7] * inv);
  *reinterpret_cast<uint4*>(out + (static_cast<size_t>(token) * n_heads + e.head) * D + c * 8) = o4;
}

}  // namespace hc
