// The context behind the C ABI of include/headcast.h: device buffers, the state of the cache ring, the cached work
// lists, error reporting and the tensor maps of the cache buffers.  Private to headcast_api.cu (one translation unit).
#pragma once
#include "../../include/headcast.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <queue>
#include <string>
#include <vector>

#include "attn_kernel.cuh"
#include "copy_kernels.cuh"
#include "move_kernels.cuh"
#include "score_kernels.cuh"
#include "tmap.h"

using namespace hc;

namespace {

enum { STATE_FILLING = 0, STATE_SPLIT = 1 };
enum { MAP_MONO = 0, MAP_SD = 1, MAP_GLOBAL = 2, MAP_SPATIAL = 3, N_MAP_PAIRS = 4 };

template <typename T>
struct DevBuf {  // grow-only device array
  T* ptr = nullptr;
  size_t cap = 0;
  cudaError_t reserve(size_t n) {
    if (n <= cap) return cudaSuccess;
    if (ptr) cudaFree(ptr);
    ptr = nullptr;
    cap = 0;
    cudaError_t e = cudaMalloc(&ptr, n * sizeof(T));
    if (e == cudaSuccess) cap = n;
    return e;
  }
  void release() {
    if (ptr) cudaFree(ptr);
    ptr = nullptr;
    cap = 0;
  }
};

struct Schedule {
  int key_filled = -1;  // cache fill the lists were built for
  std::vector<WorkItem> items;
  std::vector<int32_t> cta_first;
  std::vector<CombineEntry> combine;       // query tiles to merge, up to COMBINE_LONG_PARTS pieces each
  std::vector<CombineEntry> combine_long;  // those cut into more pieces (combine_long_kernel)
  std::vector<ClsGroup> cls_groups;  // classification only: key ranges of one query pair, merged three ways
  std::vector<ClsPart> cls_parts;
  DevBuf<WorkItem> items_dev;
  DevBuf<int32_t> cta_first_dev;
  DevBuf<CombineEntry> combine_dev, combine_long_dev;
  DevBuf<ClsGroup> cls_groups_dev;
  DevBuf<ClsPart> cls_parts_dev;
  int n_slots = 0;
  int dyn_first = 0, dyn_end = 0;  // items [dyn_first, dyn_end) form the shared queue the CTAs draw from when their own list is done
  bool uploaded = false;
  double flops = 0.0;
  void release() {
    items_dev.release();
    cta_first_dev.release();
    combine_dev.release();
    combine_long_dev.release();
    cls_groups_dev.release();
    cls_parts_dev.release();
  }
};

}  // namespace

struct headcast_ctx {
  headcast_config cfg;
  int H, D, L, T_f, F_b, n_blk, CH, G_h, G_w;
  float scale;
  int state = STATE_FILLING;
  std::vector<int> slots;  // logical block -> physical ring slot (index 0 = sink block)
  bool have_labels = false;
  std::vector<int32_t> labels;
  int n_cls[4] = {0, 0, 0, 0};
  int sd_slots = 1;   // blocks per head in the Sink-Dummy buffer (2 with sd_mode 1)
  int sd_valid = 0;   // of which hold data
  int dummy_cur = 0;  // slot holding a Dummy head's newest block
  int8_t cls[MAX_HEADS], idx[MAX_HEADS];
  std::vector<int> row_edges, col_edges;
  std::vector<CellGeom> cells;
  std::vector<int> cell_tok_off;  // tokens per frame in earlier cells

  __nv_bfloat16 *mono_k = nullptr, *mono_v = nullptr;
  __nv_bfloat16 *arena_k = nullptr, *arena_v = nullptr;  // zeroed at create; the per-archetype buffers are carved from it
  __nv_bfloat16 *sd_k = nullptr, *sd_v = nullptr, *g_k = nullptr, *g_v = nullptr, *sp_k = nullptr, *sp_v = nullptr;
  int32_t *sp_base = nullptr, *sp_nc = nullptr;
  CellGeom* cells_dev = nullptr;
  CUtensorMap maps[2 * N_MAP_PAIRS];  // host copies; every attention launch carries them as kernel parameters
  // bulk tile movement (move_kernels.cuh): rectangles of the token grid per Spatial cell, their distinct box shapes,
  // and the source tensor maps - of the monolithic cache (built at create) and of recently seen caller blocks
  struct MoveShape { int cw, rows; };
  struct MoveMaps { const void *k = nullptr, *v = nullptr; CUtensorMap rows[2], box[2][MOVE_MAX_SHAPES]; };
  bool move_ok = false;     // false: the geometry does not fit the bulk path (very wide cells, too many cell shapes)
  std::vector<MoveBox> move_boxes;
  std::vector<MoveShape> move_shapes;
  MoveBox* move_boxes_dev = nullptr;
  MoveMaps move_mono;
  MoveMaps move_recent[8];
  int move_next = 0;
  int32_t* status_dev = nullptr;
  int32_t* dyn_counter_dev = nullptr;  // [2]: next queue position, CTAs done (the last one clears both)

  Schedule sched_dense, sched_hc, sched_cls, sched_proxy;
  // headcast_attend_host: the stages of its pipeline, each with its own work list - the first half of the Global
  // heads' rows, the Sink + Dummy heads, the Spatial heads, the second half of the Global heads' rows
  static constexpr int N_HOST_STAGES = 4;
  Schedule sched_stage[N_HOST_STAGES];
  DevBuf<__nv_bfloat16> stage_q, stage_out, stage_k, stage_v;  // device copies of host tensors
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  cudaEvent_t ev_host[2 + 2 * N_HOST_STAGES] = {};
  DevBuf<float> part_o;
  DevBuf<float2> part_ml;
  DevBuf<float> part_mid;
  DevBuf<float> cls_o, cls_lse, cls_tok, cls_scores;
  DevBuf<int32_t> cls_labels;

  int n_sm = 148;
  int64_t launches = 0;
  bool tracing = false;  // record per-item start/end times in the attention kernel
  DevBuf<unsigned long long> trace_dev;
  std::vector<WorkItem> trace_items;
  std::vector<int32_t> trace_cta_first;
  bool timing = false;  // record events around the attention kernel of each call
  cudaEvent_t ev_a = nullptr, ev_b = nullptr;
  bool ev_valid = false;
  std::string err;
};

namespace {

int fail(headcast_ctx* c, int code, const char* fmt, ...) {
  if (c) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    c->err = buf;
  }
  return code;
}

#define HC_CUDA(c, expr)                                                                           \
  do {                                                                                             \
    cudaError_t e_ = (expr);                                                                       \
    if (e_ != cudaSuccess)                                                                         \
      return fail((c), e_ == cudaErrorMemoryAllocation ? HC_ERR_NOMEM : HC_ERR_CUDA, "%s: %s", #expr, \
                  cudaGetErrorString(e_));                                                         \
  } while (0)

std::vector<int> default_edges(int grid, int cell) {
  const int n = std::max(1, static_cast<int>(std::floor(static_cast<double>(grid) / cell + 0.5)));
  std::vector<int> e(n + 1);
  for (int i = 0; i <= n; ++i) e[i] = static_cast<int>((static_cast<long long>(i) * grid) / n);
  return e;
}

bool edges_ok(const std::vector<int>& e, int grid) {
  if (e.size() < 2 || e.front() != 0 || e.back() != grid) return false;
  for (size_t i = 1; i < e.size(); ++i)
    if (e[i] <= e[i - 1]) return false;
  return true;
}

bool aligned16(const void* p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

size_t cache_elems(const headcast_ctx* c, int heads) {
  return static_cast<size_t>(heads) * c->n_blk * c->L * c->D;
}

// ---------------------------------------------------------------------------------- tensor maps
int build_maps(headcast_ctx* c) {
  CUtensorMap* maps = c->maps;
  std::memset(maps, 0, sizeof(c->maps));
  const uint64_t win_rows = static_cast<uint64_t>(c->n_blk) * c->L;
  bool ok = true;
  if (c->mono_k) {
    ok = ok && make_tmap_bf16_2d(&maps[2 * MAP_MONO], c->mono_k, static_cast<uint64_t>(c->H) * c->D, win_rows,
                                 static_cast<uint64_t>(c->H) * c->D, 128);
    ok = ok && make_tmap_bf16_2d(&maps[2 * MAP_MONO + 1], c->mono_v, static_cast<uint64_t>(c->H) * c->D, win_rows,
                                 static_cast<uint64_t>(c->H) * c->D, 128);
  }
  if (c->sd_k) {
    const uint64_t rows = static_cast<uint64_t>(c->n_cls[CLS_SINK] + c->n_cls[CLS_DUMMY]) * c->sd_slots * c->L;
    ok = ok && make_tmap_bf16_2d(&maps[2 * MAP_SD], c->sd_k, c->D, rows, c->D, 128);
    ok = ok && make_tmap_bf16_2d(&maps[2 * MAP_SD + 1], c->sd_v, c->D, rows, c->D, 128);
  }
  if (c->g_k) {
    const uint64_t rows = c->n_cls[CLS_GLOBAL] * win_rows;
    ok = ok && make_tmap_bf16_2d(&maps[2 * MAP_GLOBAL], c->g_k, c->D, rows, c->D, 128);
    ok = ok && make_tmap_bf16_2d(&maps[2 * MAP_GLOBAL + 1], c->g_v, c->D, rows, c->D, 128);
  }
  if (c->sp_k) {
    const uint64_t rows = c->n_cls[CLS_SPATIAL] * win_rows;
    ok = ok && make_tmap_bf16_2d(&maps[2 * MAP_SPATIAL], c->sp_k, c->D, rows, c->D, 128);
    ok = ok && make_tmap_bf16_2d(&maps[2 * MAP_SPATIAL + 1], c->sp_v, c->D, rows, c->D, 128);
  }
  if (!ok) return fail(c, HC_ERR_CUDA, "cuTensorMapEncodeTiled failed or is unavailable");
  return HC_OK;
}

}  // namespace
