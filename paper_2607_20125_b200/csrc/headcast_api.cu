// C ABI of the HeadCast attention path (see include/headcast.h): context, state machine, cache ring,
// tile scheduling, and the launches of the kernels in attn_kernel.cuh / copy_kernels.cuh /
// score_kernels.cuh.  No CPU fallback exists: every step of the path runs in those kernels.
#include "context.h"
#include "schedule.h"

namespace {

int upload_schedule(headcast_ctx* c, Schedule& s, cudaStream_t st) {
  if (s.uploaded) return HC_OK;
  HC_CUDA(c, s.items_dev.reserve(std::max<size_t>(1, s.items.size())));
  HC_CUDA(c, s.cta_first_dev.reserve(s.cta_first.size()));
  HC_CUDA(c, s.combine_dev.reserve(std::max<size_t>(1, s.combine.size())));
  if (!s.items.empty())
    HC_CUDA(c, cudaMemcpyAsync(s.items_dev.ptr, s.items.data(), s.items.size() * sizeof(WorkItem),
                               cudaMemcpyHostToDevice, st));
  HC_CUDA(c, cudaMemcpyAsync(s.cta_first_dev.ptr, s.cta_first.data(), s.cta_first.size() * sizeof(int32_t),
                             cudaMemcpyHostToDevice, st));
  if (!s.combine.empty())
    HC_CUDA(c, cudaMemcpyAsync(s.combine_dev.ptr, s.combine.data(), s.combine.size() * sizeof(CombineEntry),
                               cudaMemcpyHostToDevice, st));
  if (!s.combine_long.empty()) {
    HC_CUDA(c, s.combine_long_dev.reserve(s.combine_long.size()));
    HC_CUDA(c, cudaMemcpyAsync(s.combine_long_dev.ptr, s.combine_long.data(), s.combine_long.size() * sizeof(CombineEntry),
                               cudaMemcpyHostToDevice, st));
  }
  if (!s.cls_groups.empty()) {
    HC_CUDA(c, s.cls_groups_dev.reserve(s.cls_groups.size()));
    HC_CUDA(c, s.cls_parts_dev.reserve(std::max<size_t>(1, s.cls_parts.size())));
    HC_CUDA(c, cudaMemcpyAsync(s.cls_groups_dev.ptr, s.cls_groups.data(), s.cls_groups.size() * sizeof(ClsGroup),
                               cudaMemcpyHostToDevice, st));
    HC_CUDA(c, cudaMemcpyAsync(s.cls_parts_dev.ptr, s.cls_parts.data(), s.cls_parts.size() * sizeof(ClsPart),
                               cudaMemcpyHostToDevice, st));
  }
  if (s.n_slots > 0) {
    HC_CUDA(c, c->part_o.reserve(static_cast<size_t>(s.n_slots) * 256 * c->D));
    HC_CUDA(c, c->part_ml.reserve(static_cast<size_t>(s.n_slots) * 256));
    HC_CUDA(c, c->part_mid.reserve(static_cast<size_t>(s.n_slots) * 256));
  }
  // The lists are uploaded once per cache fill and reused by later calls, which may come on another stream: wait
  // here, once, so that no later launch can see a half-written list (the host vectors are pageable, so the copies
  // have mostly completed by now anyway).
  HC_CUDA(c, cudaStreamSynchronize(st));
  s.uploaded = true;
  return HC_OK;
}

template <int D, bool PROXY>
int launch_attn_t(headcast_ctx* c, const AttnParams& p, cudaStream_t st) {
  // the attribute belongs to the (function, device) pair: one flag per device, so that a process that drives several
  // GPUs sets it on each of them
  static bool configured[64] = {};
  int dev = 0;
  HC_CUDA(c, cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    HC_CUDA(c, cudaFuncSetAttribute(attn_kernel<D, PROXY>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    AttnSmem<D>::DYN_BYTES));
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  if (c->timing) HC_CUDA(c, cudaEventRecord(c->ev_a, st));
  attn_kernel<D, PROXY><<<c->n_sm, ATTN_THREADS, AttnSmem<D>::DYN_BYTES, st>>>(p);
  HC_CUDA(c, cudaGetLastError());
  if (c->timing) {
    HC_CUDA(c, cudaEventRecord(c->ev_b, st));
    c->ev_valid = true;
  }
  ++c->launches;
  return HC_OK;
}

int run_schedule(headcast_ctx* c, Schedule& s, const void* q, void* out, bool proxy, cudaStream_t st) {
  int rc = upload_schedule(c, s, st);
  if (rc != HC_OK) return rc;
  if (s.items.empty()) return HC_OK;
  AttnParams p;
  std::memset(&p, 0, sizeof(p));
  p.items = s.items_dev.ptr;
  p.cta_first = s.cta_first_dev.ptr;
  static_assert(sizeof(p.maps) == sizeof(c->maps), "one K and one V map per buffer");
  std::memcpy(p.maps, c->maps, sizeof(p.maps));
  p.cells = c->cells_dev;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.part_o = c->part_o.ptr;
  p.part_ml = c->part_ml.ptr;
  p.part_mid = c->part_mid.ptr;
  p.n_heads = c->H;
  p.tokens_per_frame = c->T_f;
  p.grid_w = c->G_w;
  p.block_tokens = c->L;
  p.scale_log2e = c->scale * 1.4426950408889634f;
  p.status = c->status_dev;
  p.dyn_first = s.dyn_first;
  p.dyn_end = s.dyn_end;
  p.dyn_counter = c->dyn_counter_dev;
  p.trace = nullptr;
  if (c->tracing) {
    const size_t trace_words = 2 * s.items.size();
    HC_CUDA(c, c->trace_dev.reserve(trace_words));
    HC_CUDA(c, cudaMemsetAsync(c->trace_dev.ptr, 0, trace_words * sizeof(unsigned long long), st));
    p.trace = c->trace_dev.ptr;
    c->trace_items = s.items;
    c->trace_cta_first = s.cta_first;
  }
  p.radius = c->cfg.proxy_radius;
  if (proxy) {
    const int newest = c->slots.back();
    p.mid_seg_lo = c->F_b;
    p.mid_seg_hi = n_filled(c) * c->F_b;
    p.last_seg_lo = newest * c->F_b;
    p.last_seg_hi = (newest + 1) * c->F_b;
  }
  if (c->D == 128)
    rc = proxy ? launch_attn_t<128, true>(c, p, st) : launch_attn_t<128, false>(c, p, st);
  else
    rc = proxy ? launch_attn_t<64, true>(c, p, st) : launch_attn_t<64, false>(c, p, st);
  if (rc != HC_OK) return rc;
  if (!s.cls_groups.empty()) {
    // classification: merge the pieces of every query pair and score its rows (score_kernels.cuh)
    const unsigned blocks = static_cast<unsigned>(s.cls_groups.size()) * 2 * (128 / COMBINE_ROWS);
    const unsigned threads = COMBINE_ROWS * (c->D / 8);
    if (proxy) {
      if (c->D == 128)
        proxy_combine_kernel<128><<<blocks, threads, 0, st>>>(s.cls_groups_dev.ptr, s.cls_parts_dev.ptr, c->part_o.ptr, c->part_ml.ptr,
                                                              c->part_mid.ptr, c->cls_o.ptr, c->cls_lse.ptr, c->cls_tok.ptr, c->H, c->L);
      else
        proxy_combine_kernel<64><<<blocks, threads, 0, st>>>(s.cls_groups_dev.ptr, s.cls_parts_dev.ptr, c->part_o.ptr, c->part_ml.ptr,
                                                             c->part_mid.ptr, c->cls_o.ptr, c->cls_lse.ptr, c->cls_tok.ptr, c->H, c->L);
    } else {
      if (c->D == 128)
        cls_combine_kernel<128><<<blocks, threads, 0, st>>>(s.cls_groups_dev.ptr, s.cls_parts_dev.ptr, c->part_o.ptr, c->part_ml.ptr,
                                                            c->cls_o.ptr, c->cls_lse.ptr, c->cls_tok.ptr, c->H, c->L);
      else
        cls_combine_kernel<64><<<blocks, threads, 0, st>>>(s.cls_groups_dev.ptr, s.cls_parts_dev.ptr, c->part_o.ptr, c->part_ml.ptr,
                                                           c->cls_o.ptr, c->cls_lse.ptr, c->cls_tok.ptr, c->H, c->L);
    }
    HC_CUDA(c, cudaGetLastError());
    ++c->launches;
  }
  if (!s.combine.empty()) {
    const unsigned blocks = static_cast<unsigned>(s.combine.size()) * (128 / COMBINE_ROWS);
    if (c->D == 128)
      combine_kernel<128><<<blocks, COMBINE_ROWS * 16, 0, st>>>(s.combine_dev.ptr, c->cells_dev, c->part_o.ptr,
                                                                c->part_ml.ptr, p.out, c->H, c->T_f, c->G_w);
    else
      combine_kernel<64><<<blocks, COMBINE_ROWS * 8, 0, st>>>(s.combine_dev.ptr, c->cells_dev, c->part_o.ptr,
                                                              c->part_ml.ptr, p.out, c->H, c->T_f, c->G_w);
    HC_CUDA(c, cudaGetLastError());
    ++c->launches;
  }
  if (!s.combine_long.empty()) {
    const unsigned blocks = static_cast<unsigned>(s.combine_long.size()) * 128;  // one block per query row
    if (c->D == 128)
      combine_long_kernel<128><<<blocks, COMBINE_LANES * 16, 0, st>>>(s.combine_long_dev.ptr, c->cells_dev, c->part_o.ptr,
                                                                      c->part_ml.ptr, p.out, c->H, c->T_f, c->G_w);
    else
      combine_long_kernel<64><<<blocks, COMBINE_LANES * 8, 0, st>>>(s.combine_long_dev.ptr, c->cells_dev, c->part_o.ptr,
                                                                     c->part_ml.ptr, p.out, c->H, c->T_f, c->G_w);
    HC_CUDA(c, cudaGetLastError());
    ++c->launches;
  }
  return HC_OK;
}

// Self-test of the bounded-wait machinery: one CTA waits on an mbarrier that nobody ever arrives on, gives up after
// limit_ns, records `code` in the status word and returns normally (no trap, no fault: the context stays usable).
__global__ void bounded_wait_selftest_kernel(int32_t* status, unsigned long long limit_ns, int code) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  volatile int* abortp = &abort_flag;
  mbar_wait_limit(&bar, 0, abortp, status, code, limit_ns);  // every thread waits; the first to expire raises the flag
}

void fill_route(headcast_ctx* c, RouteParams& r) {
  std::memset(&r, 0, sizeof(r));
  r.mono_k = reinterpret_cast<uint4*>(c->mono_k);
  r.mono_v = reinterpret_cast<uint4*>(c->mono_v);
  r.sd_k = reinterpret_cast<uint4*>(c->sd_k);
  r.sd_v = reinterpret_cast<uint4*>(c->sd_v);
  r.g_k = reinterpret_cast<uint4*>(c->g_k);
  r.g_v = reinterpret_cast<uint4*>(c->g_v);
  r.sp_k = reinterpret_cast<uint4*>(c->sp_k);
  r.sp_v = reinterpret_cast<uint4*>(c->sp_v);
  r.sp_base = c->sp_base;
  r.sp_nc = c->sp_nc;
  r.L = c->L;
  r.H = c->H;
  r.chunks = c->CH;
  r.tokens_per_frame = c->T_f;
  r.frames_per_block = c->F_b;
  r.n_blocks = c->n_blk;
  r.n_sink = c->n_cls[CLS_SINK];
  r.sd_slots = c->sd_slots;
  for (int i = 0; i < MAX_BLOCKS; ++i) r.sd_slot_sink[i] = r.sd_slot_dummy[i] = -1;
  for (int h = 0; h < c->H; ++h) {
    r.cls[h] = (c->state == STATE_SPLIT || c->sd_k || c->g_k || c->sp_k) ? c->cls[h] : static_cast<int8_t>(CLS_NONE);
    r.idx[h] = c->idx[h];
  }
}

// Source tensor maps of the bulk path for a [rows][H*d] tensor at k / v.
bool build_move_maps(headcast_ctx* c, headcast_ctx::MoveMaps& m, const void* k, const void* v, uint64_t rows) {
  const uint64_t row_elems = static_cast<uint64_t>(c->H) * c->D;
  const uint32_t tile_rows = MOVE_STAGE_BYTES / (c->D * 2);
  const void* base[2] = {k, v};
  for (int kv = 0; kv < 2; ++kv) {
    if (!make_tmap_bf16_rows(&m.rows[kv], base[kv], row_elems, rows, c->D, tile_rows)) return false;
    for (size_t s = 0; s < c->move_shapes.size(); ++s)
      if (!make_tmap_bf16_grid(&m.box[kv][s], base[kv], row_elems, rows, c->G_w, c->D, c->move_shapes[s].cw, c->move_shapes[s].rows))
        return false;
  }
  m.k = k;
  m.v = v;
  return true;
}

// The same routing as route_block_kernel (RouteParams says which source block feeds which buffer), as bulk tile jobs.
int launch_move(headcast_ctx* c, const RouteParams& r, int n_src, cudaStream_t st) {
  static bool configured[64] = {};
  int dev = 0;
  HC_CUDA(c, cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    HC_CUDA(c, cudaFuncSetAttribute(move_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MOVE_SMEM_BYTES));
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  MoveParams p;
  std::memset(&p, 0, sizeof(p));
  const headcast_ctx::MoveMaps* maps = nullptr;
  if (r.src_stride != 0) {
    maps = &c->move_mono;
  } else {
    for (auto& m : c->move_recent)
      if (m.k == r.src_k && m.v == r.src_v && m.k) maps = &m;
    if (!maps) {
      headcast_ctx::MoveMaps& m = c->move_recent[c->move_next];
      c->move_next = (c->move_next + 1) % 8;
      m.k = m.v = nullptr;
      if (!build_move_maps(c, m, r.src_k, r.src_v, c->L)) return fail(c, HC_ERR_CUDA, "cuTensorMapEncodeTiled failed for the block to append");
      maps = &m;
    }
  }
  std::memcpy(p.map_rows, maps->rows, sizeof(p.map_rows));
  std::memcpy(p.map_box, maps->box, sizeof(p.map_box));
  p.src_k = reinterpret_cast<const __nv_bfloat16*>(r.src_k);
  p.src_v = reinterpret_cast<const __nv_bfloat16*>(r.src_v);
  p.mono_k = reinterpret_cast<__nv_bfloat16*>(r.mono_k);
  p.mono_v = reinterpret_cast<__nv_bfloat16*>(r.mono_v);
  p.sd_k = reinterpret_cast<__nv_bfloat16*>(r.sd_k);
  p.sd_v = reinterpret_cast<__nv_bfloat16*>(r.sd_v);
  p.g_k = reinterpret_cast<__nv_bfloat16*>(r.g_k);
  p.g_v = reinterpret_cast<__nv_bfloat16*>(r.g_v);
  p.sp_k = reinterpret_cast<__nv_bfloat16*>(r.sp_k);
  p.sp_v = reinterpret_cast<__nv_bfloat16*>(r.sp_v);
  p.boxes = c->move_boxes_dev;
  p.status = c->status_dev;
  p.src_block_rows = r.src_stride ? c->L : 0;
  p.n_boxes = static_cast<int32_t>(c->move_boxes.size());
  p.L = c->L; p.H = c->H; p.D = c->D; p.F_b = c->F_b; p.G_h = c->G_h; p.G_w = c->G_w;
  p.n_blocks = c->n_blk;
  p.n_sink = r.n_sink;
  p.sd_slots = r.sd_slots;
  p.rows_per_tile = MOVE_STAGE_BYTES / (c->D * 2);
  p.tiles_rm = (c->L + p.rows_per_tile - 1) / p.rows_per_tile;
  p.copy_mono = r.copy_mono;
  p.copy_window = r.copy_window;
  const long long block_bytes = static_cast<long long>(c->L) * c->H * c->D * 2;
  p.mono_chunks = r.copy_mono ? static_cast<int32_t>((block_bytes + MOVE_STAGE_BYTES - 1) / MOVE_STAGE_BYTES) : 0;
  p.n_src = n_src;
  for (int h = 0; h < c->H; ++h) {
    p.cls[h] = r.cls[h];
    p.idx[h] = r.idx[h];
    if (r.cls[h] == CLS_SPATIAL && r.copy_window) p.sp[p.n_sp++] = static_cast<int8_t>(h);
  }
  for (int k = 0; k < 4; ++k)
    for (int h = 0; h < c->H; ++h) {
      const int cl = r.cls[h];
      if ((cl == CLS_GLOBAL && r.copy_window) || (cl == CLS_SINK && (k == 0 || k == 2)) || (cl == CLS_DUMMY && (k == 1 || k == 2)))
        p.rm[k][p.n_rm[k]++] = static_cast<int8_t>(h);
    }
  long long jobs = 0;
  for (int i = 0; i < n_src; ++i) {
    p.slots[i] = r.slots[i];
    p.sd_slot_sink[i] = r.sd_slot_sink[i];
    p.sd_slot_dummy[i] = r.sd_slot_dummy[i];
    p.kind[i] = r.kind[i];
    p.job_first[i] = static_cast<int32_t>(jobs);
    jobs += 2ll * (static_cast<long long>(p.n_rm[p.kind[i]]) * p.tiles_rm + static_cast<long long>(p.n_sp) * p.F_b * p.n_boxes + p.mono_chunks);
  }
  p.job_first[n_src] = static_cast<int32_t>(jobs);
  if (jobs == 0) return HC_OK;
  if (jobs >= (1ll << 31)) return fail(c, HC_ERR_UNSUPPORTED, "too many tile jobs");
  const int ctas = static_cast<int>(std::min<long long>(c->n_sm, (jobs + MOVE_ENGINES - 1) / MOVE_ENGINES));
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(ctas);
  lc.blockDim = dim3(MOVE_ENGINES * 32);
  lc.dynamicSmemBytes = MOVE_SMEM_BYTES;
  lc.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see the kernel: it waits for its predecessor itself
  attr.val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = &attr;
  lc.numAttrs = 1;
  HC_CUDA(c, cudaLaunchKernelEx(&lc, move_kernel, p));
  HC_CUDA(c, cudaGetLastError());
  ++c->launches;
  return HC_OK;
}

int launch_route(headcast_ctx* c, RouteParams& r, int n_src, cudaStream_t st) {
  // which heads each kind of source row feeds (see RouteParams::kind)
  for (int k = 0; k < 4; ++k) {
    r.n_kept[k] = 0;
    for (int h = 0; h < r.H; ++h) {
      const int cl = r.cls[h];
      const bool keep = r.copy_mono || ((cl == CLS_GLOBAL || cl == CLS_SPATIAL) && r.copy_window) ||
                        (cl == CLS_SINK && (k == 0 || k == 2)) || (cl == CLS_DUMMY && (k == 1 || k == 2));
      if (keep) r.kept[k][r.n_kept[k]++] = static_cast<int8_t>(h);
    }
  }
  int max_kept = 0;
  for (int i = 0; i < n_src; ++i) {
    const bool s = r.sd_slot_sink[i] >= 0, d = r.sd_slot_dummy[i] >= 0;
    r.kind[i] = static_cast<int8_t>(s && d ? 2 : s ? 0 : d ? 1 : 3);
    max_kept = std::max<int>(max_kept, r.n_kept[r.kind[i]]);
  }
  if (max_kept == 0) return HC_OK;  // nothing to move (e.g. an append when every head is a Sink head)
  if (c->move_ok) return launch_move(c, r, n_src, st);
  const int per_token = max_kept * r.chunks;  // <= 64 heads * 16 chunks = 1024
  const int tokens_per_iter = std::max(1, 256 / per_token);
  const int threads = tokens_per_iter * per_token;
  const int resident = std::max(1, 2048 / threads);  // blocks per SM
  const int per_src = std::max(1, (c->n_sm * resident + n_src - 1) / n_src);
  const int needed = (r.L + tokens_per_iter * ROUTE_UNROLL - 1) / (tokens_per_iter * ROUTE_UNROLL);
  route_block_kernel<<<dim3(std::max(1, std::min(needed, per_src)), n_src), threads, 0, st>>>(r);
  HC_CUDA(c, cudaGetLastError());
  ++c->launches;
  return HC_OK;
}

int read_status(headcast_ctx* c, cudaStream_t st) {
  int32_t status = 0;
  HC_CUDA(c, cudaMemcpyAsync(&status, c->status_dev, sizeof(status), cudaMemcpyDeviceToHost, st));
  HC_CUDA(c, cudaStreamSynchronize(st));
  if (status != 0) {
    cudaMemsetAsync(c->status_dev, 0, sizeof(int32_t), st);
    cudaMemsetAsync(c->dyn_counter_dev, 0, 2 * sizeof(int32_t), st);  // a kernel that gave up may have left the queue half drawn
    return fail(c, HC_ERR_TIMEOUT, "a kernel gave up on a bounded wait (site %d)", status);
  }
  return HC_OK;
}

void assign_classes(headcast_ctx* c) {
  for (int k = 0; k < 4; ++k) c->n_cls[k] = 0;
  for (int h = 0; h < c->H; ++h) {
    c->cls[h] = static_cast<int8_t>(c->labels[h]);
    c->idx[h] = static_cast<int8_t>(c->n_cls[c->labels[h]]++);
  }
}

}  // namespace

// Host-only half of headcast_create: validates cfg and fills sizes, cell geometry and the cell-major token tables.
static int init_host(headcast_ctx* c, const headcast_config* cfg, std::vector<int32_t>& sp_base, std::vector<int32_t>& sp_nc) {
  if (cfg->n_heads < 1 || cfg->n_heads > MAX_HEADS || (cfg->head_dim != 64 && cfg->head_dim != 128) ||
      cfg->grid_h < 1 || cfg->grid_w < 1 || cfg->frames_per_block < 1 || cfg->n_blocks < 2 ||
      cfg->n_blocks > MAX_BLOCKS || cfg->cell_h < 1 || cfg->cell_w < 1 || cfg->proxy_radius < 0 ||
      !(cfg->softmax_scale >= 0.0f) || cfg->sd_mode < 0 || cfg->sd_mode > 1 || cfg->rule < 0 || cfg->rule > 1 ||
      (cfg->rule == 1 && !(cfg->mass_tau > 0.0f && cfg->mass_tau <= 1.0f)))
    return HC_ERR_INVALID_ARG;
  const long long L = static_cast<long long>(cfg->frames_per_block) * cfg->grid_h * cfg->grid_w;
  if (L * cfg->n_blocks * cfg->n_heads * cfg->head_dim >= (1LL << 40) || L * cfg->n_blocks * cfg->n_heads >= (1LL << 31))
    return HC_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->H = cfg->n_heads;
  c->D = cfg->head_dim;
  c->G_h = cfg->grid_h;
  c->G_w = cfg->grid_w;
  c->F_b = cfg->frames_per_block;
  c->T_f = cfg->grid_h * cfg->grid_w;
  c->L = static_cast<int>(L);
  c->n_blk = cfg->n_blocks;
  c->CH = c->D / 8;
  c->sd_slots = cfg->sd_mode ? 2 : 1;
  c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt(static_cast<float>(c->D));
  c->row_edges = (cfg->row_edges_host && cfg->n_row_edges > 0)
                     ? std::vector<int>(cfg->row_edges_host, cfg->row_edges_host + cfg->n_row_edges)
                     : default_edges(c->G_h, cfg->cell_h);
  c->col_edges = (cfg->col_edges_host && cfg->n_col_edges > 0)
                     ? std::vector<int>(cfg->col_edges_host, cfg->col_edges_host + cfg->n_col_edges)
                     : default_edges(c->G_w, cfg->cell_w);
  c->cfg.row_edges_host = c->cfg.col_edges_host = nullptr;
  if (!edges_ok(c->row_edges, c->G_h) || !edges_ok(c->col_edges, c->G_w)) return HC_ERR_INVALID_ARG;
  c->labels.assign(c->H, HC_GLOBAL);
  for (int h = 0; h < c->H; ++h) {
    c->cls[h] = CLS_NONE;
    c->idx[h] = 0;
  }
  // deployed cells and the cell-major token order of the Spatial buffers
  sp_base.assign(c->T_f, 0);
  sp_nc.assign(c->T_f, 0);
  int tok_off = 0;
  for (size_t i = 0; i + 1 < c->row_edges.size(); ++i)
    for (size_t j = 0; j + 1 < c->col_edges.size(); ++j) {
      CellGeom g = {c->row_edges[i], c->col_edges[j], c->row_edges[i + 1] - c->row_edges[i],
                    c->col_edges[j + 1] - c->col_edges[j]};
      c->cells.push_back(g);
      c->cell_tok_off.push_back(tok_off);
      for (int dy = 0; dy < g.ch; ++dy)
        for (int dx = 0; dx < g.cw; ++dx) {
          const int pos = (g.y0 + dy) * c->G_w + g.x0 + dx;
          sp_base[pos] = c->n_blk * c->F_b * tok_off + dy * g.cw + dx;
          sp_nc[pos] = g.ch * g.cw;
        }
      tok_off += g.ch * g.cw;
    }
  // bulk tile movement: every cell (or, for a cell larger than a stage, every band of its rows) is one rectangle of
  // the token grid; rectangles of equal (width, rows) share a tensor map
  const int stage_tokens = MOVE_STAGE_BYTES / (c->D * 2);
  c->move_ok = true;
  c->move_boxes.clear();
  c->move_shapes.clear();
  for (size_t ci = 0; ci < c->cells.size() && c->move_ok; ++ci) {
    const CellGeom& g = c->cells[ci];
    if (g.cw > stage_tokens || g.cw > 256) {
      c->move_ok = false;
      break;
    }
    const int rb = std::min(std::min(g.ch, 256), std::max(1, stage_tokens / g.cw));
    int shape = -1;
    for (size_t s = 0; s < c->move_shapes.size(); ++s)
      if (c->move_shapes[s].cw == g.cw && c->move_shapes[s].rows == rb) shape = static_cast<int>(s);
    if (shape < 0) {
      if (c->move_shapes.size() == MOVE_MAX_SHAPES) {
        c->move_ok = false;
        break;
      }
      shape = static_cast<int>(c->move_shapes.size());
      c->move_shapes.push_back({g.cw, rb});
    }
    for (int r0 = 0; r0 < g.ch; r0 += rb) {
      MoveBox b;
      b.y0 = g.y0 + r0;
      b.x0 = g.x0;
      b.cw = g.cw;
      b.rows = std::min(rb, g.ch - r0);
      b.shape = shape;
      b.box_tokens = g.cw * rb;
      b.cell_tok_off = c->cell_tok_off[ci];
      b.nc = g.ch * g.cw;
      b.first_tok = r0 * g.cw;
      c->move_boxes.push_back(b);
    }
  }
  return HC_OK;
}

// =====================================================================================================
extern "C" {

void headcast_default_config(headcast_config* cfg) {
  if (!cfg) return;
  std::memset(cfg, 0, sizeof(*cfg));
  cfg->frames_per_block = 3;
  cfg->cell_h = 10;
  cfg->cell_w = 10;
  cfg->proxy_radius = 2;
  cfg->theta_sink = cfg->theta_dummy = cfg->theta_spatial = 0.95f;
  cfg->theta_score = 0.755f;
  cfg->gamma = 5.0f;
  cfg->softmax_scale = 0.0f;
  cfg->rule = HC_RULE_COSINE;
  cfg->mass_tau = 0.9f;
}

int headcast_create(const headcast_config* cfg, headcast_ctx** out) {
  if (!cfg || !out) return HC_ERR_INVALID_ARG;
  *out = nullptr;
  headcast_ctx* c = new (std::nothrow) headcast_ctx();
  if (!c) return HC_ERR_NOMEM;
  std::vector<int32_t> sp_base, sp_nc;
  {
    const int rc = init_host(c, cfg, sp_base, sp_nc);
    if (rc != HC_OK) {
      delete c;
      return rc;
    }
  }
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    delete c;
    return HC_ERR_CUDA;
  }
  if (prop.major != 10) {
    delete c;
    return HC_ERR_UNSUPPORTED;
  }
  c->n_sm = prop.multiProcessorCount;
  const size_t mono_bytes = cache_elems(c, c->H) * sizeof(__nv_bfloat16);
  cudaError_t e = cudaSuccess;
  auto step = [&](cudaError_t r) { if (e == cudaSuccess) e = r; };
  // the monolithic cache comes from the stream-ordered allocator, so that the split can release it in stream order
  // (cudaFreeAsync) instead of stalling the host and the device in a cudaFree
  step(cudaMallocAsync(reinterpret_cast<void**>(&c->mono_k), mono_bytes, nullptr));
  step(cudaMallocAsync(reinterpret_cast<void**>(&c->mono_v), mono_bytes, nullptr));
  step(cudaMalloc(&c->arena_k, mono_bytes));
  step(cudaMalloc(&c->arena_v, mono_bytes));
  step(cudaMalloc(&c->sp_base, c->T_f * sizeof(int32_t)));
  step(cudaMalloc(&c->sp_nc, c->T_f * sizeof(int32_t)));
  step(cudaMalloc(&c->cells_dev, c->cells.size() * sizeof(CellGeom)));
  step(cudaMalloc(&c->status_dev, sizeof(int32_t)));
  step(cudaMalloc(&c->dyn_counter_dev, 2 * sizeof(int32_t)));
  if (e == cudaSuccess) step(cudaMemset(c->dyn_counter_dev, 0, 2 * sizeof(int32_t)));
  if (c->move_ok) step(cudaMalloc(&c->move_boxes_dev, std::max<size_t>(1, c->move_boxes.size()) * sizeof(MoveBox)));
  if (e == cudaSuccess) {
    step(cudaMemset(c->mono_k, 0, mono_bytes));
    step(cudaMemset(c->mono_v, 0, mono_bytes));
    step(cudaMemset(c->arena_k, 0, mono_bytes));
    step(cudaMemset(c->arena_v, 0, mono_bytes));
    step(cudaMemset(c->status_dev, 0, sizeof(int32_t)));
    step(cudaMemcpy(c->sp_base, sp_base.data(), c->T_f * sizeof(int32_t), cudaMemcpyHostToDevice));
    step(cudaMemcpy(c->sp_nc, sp_nc.data(), c->T_f * sizeof(int32_t), cudaMemcpyHostToDevice));
    step(cudaMemcpy(c->cells_dev, c->cells.data(), c->cells.size() * sizeof(CellGeom), cudaMemcpyHostToDevice));
    if (c->move_ok && !c->move_boxes.empty())
      step(cudaMemcpy(c->move_boxes_dev, c->move_boxes.data(), c->move_boxes.size() * sizeof(MoveBox), cudaMemcpyHostToDevice));
  }
  if (e == cudaSuccess && c->move_ok &&
      !build_move_maps(c, c->move_mono, c->mono_k, c->mono_v, static_cast<uint64_t>(c->n_blk) * c->L))
    c->move_ok = false;  // the per-thread copy kernel serves every geometry

  int rc = HC_OK;
  if (e != cudaSuccess) rc = (e == cudaErrorMemoryAllocation) ? HC_ERR_NOMEM : HC_ERR_CUDA;
  if (rc == HC_OK) rc = build_maps(c);
  if (rc == HC_OK && cudaDeviceSynchronize() != cudaSuccess) rc = HC_ERR_CUDA;
  if (rc != HC_OK) {
    headcast_destroy(c);
    return rc;
  }
  *out = c;
  return HC_OK;
}

int headcast_destroy(headcast_ctx* c) {
  if (!c) return HC_OK;
  cudaDeviceSynchronize();
  if (c->mono_k) cudaFreeAsync(c->mono_k, nullptr);
  if (c->mono_v) cudaFreeAsync(c->mono_v, nullptr);
  cudaDeviceSynchronize();
  void* ptrs[] = {c->arena_k, c->arena_v, c->sp_base, c->sp_nc, c->cells_dev, c->status_dev, c->dyn_counter_dev, c->move_boxes_dev};
  for (void* p : ptrs)
    if (p) cudaFree(p);
  if (c->ev_a) cudaEventDestroy(c->ev_a);
  if (c->ev_b) cudaEventDestroy(c->ev_b);
  c->sched_dense.release();
  c->sched_hc.release();
  c->sched_cls.release();
  c->sched_proxy.release();
  for (Schedule& g : c->sched_stage) g.release();
  c->stage_q.release();
  c->stage_out.release();
  c->stage_k.release();
  c->stage_v.release();
  if (c->copy_in) cudaStreamDestroy(c->copy_in);
  if (c->copy_out) cudaStreamDestroy(c->copy_out);
  for (cudaEvent_t e : c->ev_host)
    if (e) cudaEventDestroy(e);
  c->part_o.release();
  c->part_ml.release();
  c->part_mid.release();
  c->trace_dev.release();
  c->cls_o.release();
  c->cls_lse.release();
  c->cls_tok.release();
  c->cls_scores.release();
  c->cls_labels.release();
  delete c;
  return HC_OK;
}

int headcast_append(headcast_ctx* c, const void* k_new, const void* v_new, void* stream) {
  if (!c) return HC_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new)) return fail(c, HC_ERR_INVALID_ARG, "k_new/v_new must be 16-byte aligned device pointers");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // ring bookkeeping: the sink block never moves; when full, the oldest rolling block's slot is reused
  int slot;
  std::vector<int> next = c->slots;
  if (static_cast<int>(next.size()) < c->n_blk) {
    slot = static_cast<int>(next.size());
    next.push_back(slot);
  } else if (c->n_blk == 1) {
    slot = 0;
  } else {
    slot = next[1];
    next.erase(next.begin() + 1);
    next.push_back(slot);
  }
  const bool split = c->state == STATE_SPLIT;
  const int dummy_next = (c->sd_slots == 2) ? (c->dummy_cur ^ 1) : 0;  // the older of a Dummy head's two blocks is replaced
  RouteParams r;
  fill_route(c, r);
  r.src_k = static_cast<const uint4*>(k_new);
  r.src_v = static_cast<const uint4*>(v_new);
  r.slots[0] = static_cast<int8_t>(slot);
  r.src_stride = 0;
  r.copy_mono = c->mono_k != nullptr;
  r.sd_slot_sink[0] = static_cast<int8_t>((split && c->sd_slots == 2) ? 1 : -1);  // the anchor block stays frozen
  r.sd_slot_dummy[0] = static_cast<int8_t>(split ? dummy_next : -1);
  r.copy_window = split;
  int rc = launch_route(c, r, 1, st);
  if (rc != HC_OK) return rc;
  c->slots.swap(next);
  if (split) {
    c->dummy_cur = dummy_next;
    c->sd_valid = c->sd_slots;
  }
  return HC_OK;
}

int headcast_overwrite_last(headcast_ctx* c, const void* k_new, const void* v_new, void* stream) {
  if (!c) return HC_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new)) return fail(c, HC_ERR_INVALID_ARG, "k_new/v_new must be 16-byte aligned device pointers");
  if (c->slots.empty()) return fail(c, HC_ERR_STATE, "the cache is empty");
  const bool split = c->state == STATE_SPLIT;
  RouteParams r;
  fill_route(c, r);
  r.src_k = static_cast<const uint4*>(k_new);
  r.src_v = static_cast<const uint4*>(v_new);
  r.slots[0] = static_cast<int8_t>(c->slots.back());
  r.src_stride = 0;
  r.copy_mono = c->mono_k != nullptr;
  r.sd_slot_sink[0] = static_cast<int8_t>((split && c->sd_slots == 2 && c->sd_valid == 2) ? 1 : -1);
  r.sd_slot_dummy[0] = static_cast<int8_t>(split ? c->dummy_cur : -1);
  r.copy_window = split;
  return launch_route(c, r, 1, static_cast<cudaStream_t>(stream));
}

int headcast_full_attend(headcast_ctx* c, const void* q, void* out, void* stream) {
  if (!c) return HC_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out)) return fail(c, HC_ERR_INVALID_ARG, "q/out must be 16-byte aligned device pointers");
  if (!c->mono_k) return fail(c, HC_ERR_STATE, "the monolithic cache was released at the split (keep_monolithic = 0)");
  if (c->slots.empty()) return fail(c, HC_ERR_STATE, "the cache is empty");
  if (c->sched_dense.key_filled != n_filled(c)) build_dense_schedule(c, c->sched_dense, OUT_BF16, true);
  return run_schedule(c, c->sched_dense, q, out, false, static_cast<cudaStream_t>(stream));
}

int headcast_set_labels(headcast_ctx* c, const int32_t* labels) {
  if (!c || !labels) return HC_ERR_INVALID_ARG;
  if (c->state != STATE_FILLING) return fail(c, HC_ERR_STATE, "labels are fixed once the cache is split");
  for (int h = 0; h < c->H; ++h)
    if (labels[h] < 0 || labels[h] > 3) return fail(c, HC_ERR_INVALID_ARG, "label %d of head %d is not an archetype", labels[h], h);
  c->labels.assign(labels, labels + c->H);
  c->have_labels = true;
  return HC_OK;
}

int headcast_get_labels(const headcast_ctx* c, int32_t* labels) {
  if (!c || !labels) return HC_ERR_INVALID_ARG;
  if (!c->have_labels) return HC_ERR_STATE;
  std::copy(c->labels.begin(), c->labels.end(), labels);
  return HC_OK;
}

int headcast_classify(headcast_ctx* c, const void* q, int32_t* labels_host, float* scores_host, void* stream) {
  if (!c || !labels_host) return HC_ERR_INVALID_ARG;
  if (!aligned16(q)) return fail(c, HC_ERR_INVALID_ARG, "q must be a 16-byte aligned device pointer");
  if (c->state != STATE_FILLING) return fail(c, HC_ERR_STATE, "classification runs on the monolithic cache, before the split");
  if (n_filled(c) < 2) return fail(c, HC_ERR_STATE, "classification needs at least two cached blocks");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t rows = static_cast<size_t>(c->L) * c->H;
  HC_CUDA(c, c->cls_o.reserve(rows * c->D));  // the reference output (fp32); the proxy outputs never leave registers
  HC_CUDA(c, c->cls_lse.reserve(rows));
  HC_CUDA(c, c->cls_tok.reserve(TOK_N * rows));
  HC_CUDA(c, c->cls_scores.reserve(static_cast<size_t>(c->H) * HC_N_SCORES));
  HC_CUDA(c, c->cls_labels.reserve(c->H));
  const int newest = c->slots.back();
  const int cls_key = n_filled(c) * 64 + newest;  // the work lists depend on the fill and on where the newest block sits
  if (c->sched_cls.key_filled != cls_key) {
    // Reference (Eq. 2), Sink proxy and Dummy proxy from one sweep over the keys: the sweep is cut into the first
    // block, the middle blocks and the newest block (physical ring slots: the middle ones are one or two runs),
    // every piece leaves a partial result and cls_combine_kernel merges them three ways.
    std::vector<Proto> protos;
    Schedule& s = c->sched_cls;
    s.cls_groups.clear();
    const int nf = n_filled(c);
    struct Range { int slot_lo, slot_hi, tag; };
    std::vector<Range> ranges;
    ranges.push_back({0, 1, 0});
    if (newest > 1) ranges.push_back({1, newest, 1});
    if (newest + 1 < nf) ranges.push_back({newest + 1, nf, 1});
    if (newest != 0) ranges.push_back({newest, newest + 1, 2});
    for (int h = 0; h < c->H; ++h)
      for (int q0 = 0; q0 < c->L; q0 += 256) {
        ClsGroup g;
        g.head = h;
        g.q_start = q0;
        g.q_count[0] = std::min(128, c->L - q0);
        g.q_count[1] = std::max(0, std::min(128, c->L - q0 - 128));
        g.first_part = 0;
        g.n_parts = 0;
        const int group = static_cast<int>(s.cls_groups.size());
        s.cls_groups.push_back(g);
        for (const Range& r : ranges) {
          WorkItem w = range_item(h, MAP_MONO, h * c->D, static_cast<long long>(r.slot_lo) * c->L, (r.slot_hi - r.slot_lo) * c->L);
          Proto p;
          p.w = w;
          p.w.q_start[0] = q0;
          p.w.q_start[1] = q0 + 128;
          p.w.q_count[0] = g.q_count[0];
          p.w.q_count[1] = g.q_count[1];
          p.n_tiles = w.tiles_per_seg;
          p.w.tile_begin = 0;
          p.w.tile_end = p.n_tiles;
          p.cls_group = group;
          p.cls_tag = r.tag;
          protos.push_back(p);
        }
      }
    finalize_schedule(c, s, protos, true);
    s.key_filled = cls_key;
  }
  // the reference sweep is on its way before the host builds the proxy's work list
  int rc = run_schedule(c, c->sched_cls, q, nullptr, false, st);
  if (rc != HC_OK) return rc;
  if (c->sched_proxy.key_filled != cls_key) {
    // Spatial proxy: per query-tile pair, the band of grid rows within r of any of its queries, in every cached frame
    std::vector<Proto> protos;
    c->sched_proxy.cls_groups.clear();
    const int r = c->cfg.proxy_radius;
    for (int h = 0; h < c->H; ++h)
      for (int q0 = 0; q0 < c->L; q0 += 256) {
        const int q1 = std::min(c->L, q0 + 256) - 1;
        int a = 0, b = c->T_f;
        if (q0 / c->T_f == q1 / c->T_f) {
          const int ylo = std::max(0, (q0 % c->T_f) / c->G_w - r), yhi = std::min(c->G_h - 1, (q1 % c->T_f) / c->G_w + r);
          a = ylo * c->G_w;
          b = (yhi + 1) * c->G_w;
        }
        WorkItem w = range_item(h, MAP_MONO, h * c->D, a, b - a);
        w.seg_stride = c->T_f;
        Proto p;
        p.w = w;
        p.w.q_start[0] = q0;
        p.w.q_start[1] = q0 + 128;
        p.w.q_count[0] = std::min(128, c->L - q0);
        p.w.q_count[1] = std::max(0, std::min(128, c->L - q0 - 128));
        p.n_tiles = w.tiles_per_seg * n_filled(c) * c->F_b;
        p.w.tile_begin = 0;
        p.w.tile_end = p.n_tiles;
        // whole or cut into pieces, a band leaves partial results that proxy_combine_kernel merges and scores
        ClsGroup g;
        g.head = h;
        g.q_start = q0;
        g.q_count[0] = p.w.q_count[0];
        g.q_count[1] = p.w.q_count[1];
        g.first_part = 0;
        g.n_parts = 0;
        p.cls_group = static_cast<int>(c->sched_proxy.cls_groups.size());
        p.cls_tag = 0;
        c->sched_proxy.cls_groups.push_back(g);
        protos.push_back(p);
      }
    finalize_schedule(c, c->sched_proxy, protos, true);
    c->sched_proxy.key_filled = cls_key;
  }
  rc = run_schedule(c, c->sched_proxy, q, nullptr, true, st);
  if (rc != HC_OK) return rc;
  {
    DecideParams d;
    d.tok = c->cls_tok.ptr;
    d.scores = c->cls_scores.ptr;
    d.labels = c->cls_labels.ptr;
    d.L = c->L;
    d.H = c->H;
    d.D = c->D;
    const double rank = 0.05 * (c->L - 1);
    d.rank_lo = static_cast<int32_t>(std::floor(rank));
    d.rank_frac = static_cast<float>(rank - std::floor(rank));
    d.theta_sink = c->cfg.theta_sink;
    d.theta_dummy = c->cfg.theta_dummy;
    d.theta_spatial = c->cfg.theta_spatial;
    d.theta_score = c->cfg.theta_score;
    d.gamma = c->cfg.gamma;
    d.rule = c->cfg.rule;
    d.mass_tau = c->cfg.mass_tau;
    head_decide_kernel<<<c->H, 1024, 0, st>>>(d);
    HC_CUDA(c, cudaGetLastError());
    ++c->launches;
  }
  std::vector<float> scores(static_cast<size_t>(c->H) * HC_N_SCORES);
  HC_CUDA(c, cudaMemcpyAsync(labels_host, c->cls_labels.ptr, c->H * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  HC_CUDA(c, cudaMemcpyAsync(scores.data(), c->cls_scores.ptr, scores.size() * sizeof(float), cudaMemcpyDeviceToHost, st));
  rc = read_status(c, st);
  if (rc != HC_OK) return rc;
  if (scores_host) std::copy(scores.begin(), scores.end(), scores_host);
  c->labels.assign(labels_host, labels_host + c->H);
  c->have_labels = true;
  return HC_OK;
}

int headcast_split_cache(headcast_ctx* c, void* stream) {
  if (!c) return HC_ERR_INVALID_ARG;
  if (c->state != STATE_FILLING) return fail(c, HC_ERR_STATE, "the cache is already split");
  if (!c->have_labels) return fail(c, HC_ERR_STATE, "no labels: call headcast_classify or headcast_set_labels first");
  if (c->slots.empty()) return fail(c, HC_ERR_STATE, "the cache is empty");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  assign_classes(c);
  // carve the three buffers out of the arena reserved (and zeroed) at create: no allocation on this path
  const int n_sd = c->n_cls[CLS_SINK] + c->n_cls[CLS_DUMMY];
  const size_t sd_elems = static_cast<size_t>(n_sd) * c->sd_slots * c->L * c->D;
  const size_t g_elems = cache_elems(c, c->n_cls[CLS_GLOBAL]);
  const size_t sp_elems = cache_elems(c, c->n_cls[CLS_SPATIAL]);
  c->sd_k = sd_elems ? c->arena_k : nullptr;
  c->sd_v = sd_elems ? c->arena_v : nullptr;
  c->g_k = g_elems ? c->arena_k + sd_elems : nullptr;
  c->g_v = g_elems ? c->arena_v + sd_elems : nullptr;
  c->sp_k = sp_elems ? c->arena_k + sd_elems + g_elems : nullptr;
  c->sp_v = sp_elems ? c->arena_v + sd_elems + g_elems : nullptr;
  {
    // one launch: grid row i gathers cached block i (ring slot slots[i]) out of the monolithic cache
    RouteParams r;
    fill_route(c, r);
    r.src_k = reinterpret_cast<const uint4*>(c->mono_k);
    r.src_v = reinterpret_cast<const uint4*>(c->mono_v);
    r.src_stride = static_cast<long long>(c->L) * c->H * c->CH;
    for (size_t i = 0; i < c->slots.size(); ++i) r.slots[i] = static_cast<int8_t>(c->slots[i]);
    r.copy_mono = 0;
    const int n = static_cast<int>(c->slots.size());
    r.sd_slot_sink[0] = 0;  // the first block is the Sink heads' anchor
    if (c->sd_slots == 2 && n >= 2) {
      r.sd_slot_sink[n - 1] = 1;   // anchor + current block
      r.sd_slot_dummy[n - 2] = 0;  // previous + current block
      r.sd_slot_dummy[n - 1] = 1;
      c->dummy_cur = 1;
      c->sd_valid = 2;
    } else {
      r.sd_slot_dummy[n - 1] = 0;
      c->dummy_cur = 0;
      c->sd_valid = 1;
    }
    r.copy_window = 1;
    int rc = launch_route(c, r, static_cast<int>(c->slots.size()), st);
    if (rc != HC_OK) return rc;
  }
  if (!c->cfg.keep_monolithic) {  // released in stream order, after the gather that reads it
    HC_CUDA(c, cudaFreeAsync(c->mono_k, st));
    HC_CUDA(c, cudaFreeAsync(c->mono_v, st));
    c->mono_k = c->mono_v = nullptr;
  }
  c->state = STATE_SPLIT;
  c->sched_hc.key_filled = -1;
  return build_maps(c);
}

int headcast_attend(headcast_ctx* c, const void* q, void* out, void* stream) {
  if (!c) return HC_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out)) return fail(c, HC_ERR_INVALID_ARG, "q/out must be 16-byte aligned device pointers");
  if (c->state != STATE_SPLIT) return fail(c, HC_ERR_STATE, "head-specific attention needs the split cache");
  if (c->sched_hc.key_filled != n_filled(c) * 4 + c->sd_valid) build_headcast_schedule(c, c->sched_hc);
  return run_schedule(c, c->sched_hc, q, out, false, static_cast<cudaStream_t>(stream));
}

namespace {

int init_host_path(headcast_ctx* c) {
  if (!c->copy_in) HC_CUDA(c, cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking));
  if (!c->copy_out) HC_CUDA(c, cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking));
  for (cudaEvent_t& e : c->ev_host)
    if (!e) HC_CUDA(c, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  return HC_OK;
}

}  // namespace

int headcast_append_host(headcast_ctx* c, const void* k_host, const void* v_host, void* stream) {
  if (!c || !k_host || !v_host) return HC_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t elems = static_cast<size_t>(c->L) * c->H * c->D;
  HC_CUDA(c, c->stage_k.reserve(elems));
  HC_CUDA(c, c->stage_v.reserve(elems));
  HC_CUDA(c, cudaMemcpyAsync(c->stage_k.ptr, k_host, elems * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice, st));
  HC_CUDA(c, cudaMemcpyAsync(c->stage_v.ptr, v_host, elems * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice, st));
  return headcast_append(c, c->stage_k.ptr, c->stage_v.ptr, stream);
}

int headcast_attend_host(headcast_ctx* c, const void* q_host, void* out_host, void* stream) {
  if (!c || !q_host || !out_host) return HC_ERR_INVALID_ARG;
  if (c->state != STATE_SPLIT) return fail(c, HC_ERR_STATE, "head-specific attention needs the split cache");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = init_host_path(c);
  if (rc != HC_OK) return rc;
  const size_t elems = static_cast<size_t>(c->L) * c->H * c->D;
  HC_CUDA(c, c->stage_q.reserve(elems));
  HC_CUDA(c, c->stage_out.reserve(elems));
  const int key = n_filled(c) * 4 + c->sd_valid;
  // Stages: a stage's queries are copied in (strided: the rows of [L][H][d] hold all heads), attended and copied out
  // as a unit, so that the next stage's queries arrive and the previous stage's outputs leave while this stage
  // computes.  The Global heads do most of the arithmetic per byte moved, so their query rows are halved (at a
  // multiple of 256 rows: the query-tile pairs stay the same) and the halves go first and last: the kernels start
  // after a small copy, and when they end only a small copy is left; the other heads' copies hide in between.
  const int mid = std::min(c->L, ((c->L / 2 + 255) / 256) * 256);  // blocks of up to 256 tokens have one stage per group
  struct Stage { int group, lo, hi; };
  const Stage stages[headcast_ctx::N_HOST_STAGES] = {{0, 0, mid}, {2, 0, c->L}, {1, 0, c->L}, {0, mid, c->L}};
  for (int i = 0; i < headcast_ctx::N_HOST_STAGES; ++i)
    if (c->sched_stage[i].key_filled != key)
      build_headcast_schedule(c, c->sched_stage[i], stages[i].group, stages[i].lo, stages[i].hi);
  const size_t pitch = static_cast<size_t>(c->H) * c->D * sizeof(__nv_bfloat16);
  auto copy_stage = [&](const Stage& sg, bool in) -> int {
    const int rows = sg.hi - sg.lo;
    if (rows <= 0) return HC_OK;
    for (int h0 = 0; h0 < c->H;) {
      auto group_of = [&](int h) { return c->cls[h] == CLS_GLOBAL ? 0 : c->cls[h] == CLS_SPATIAL ? 1 : 2; };
      if (group_of(h0) != sg.group) {
        ++h0;
        continue;
      }
      int h1 = h0 + 1;
      while (h1 < c->H && group_of(h1) == sg.group) ++h1;
      const size_t off = static_cast<size_t>(sg.lo) * c->H * c->D + static_cast<size_t>(h0) * c->D;
      const size_t width = static_cast<size_t>(h1 - h0) * c->D * sizeof(__nv_bfloat16);
      if (in)
        HC_CUDA(c, cudaMemcpy2DAsync(c->stage_q.ptr + off, pitch, static_cast<const __nv_bfloat16*>(q_host) + off, pitch, width,
                                     rows, cudaMemcpyHostToDevice, c->copy_in));
      else
        HC_CUDA(c, cudaMemcpy2DAsync(static_cast<__nv_bfloat16*>(out_host) + off, pitch, c->stage_out.ptr + off, pitch, width,
                                     rows, cudaMemcpyDeviceToHost, c->copy_out));
      h0 = h1;
    }
    return HC_OK;
  };
  // everything enqueued on `stream` before this call (an append, the previous call's copies) comes first
  HC_CUDA(c, cudaEventRecord(c->ev_host[0], st));
  HC_CUDA(c, cudaStreamWaitEvent(c->copy_in, c->ev_host[0], 0));
  HC_CUDA(c, cudaStreamWaitEvent(c->copy_out, c->ev_host[0], 0));
  for (int i = 0; i < headcast_ctx::N_HOST_STAGES; ++i) {
    if (c->sched_stage[i].items.empty()) continue;
    if ((rc = copy_stage(stages[i], true)) != HC_OK) return rc;
    HC_CUDA(c, cudaEventRecord(c->ev_host[2 + 2 * i], c->copy_in));
    HC_CUDA(c, cudaStreamWaitEvent(st, c->ev_host[2 + 2 * i], 0));
    if ((rc = run_schedule(c, c->sched_stage[i], c->stage_q.ptr, c->stage_out.ptr, false, st)) != HC_OK) return rc;
    HC_CUDA(c, cudaEventRecord(c->ev_host[3 + 2 * i], st));
    HC_CUDA(c, cudaStreamWaitEvent(c->copy_out, c->ev_host[3 + 2 * i], 0));
    if ((rc = copy_stage(stages[i], false)) != HC_OK) return rc;
  }
  HC_CUDA(c, cudaEventRecord(c->ev_host[1], c->copy_out));
  HC_CUDA(c, cudaStreamWaitEvent(st, c->ev_host[1], 0));
  return HC_OK;
}

int headcast_export_cache(headcast_ctx* c, int32_t head, void* k_out, void* v_out, int32_t* n_tokens_host, void* stream) {
  if (!c || head < 0 || head >= c->H) return HC_ERR_INVALID_ARG;
  if ((k_out && !aligned16(k_out)) || (v_out && !aligned16(v_out))) return fail(c, HC_ERR_INVALID_ARG, "outputs must be 16-byte aligned");
  ExportParams e;
  std::memset(&e, 0, sizeof(e));
  e.dst_k = static_cast<uint4*>(k_out);
  e.dst_v = static_cast<uint4*>(v_out);
  e.sp_base = c->sp_base;
  e.sp_nc = c->sp_nc;
  e.L = c->L;
  e.H = c->H;
  e.chunks = c->CH;
  e.tokens_per_frame = c->T_f;
  e.frames_per_block = c->F_b;
  e.n_blocks = c->n_blk;
  e.sd_slots = c->sd_slots;
  const int cl = (c->state == STATE_SPLIT) ? static_cast<int>(c->cls[head]) : static_cast<int>(CLS_NONE);
  if (cl == CLS_NONE) {
    e.layout = 0; e.head = head; e.src_k = reinterpret_cast<const uint4*>(c->mono_k); e.src_v = reinterpret_cast<const uint4*>(c->mono_v);
  } else if (cl == CLS_GLOBAL) {
    e.layout = 1; e.head = c->idx[head]; e.src_k = reinterpret_cast<const uint4*>(c->g_k); e.src_v = reinterpret_cast<const uint4*>(c->g_v);
  } else if (cl == CLS_SPATIAL) {
    e.layout = 2; e.head = c->idx[head]; e.src_k = reinterpret_cast<const uint4*>(c->sp_k); e.src_v = reinterpret_cast<const uint4*>(c->sp_v);
  } else {
    e.layout = 3; e.head = (cl == CLS_SINK) ? c->idx[head] : c->n_cls[CLS_SINK] + c->idx[head];
    e.src_k = reinterpret_cast<const uint4*>(c->sd_k); e.src_v = reinterpret_cast<const uint4*>(c->sd_v);
  }
  if (e.layout == 3) {
    e.n_logical = c->sd_valid;
    if (cl == CLS_SINK) {
      e.slots[0] = 0;
      e.slots[1] = 1;
    } else if (c->sd_valid == 2) {
      e.slots[0] = c->dummy_cur ^ 1;  // previous block first
      e.slots[1] = c->dummy_cur;
    } else {
      e.slots[0] = c->dummy_cur;
    }
  } else {
    e.n_logical = n_filled(c);
    for (int i = 0; i < e.n_logical; ++i) e.slots[i] = c->slots[i];
  }
  if (n_tokens_host) *n_tokens_host = e.n_logical * c->L;
  if (e.n_logical == 0 || (!k_out && !v_out)) return HC_OK;
  const long long total = static_cast<long long>(e.n_logical) * c->L * c->CH;
  const int blocks = static_cast<int>(std::min<long long>((total + 255) / 256, c->n_sm * 16LL));
  export_head_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(e);
  HC_CUDA(c, cudaGetLastError());
  ++c->launches;
  return HC_OK;
}

int headcast_n_filled(const headcast_ctx* c) { return c ? n_filled(c) : HC_ERR_INVALID_ARG; }

int64_t headcast_launch_count(const headcast_ctx* c) { return c ? c->launches : 0; }

double headcast_attend_flops(const headcast_ctx* c, int32_t dense) {
  if (!c) return 0.0;
  const int nf = n_filled(c);
  if (dense) return 4.0 * c->H * static_cast<double>(c->L) * nf * c->L * c->D;
  if (!c->have_labels) return 0.0;
  double cell_sq = 0.0;
  for (const CellGeom& g : c->cells) cell_sq += static_cast<double>(g.ch * g.cw) * (g.ch * g.cw);
  double f = 0.0;
  for (int h = 0; h < c->H; ++h) {
    if (c->labels[h] == HC_SINK || c->labels[h] == HC_DUMMY)
      f += 4.0 * c->L * static_cast<double>(c->state == STATE_SPLIT ? c->sd_valid : std::min(c->sd_slots, nf)) * c->L * c->D;
    else if (c->labels[h] == HC_GLOBAL) f += 4.0 * c->L * static_cast<double>(nf) * c->L * c->D;
    else f += 4.0 * c->F_b * static_cast<double>(nf) * c->F_b * cell_sq * c->D;
  }
  return f;
}

int headcast_set_kernel_timing(headcast_ctx* c, int32_t enable) {
  if (!c) return HC_ERR_INVALID_ARG;
  if (enable && !c->ev_a) {
    HC_CUDA(c, cudaEventCreate(&c->ev_a));
    HC_CUDA(c, cudaEventCreate(&c->ev_b));
  }
  c->timing = enable != 0;
  c->ev_valid = false;
  return HC_OK;
}

int headcast_last_attention_kernel_ms(headcast_ctx* c, float* ms_host) {
  if (!c || !ms_host) return HC_ERR_INVALID_ARG;
  if (!c->ev_valid) return fail(c, HC_ERR_STATE, "no attention kernel was timed yet");
  HC_CUDA(c, cudaEventSynchronize(c->ev_b));
  HC_CUDA(c, cudaEventElapsedTime(ms_host, c->ev_a, c->ev_b));
  return HC_OK;
}

int headcast_set_tracing(headcast_ctx* c, int32_t enable) {
  if (!c) return HC_ERR_INVALID_ARG;
  c->tracing = enable != 0;
  return HC_OK;
}

int headcast_read_trace(headcast_ctx* c, int64_t* rows_host, int32_t capacity, int32_t* n_items_host) {
  if (!c || !n_items_host) return HC_ERR_INVALID_ARG;
  const int n = static_cast<int>(c->trace_items.size());
  *n_items_host = n;
  if (!rows_host || n == 0) return HC_OK;
  HC_CUDA(c, cudaDeviceSynchronize());
  std::vector<unsigned long long> t(2 * static_cast<size_t>(n));
  HC_CUDA(c, cudaMemcpy(t.data(), c->trace_dev.ptr, t.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  int cta = 0;
  for (int i = 0; i < n && i < capacity; ++i) {
    while (cta + 1 < static_cast<int>(c->trace_cta_first.size()) && c->trace_cta_first[cta + 1] <= i) ++cta;
    const WorkItem& w = c->trace_items[i];
    int64_t* r = rows_host + 8 * static_cast<size_t>(i);
    r[0] = cta;
    r[1] = w.head;
    r[2] = w.cell;
    r[3] = w.q_count[0] + w.q_count[1];
    r[4] = w.tile_end - w.tile_begin;
    r[5] = w.out_mode;
    r[6] = static_cast<int64_t>(t[2 * i]);
    r[7] = static_cast<int64_t>(t[2 * i + 1]);
  }
  return HC_OK;
}

int headcast_plan_schedule(const headcast_config* cfg, const int32_t* labels_host, int32_t n_filled, int32_t n_ctas,
                           int32_t dense, int32_t* items_host, int32_t capacity, int32_t* n_items_host,
                           int32_t* cta_first_host) {
  if (!cfg || !n_items_host || n_filled < 1 || n_ctas < 1 || n_ctas > 4096) return HC_ERR_INVALID_ARG;
  headcast_ctx c;
  std::vector<int32_t> sp_base, sp_nc;
  int rc = init_host(&c, cfg, sp_base, sp_nc);
  if (rc != HC_OK) return rc;
  if (n_filled > c.n_blk) return HC_ERR_INVALID_ARG;
  c.n_sm = n_ctas;
  for (int i = 0; i < n_filled; ++i) c.slots.push_back(i);
  Schedule s;
  if (dense) {
    build_dense_schedule(&c, s, OUT_BF16, true);
  } else {
    if (!labels_host) return HC_ERR_INVALID_ARG;
    for (int h = 0; h < c.H; ++h)
      if (labels_host[h] < 0 || labels_host[h] > 3) return HC_ERR_INVALID_ARG;
    c.labels.assign(labels_host, labels_host + c.H);
    assign_classes(&c);
    c.sd_valid = std::min(c.sd_slots, n_filled);
    c.dummy_cur = c.sd_valid - 1;
    build_headcast_schedule(&c, s);
  }
  *n_items_host = static_cast<int32_t>(s.items.size());
  static_assert(sizeof(WorkItem) == 16 * sizeof(int32_t), "work items are exported as 16 int32 each");
  if (items_host)
    std::memcpy(items_host, s.items.data(), std::min<size_t>(s.items.size(), capacity) * sizeof(WorkItem));
  if (cta_first_host) std::copy(s.cta_first.begin(), s.cta_first.end(), cta_first_host);
  return HC_OK;
}

int headcast_selftest_bounded_wait(headcast_ctx* c, int32_t limit_ms, void* stream) {
  if (!c || limit_ms < 1 || limit_ms > 1000) return HC_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(c->status_dev, static_cast<unsigned long long>(limit_ms) * 1000000ull, 99);
  HC_CUDA(c, cudaGetLastError());
  ++c->launches;
  return read_status(c, st);
}

int headcast_check(headcast_ctx* c, void* stream) {
  if (!c) return HC_ERR_INVALID_ARG;
  return read_status(c, static_cast<cudaStream_t>(stream));
}

const char* headcast_last_error(const headcast_ctx* c) { return c ? c->err.c_str() : "null context"; }

}  // extern "C"

// =====================================================================================================
// Allocation-free dense attention
// =====================================================================================================
// Everything the attention kernel needs in global memory besides the caller's tensors - the work list, the per-CTA
// ranges and the status word - lives in one file-scope device array of fixed size (the two tensor maps travel as
// kernel parameters).  Each GPU that loads the
// library carries these bytes until the process exits.
namespace {

constexpr int NOALLOC_MAX_ITEMS = HEADCAST_NOALLOC_MAX_ITEMS;
constexpr int NOALLOC_MAX_CTAS = 1024;

struct NoAllocScratch {
  WorkItem items[NOALLOC_MAX_ITEMS];
  int32_t cta_first[NOALLOC_MAX_CTAS + 1];
  int32_t status;
};

static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

constexpr int NOALLOC_MAX_DEVICES = 64;
struct NoAllocDevice {
  NoAllocScratch* scratch = nullptr;  // device address of g_noalloc_scratch on that GPU
  int n_sm = 0;
};
NoAllocDevice g_noalloc_dev[NOALLOC_MAX_DEVICES];

char g_noalloc_error[256] = "";

int noalloc_fail(int code, const char* msg, cudaError_t e = cudaSuccess) {
  if (e != cudaSuccess)
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s: %s", msg, cudaGetErrorString(e));
  else
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s", msg);
  return code;
}

// Once per device, with that device current: the array's name is only a host-side handle, the kernel needs the
// address cudaGetSymbolAddress reports for the current device.
int noalloc_setup(int dev) {
  NoAllocDevice& d = g_noalloc_dev[dev];
  if (d.scratch) return HC_OK;
  cudaDeviceProp prop;
  cudaError_t e = cudaGetDeviceProperties(&prop, dev);
  if (e != cudaSuccess) return noalloc_fail(HC_ERR_CUDA, "cudaGetDeviceProperties", e);
  if (prop.major != 10) return noalloc_fail(HC_ERR_UNSUPPORTED, "this library needs an sm_100 device");
  void* ptr = nullptr;
  e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
  if (e != cudaSuccess || !ptr) return noalloc_fail(HC_ERR_CUDA, "cudaGetSymbolAddress(g_noalloc_scratch)", e);
  e = cudaFuncSetAttribute(attn_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<128>::DYN_BYTES);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(attn_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<64>::DYN_BYTES);
  if (e != cudaSuccess) return noalloc_fail(HC_ERR_CUDA, "cudaFuncSetAttribute", e);
  d.n_sm = std::min(prop.multiProcessorCount, NOALLOC_MAX_CTAS);
  d.scratch = static_cast<NoAllocScratch*>(ptr);
  return HC_OK;
}

}  // namespace

extern "C" {

int headcast_dense_attend_noalloc(const void* q, const void* k, const void* v, void* out, int32_t n_queries,
                                  int32_t n_keys, int32_t n_heads, int32_t head_dim, float softmax_scale, void* stream) {
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
    return noalloc_fail(HC_ERR_INVALID_ARG, "q, k, v and out must be 16-byte aligned device pointers");
  if (n_queries < 1 || n_keys < 1 || n_heads < 1 || n_heads > MAX_HEADS || (head_dim != 64 && head_dim != 128) ||
      !(softmax_scale >= 0.f))
    return noalloc_fail(HC_ERR_INVALID_ARG, "sizes out of range (head_dim 64 or 128, 1..64 heads)");
  const long long n_items = static_cast<long long>(n_heads) * ((n_queries + 255) / 256);
  if (n_items > NOALLOC_MAX_ITEMS)
    return noalloc_fail(HC_ERR_UNSUPPORTED,
                        "too large for the fixed scratch: n_heads * ceil(n_queries / 256) must not exceed "
                        "HEADCAST_NOALLOC_MAX_ITEMS");
  if (static_cast<long long>(n_keys) * n_heads * head_dim >= (1LL << 40) || static_cast<long long>(n_queries) * n_heads >= (1LL << 31))
    return noalloc_fail(HC_ERR_INVALID_ARG, "sizes out of range");
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return noalloc_fail(HC_ERR_CUDA, "cudaGetDevice", e);
  if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return noalloc_fail(HC_ERR_UNSUPPORTED, "device index beyond 63");
  int rc = noalloc_setup(dev);
  if (rc != HC_OK) return rc;
  const NoAllocDevice& d = g_noalloc_dev[dev];
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    // the work list is copied from a host image that the next call rewrites: a captured copy would re-read it at
    // every replay, so capturing streams are turned away
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    e = cudaStreamIsCapturing(st, &cap);
    if (e != cudaSuccess) return noalloc_fail(HC_ERR_CUDA, "cudaStreamIsCapturing", e);
    if (cap != cudaStreamCaptureStatusNone)
      return noalloc_fail(HC_ERR_UNSUPPORTED, "headcast_dense_attend_noalloc cannot be called on a capturing stream");
  }

  // host image of the scratch: thread-local static storage, no heap
  static thread_local NoAllocScratch host;
  const uint64_t row_elems = static_cast<uint64_t>(n_heads) * head_dim;
  AttnParams p;
  std::memset(&p, 0, sizeof(p));
  if (!make_tmap_bf16_2d(&p.maps[0], k, row_elems, n_keys, row_elems, 128) ||
      !make_tmap_bf16_2d(&p.maps[1], v, row_elems, n_keys, row_elems, 128))
    return noalloc_fail(HC_ERR_CUDA, "cuTensorMapEncodeTiled failed or is unavailable");
  // whole query-tile pairs, dealt round-robin to one CTA per SM (every item has the same key range)
  const int n_cta = d.n_sm;
  int n = 0;
  for (int b = 0; b < n_cta; ++b) {
    host.cta_first[b] = n;
    for (long long i = b; i < n_items; i += n_cta) {
      const int h = static_cast<int>(i % n_heads), q0 = static_cast<int>(i / n_heads) * 256;
      WorkItem w = range_item(h, 0, h * head_dim, 0, n_keys);
      w.q_start[0] = q0;
      w.q_start[1] = q0 + 128;
      w.q_count[0] = std::min(128, n_queries - q0);
      w.q_count[1] = std::max(0, std::min(128, n_queries - q0 - 128));
      w.tile_begin = 0;
      w.tile_end = w.tiles_per_seg;
      host.items[n++] = w;
    }
  }
  host.cta_first[n_cta] = n;
  host.status = 0;  // the array keeps the previous call's contents: the status word must start at zero
  e = cudaMemcpyAsync(d.scratch->items, host.items, static_cast<size_t>(n) * sizeof(WorkItem), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(d.scratch->cta_first, host.cta_first, (n_cta + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(&d.scratch->status, &host.status, sizeof(int32_t), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return noalloc_fail(HC_ERR_CUDA, "copying the work list into the static scratch", e);

  p.items = d.scratch->items;
  p.cta_first = d.scratch->cta_first;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.n_heads = n_heads;
  p.tokens_per_frame = n_queries;
  p.grid_w = 1;
  p.block_tokens = n_queries;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / std::sqrt(static_cast<float>(head_dim));
  p.scale_log2e = scale * 1.4426950408889634f;
  p.status = &d.scratch->status;
  if (head_dim == 128)
    attn_kernel<128, false><<<n_cta, ATTN_THREADS, AttnSmem<128>::DYN_BYTES, st>>>(p);
  else
    attn_kernel<64, false><<<n_cta, ATTN_THREADS, AttnSmem<64>::DYN_BYTES, st>>>(p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return noalloc_fail(HC_ERR_CUDA, "launching the attention kernel", e);
  return HC_OK;
}

int headcast_noalloc_status(void* stream) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES || !g_noalloc_dev[dev].scratch)
    return noalloc_fail(HC_ERR_STATE, "headcast_dense_attend_noalloc has not run on this device");
  int32_t status = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(&status, &g_noalloc_dev[dev].scratch->status, sizeof(status), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return noalloc_fail(HC_ERR_CUDA, "reading the status word", e);
  if (status != 0) return noalloc_fail(HC_ERR_TIMEOUT, "the attention kernel gave up on a bounded wait");
  return HC_OK;
}

const char* headcast_noalloc_last_error(void) { return g_noalloc_error; }

}  // extern "C"
