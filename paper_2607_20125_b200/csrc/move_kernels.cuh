// Cache split and append as bulk asynchronous tile movement (TMA in, bulk copy out).
//
// The caller's block is [L][H][d]: one head's rows are d*2 bytes long and H*d*2 bytes apart.  Every destination
// (a head's rows in the Sink-Dummy or Global buffer, one Spatial cell of one frame, a slot of the monolithic
// ring) is contiguous.  So a job is: one tiled TMA load that gathers a box out of the strided source into shared
// memory - (d columns x R tokens) for the row-major buffers, (d x cell width x cell rows) of the token grid for a
// Spatial cell, which arrives in exactly the cell-major order - followed by ONE contiguous bulk store of the valid
// bytes.  No thread touches the data; no register staging; a ragged last tile just stores fewer bytes.
//
// A CTA runs MOVE_ENGINES independent engines (lane 0 of each warp) with a private shared-memory stage and mbarrier
// each: decode job -> wait until the stage's previous store has read it -> load -> wait (bounded) -> store.
// Jobs are dealt round-robin over all engines of the grid, so neighbouring engines touch neighbouring memory.
#pragma once
#include "copy_kernels.cuh"
#include "tc05.cuh"

namespace hc {

constexpr int MOVE_ENGINES = 7;
constexpr int MOVE_STAGE_BYTES = 32768;
constexpr int MOVE_MAX_SHAPES = 4;
constexpr int MOVE_SMEM_BYTES = MOVE_ENGINES * MOVE_STAGE_BYTES + 128;

// One rectangle of the token grid that is moved as a unit for a Spatial head: `rows` grid rows, `cw` tokens wide,
// starting at (y0, x0) - a whole cell, or a band of its rows if the cell does not fit a stage.
struct MoveBox {
  int32_t y0, x0, cw, rows;
  int32_t shape;         // index of the tensor map whose box is (d, cw, box rows >= rows)
  int32_t box_tokens;    // tokens in that full box
  int32_t cell_tok_off;  // tokens per frame in earlier cells
  int32_t nc;            // tokens per frame in this cell
  int32_t first_tok;     // index of the box's first token inside its cell
};

struct MoveParams {
  const __nv_bfloat16 *src_k, *src_v;  // source base (caller's block, or the monolithic cache)
  __nv_bfloat16 *mono_k, *mono_v, *sd_k, *sd_v, *g_k, *g_v, *sp_k, *sp_v;
  const MoveBox* boxes;
  int32_t* status;
  long long src_block_rows;  // rows between consecutive source blocks (0: there is only the caller's block)
  int32_t n_boxes, L, H, D, F_b, G_h, G_w, n_blocks, n_sink, sd_slots;
  int32_t rows_per_tile, tiles_rm, mono_chunks, copy_mono, copy_window, n_src;
  int32_t job_first[MAX_BLOCKS + 1];  // jobs of source block y are [job_first[y], job_first[y + 1])
  int8_t slots[MAX_BLOCKS], sd_slot_sink[MAX_BLOCKS], sd_slot_dummy[MAX_BLOCKS], kind[MAX_BLOCKS];
  int8_t n_rm[4], rm[4][MAX_HEADS];  // heads kept in a row-major buffer, per kind of source block (see RouteParams)
  int8_t n_sp, sp[MAX_HEADS];        // Spatial heads
  int8_t cls[MAX_HEADS], idx[MAX_HEADS];
  // [0] K, [1] V.  rows: 2-D (H*d, rows), box (d, rows_per_tile); box[s]: grid view, box (d, cw_s, rows_s)
  alignas(64) CUtensorMap map_rows[2];
  CUtensorMap map_box[2][MOVE_MAX_SHAPES];
};

__device__ __forceinline__ void bulk_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void bulk_load_3d(void* dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void bulk_load_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void bulk_store_1d(void* dst, const void* src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(reinterpret_cast<uint64_t>(dst)), "r"(smem_u32(src_smem)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__global__ void __launch_bounds__(MOVE_ENGINES * 32, 1) move_kernel(const __grid_constant__ MoveParams p) {
  extern __shared__ uint8_t move_smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(move_smem_raw) + 127) & ~uintptr_t(127));
  __shared__ uint64_t bar[MOVE_ENGINES];
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    for (int e = 0; e < MOVE_ENGINES; ++e) mbar_init(&bar[e], 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  // Programmatic dependent launch: the kernel is launched with stream serialisation relaxed, so its CTAs may become
  // resident and set up their barriers while the kernel before it on the stream drains.  launch_dependents lets the
  // NEXT such kernel do the same with this one; wait returns once the preceding kernel has completed and its writes
  // are visible, and comes before this kernel's first access to global memory.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if ((threadIdx.x & 31) != 0) return;
  const int e = threadIdx.x >> 5;
  uint8_t* stage = smem + e * MOVE_STAGE_BYTES;
  volatile int* abortp = &abort_flag;
  const uint64_t pol = l2_policy_evict_first();  // the source is read once
  const int total = p.job_first[p.n_src];
  const int row_bytes = p.D * 2;
  const long long block_elems = static_cast<long long>(p.L) * p.H * p.D;
  uint32_t phase = 0;
  int y = 0;
  for (int j = blockIdx.x * MOVE_ENGINES + e; j < total; j += gridDim.x * MOVE_ENGINES) {
    while (j >= p.job_first[y + 1]) ++y;
    int jj = j - p.job_first[y];
    const int kv = jj & 1;
    jj >>= 1;
    const int slot = p.slots[y], kind = p.kind[y];
    const long long src_row0 = p.src_block_rows * slot;  // first source row of this block
    const int n_rm_jobs = p.n_rm[kind] * p.tiles_rm;
    const int n_sp_jobs = p.copy_window ? p.n_sp * p.F_b * p.n_boxes : 0;
    __nv_bfloat16* dst = nullptr;
    uint32_t box_bytes = 0, store_bytes = 0;
    bulk_wait_read0();  // the previous store of this engine has read the stage
    if (jj < n_rm_jobs) {
      // ---- d columns x rows_per_tile tokens of one head -> contiguous rows of its buffer
      const int a = jj / p.tiles_rm, tile = jj - a * p.tiles_rm;
      const int h = p.rm[kind][a], cl = p.cls[h], ix = p.idx[h];
      const int t0 = tile * p.rows_per_tile;
      long long row;  // destination row
      if (cl == CLS_SINK) {
        dst = kv ? p.sd_v : p.sd_k;
        row = (static_cast<long long>(ix) * p.sd_slots + p.sd_slot_sink[y]) * p.L + t0;
      } else if (cl == CLS_DUMMY) {
        dst = kv ? p.sd_v : p.sd_k;
        row = (static_cast<long long>(p.n_sink + ix) * p.sd_slots + p.sd_slot_dummy[y]) * p.L + t0;
      } else {
        dst = kv ? p.g_v : p.g_k;
        row = (static_cast<long long>(ix) * p.n_blocks + slot) * p.L + t0;
      }
      dst += row * p.D;
      box_bytes = p.rows_per_tile * row_bytes;
      store_bytes = min(p.rows_per_tile, p.L - t0) * row_bytes;
      mbar_arrive_expect_tx(&bar[e], box_bytes);
      bulk_load_2d(stage, &p.map_rows[kv], h * p.D, static_cast<int>(src_row0 + t0), &bar[e], pol);
    } else if (jj < n_rm_jobs + n_sp_jobs) {
      // ---- one rectangle of the token grid of one frame -> its place in the cell-major Spatial buffer
      jj -= n_rm_jobs;
      const int b = jj % p.n_boxes;
      const int rest = jj / p.n_boxes;
      const int f = rest % p.F_b, a = rest / p.F_b;
      const int h = p.sp[a], ix = p.idx[h];
      const MoveBox bx = p.boxes[b];
      const long long row = static_cast<long long>(ix) * p.n_blocks * p.L +
                            static_cast<long long>(p.n_blocks) * p.F_b * bx.cell_tok_off +
                            static_cast<long long>(slot * p.F_b + f) * bx.nc + bx.first_tok;
      dst = (kv ? p.sp_v : p.sp_k) + row * p.D;
      // the load always brings the map's full box; only the valid rows are stored
      const CUtensorMap* map = &p.map_box[kv][bx.shape];
      box_bytes = bx.box_tokens * row_bytes;
      store_bytes = bx.rows * bx.cw * row_bytes;
      const int grid_row = static_cast<int>(src_row0 / p.G_w) + f * p.G_h + bx.y0;
      mbar_arrive_expect_tx(&bar[e], box_bytes);
      bulk_load_3d(stage, map, h * p.D, bx.x0, grid_row, &bar[e], pol);
    } else {
      // ---- monolithic ring: the block is one contiguous range
      jj -= n_rm_jobs + n_sp_jobs;
      const long long off = static_cast<long long>(jj) * (MOVE_STAGE_BYTES / 2);  // in elements
      const long long left = block_elems - off;
      store_bytes = box_bytes = static_cast<uint32_t>(min(static_cast<long long>(MOVE_STAGE_BYTES / 2), left) * 2);
      dst = (kv ? p.mono_v : p.mono_k) + static_cast<long long>(slot) * block_elems + off;
      const __nv_bfloat16* src = (kv ? p.src_v : p.src_k) + src_row0 * p.H * p.D + off;
      mbar_arrive_expect_tx(&bar[e], box_bytes);
      bulk_load_1d(stage, src, box_bytes, &bar[e], pol);
    }
    if (!mbar_wait(&bar[e], phase, abortp, p.status, 41)) break;
    phase ^= 1;
    bulk_store_1d(dst, stage, store_bytes);
    bulk_commit();
  }
  bulk_wait0();  // the stores are complete before the engine leaves
}

}  // namespace hc
