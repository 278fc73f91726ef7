// One launch over several tables (Section 3.1 of the Monolith paper: a production model
// holds many embedding tables of very uneven size, most of them far too small to fill a
// GPU on their own).  Every kernel of the hot path exists a second time as a grouped
// kernel: its grid is the concatenation of the grids the tables would have launched one by
// one, a block first finds the table it belongs to, and then runs the same body on that
// table's view, scratch and batch.  The bodies are the single-table kernels' own.
#pragma once

#include "kernels_adagrad.cuh"
#include "kernels_dedup.cuh"
#include "kernels_forward.cuh"
#include "kernels_table.cuh"

namespace mono {

// One table's share of a grouped call.
struct GroupItem {
  TableView tv;
  Work wk;
  const unsigned long long* ids;
  const long long* off;
  long long n_ids, n_bags;
  float* out;                    // lookup
  uint32_t* occ_row;             // lookup: row of every occurrence
  const float* grad;             // push
  unsigned long long dedup_seed;
  uint32_t now;
  uint32_t prepared;             // lookup: 1 = rows from the per-call set (the batch was announced), 0 = from the key store
  uint32_t lane_class;           // 0..3: lane groups of 4 / 8 / 16 / 32 with one column vector per lane;
                                 // 4..6: 32 lanes with 2 / 4 / 8 vectors per lane
  uint32_t active;               // 0: the table takes no part in this call (empty batch)
};

// Which table a block of a grouped launch belongs to: start[i] .. start[i+1] are table i's
// blocks.  Returns the table and the block's number within it.
__device__ inline uint32_t find_table(const uint32_t* __restrict__ start, uint32_t n_tables, uint32_t block,
                                      uint32_t* vblock, uint32_t* vgrid) {
  uint32_t lo = 0, hi = n_tables;                        // start[lo] <= block < start[hi]
  while (hi - lo > 1) {
    const uint32_t mid = (lo + hi) >> 1;
    if (__ldg(start + mid) <= block) lo = mid; else hi = mid;
  }
  const uint32_t s0 = __ldg(start + lo), s1 = __ldg(start + lo + 1);
  *vblock = block - s0;
  *vgrid = s1 - s0;
  return lo;
}

#define MONO_GROUP_PROLOGUE                                                              \
  after_previous_kernel();                                                               \
  uint32_t vblock, vgrid;                                                                \
  const GroupItem& it = items[find_table(start, n_tables, blockIdx.x, &vblock, &vgrid)]

__global__ void __launch_bounds__(256)
group_fill_occ_bag_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  fill_occ_bag_body(it.off, it.n_bags, it.n_ids, it.wk.occ_bag, it.tv.st, vblock, vgrid);
}

__global__ void __launch_bounds__(kTileThreads, 8)
group_dedup_tile_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  dedup_tile_body(it.wk, it.ids, it.n_ids, it.off, it.n_bags, it.tv.st, it.dedup_seed, vblock);
}

template <int MODE>
__global__ void __launch_bounds__(256, 6)
group_table_update_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  table_update_body<MODE>(it.tv, it.wk, it.now, vblock, vgrid);
}

__global__ void __launch_bounds__(256)
group_sketch_add_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  if (it.tv.sketch_depth) sketch_add_body(it.tv, it.wk, vblock, vgrid);
}

__global__ void __launch_bounds__(256)
group_table_insert_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  table_insert_body(it.tv, it.wk, it.now, vblock, vgrid);
}

// the filing pass inside a push ...
__global__ void __launch_bounds__(256)
group_file_segments_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  file_segments_body(it.wk, it.n_ids, it.n_bags, nullptr, 0u, vblock, vgrid);
}

// ... and inside the lookup of announced batches, where it also leaves every occurrence's row
__global__ void __launch_bounds__(256)
group_file_rows_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  if (it.prepared) file_segments_body(it.wk, it.n_ids, it.n_bags, it.occ_row, (uint32_t)it.tv.capacity, vblock, vgrid);
}

__global__ void __launch_bounds__(256)
group_clear_primary_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  clear_primary_body(it.wk, vblock, vgrid);
}

__global__ void __launch_bounds__(128)
group_expand_parts_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  expand_parts_body(it.tv, it.wk, vblock, vgrid);
}

__global__ void __launch_bounds__(kWindows)
group_order_parts_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  order_parts_body(it.tv, it.wk, vblock, vgrid);
}

__global__ void __launch_bounds__(256)
group_fold_partials_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  fold_partials_body(it.tv, it.wk, vblock, vgrid);
}

__global__ void __launch_bounds__(kCombineThreads)
group_combine_adagrad_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  combine_adagrad_body(it.tv, it.wk, vblock, vgrid);
}

// one block per table
__global__ void __launch_bounds__(256)
group_finish_apply_kernel(const GroupItem* __restrict__ items, uint32_t n_tables, int commit) {
  after_previous_kernel();
  if (blockIdx.x < n_tables && items[blockIdx.x].active) finish_apply_body(items[blockIdx.x].tv.st, items[blockIdx.x].wk.win_count, commit);
}

// The kernels whose bodies are compiled per lane-group width.  A block's table decides the
// width, so the tables of a launch can have different dims.  WIDE = 0 covers dims up to 128
// (one 16-byte column vector per lane, classes 0..3) in one launch; the wider rows (classes
// 4..6), whose bodies need twice to four times the registers, get a launch of their own.
template <int WIDE, typename F>
__device__ inline void by_lane_class(uint32_t lane_class, F&& f) {
  if (WIDE == 0) {
    switch (lane_class) {
      case 0: f(std::integral_constant<int, 4>{}, std::integral_constant<int, 1>{}); break;
      case 1: f(std::integral_constant<int, 8>{}, std::integral_constant<int, 1>{}); break;
      case 2: f(std::integral_constant<int, 16>{}, std::integral_constant<int, 1>{}); break;
      case 3: f(std::integral_constant<int, 32>{}, std::integral_constant<int, 1>{}); break;
      default: break;
    }
  } else {
    switch (lane_class) {
      case 4: f(std::integral_constant<int, 32>{}, std::integral_constant<int, 2>{}); break;
      case 5: f(std::integral_constant<int, 32>{}, std::integral_constant<int, 4>{}); break;
      case 6: f(std::integral_constant<int, 32>{}, std::integral_constant<int, 8>{}); break;
      default: break;
    }
  }
}

// (lookup of the tables whose batches were not announced: their occurrences probe the key store)
__global__ void __launch_bounds__(256)
group_probe_rows_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  if (!it.prepared) probe_rows_body(it.tv, it.ids, it.n_ids, it.occ_row, vblock, vgrid);
}

template <int WIDE>
__global__ void __launch_bounds__(256)
group_gather_pool_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  by_lane_class<WIDE>(it.lane_class, [&](auto g, auto nv) {
    gather_pool_body<decltype(g)::value, decltype(nv)::value>(it.tv, it.occ_row, it.n_ids, it.off, it.n_bags, it.out, vblock, vgrid);
  });
}

template <int WIDE>
__global__ void __launch_bounds__(256)
group_reduce_adagrad_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  by_lane_class<WIDE>(it.lane_class, [&](auto g, auto nv) {
    reduce_adagrad_body<decltype(g)::value, decltype(nv)::value>(it.tv, it.wk, it.grad, it.n_bags, kReduceParts | kReduceShort, vblock, vgrid);
  });
}

template <int WIDE>
__global__ void __launch_bounds__(256)
group_update_singletons_kernel(const GroupItem* __restrict__ items, const uint32_t* __restrict__ start, uint32_t n_tables) {
  MONO_GROUP_PROLOGUE;
  by_lane_class<WIDE>(it.lane_class, [&](auto g, auto nv) {
    update_singletons_body<decltype(g)::value, decltype(nv)::value>(it.tv, it.wk, it.grad, it.n_bags, vblock, vgrid);
  });
}

#undef MONO_GROUP_PROLOGUE

}  // namespace mono
