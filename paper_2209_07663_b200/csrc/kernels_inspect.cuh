// Inspection kernels (not on the hot path): state of given IDs, dump of the
// whole table, and the structural audit of the cuckoo invariants of Section
// 2.1 (every key in one of its two buckets, stored exactly once).
#pragma once

#include "table_layout.cuh"

namespace mono {

// Thread-level lookup: both buckets, then the stash.  Returns the cell or null.
__device__ inline const Cell* find_cell(const TableView& tv, unsigned long long id, unsigned stash_hw) {
  if (id == kEmptyKey) return nullptr;
  const unsigned long long bk[2] = {tv.bucket0(id), tv.bucket1(id)};
  for (int b = 0; b < 2; ++b)
    for (uint32_t c = 0; c < kCellsPerBucket; ++c) {
      const Cell* p = tv.cells + bk[b] * kCellsPerBucket + c;
      if (p->key == id) return p;
    }
  for (unsigned s = 0; s < stash_hw; ++s)
    if (tv.stash[s].key == id) return tv.stash + s;
  return nullptr;
}

__global__ void __launch_bounds__(256)
probe_kernel(TableView tv, const unsigned long long* __restrict__ ids, long long n, uint8_t* resident,
             uint32_t* count, long long* last_seen) {
  const unsigned stash_hw = tv.st->stash_hw;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const Cell* p = find_cell(tv, ids[i], stash_hw);
    const unsigned long long meta = p ? p->meta : 0ull;
    const bool res = p && meta_resident(meta);
    if (resident) resident[i] = res ? 1 : 0;
    if (count) {
      uint32_t c = !p ? 0u : (res ? tv.threshold : meta_low(meta));
      if (!p && tv.sketch_depth != 0 && ids[i] != kEmptyKey) {        // probabilistic filter: the estimate, capped
        const unsigned int est = tv.sketch_estimate(ids[i]);
        c = est < tv.threshold ? est : tv.threshold;
      }
      count[i] = c;
    }
    if (last_seen) last_seen[i] = p ? (long long)meta_time(meta) : -1LL;
  }
}

__global__ void __launch_bounds__(256)
read_rows_kernel(TableView tv, const unsigned long long* __restrict__ ids, long long n, float* w, float* acc) {
  const unsigned stash_hw = tv.st->stash_hw;
  const int gl = threadIdx.x & 7;
  const long long groups = ((long long)gridDim.x * blockDim.x) >> 3;
  const uint32_t dim4 = tv.dim / 4;
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3; i < n; i += groups) {
    const Cell* p = find_cell(tv, ids[i], stash_hw);
    const bool res = p && meta_resident(p->meta);
    const uint32_t row = res ? meta_row(p->meta) : 0u;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    for (uint32_t c4 = gl; c4 < dim4; c4 += 8) {
      if (w) reinterpret_cast<float4*>(w + i * (long long)tv.dim)[c4] =
          res ? reinterpret_cast<const float4*>(tv.w_row(row))[c4] : zero;
      if (acc) reinterpret_cast<float4*>(acc + i * (long long)tv.dim)[c4] =
          res ? reinterpret_cast<const float4*>(tv.acc_row(row))[c4] : zero;
    }
  }
}

__global__ void __launch_bounds__(256)
export_kernel(TableView tv, unsigned long long n_cells, unsigned long long* ids, uint32_t* count,
              long long* last_seen, uint8_t* resident, float* w, float* acc, long long max_n) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  const unsigned long long total = n_cells + kStashCells;
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const Cell* p = i < n_cells ? tv.cells + i : tv.stash + (i - n_cells);
    const Cell c = *p;
    if (c.key == kEmptyKey) continue;
    const long long k = (long long)atomicAdd(&tv.st->export_n, 1ull);
    if (k >= max_n) continue;
    const bool res = meta_resident(c.meta);
    ids[k] = c.key;
    if (count) count[k] = res ? tv.threshold : meta_low(c.meta);
    if (last_seen) last_seen[k] = (long long)meta_time(c.meta);
    if (resident) resident[k] = res ? 1 : 0;
    for (uint32_t col = 0; col < tv.dim; ++col) {
      if (w) w[k * (long long)tv.dim + col] = res ? tv.w_row(meta_row(c.meta))[col] : 0.f;
      if (acc) acc[k * (long long)tv.dim + col] = res ? tv.acc_row(meta_row(c.meta))[col] : 0.f;
    }
  }
}

// Incremental export (Section 2.2.3 of the paper: the set of touched keys, the IDs whose
// embeddings were trained since the last synchronisation).  A streaming pass over the key
// store: every row marked as trained is appended to the caller's buffers and its mark is
// cleared; when the buffers are full the remaining marks stay for the next call.
__global__ void __launch_bounds__(256)
export_touched_kernel(TableView tv, unsigned long long n_cells, unsigned long long* ids, float* w, long long max_n) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  const unsigned long long total = n_cells + kStashCells;
  const unsigned long long rounds = (total + stride - 1) / stride;
  const int lane = threadIdx.x & 31;
  for (unsigned long long r = 0; r < rounds; ++r) {
    const unsigned long long i = r * stride + (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    Cell* p = nullptr;
    Cell c = empty_cell();
    if (i < total) { p = i < n_cells ? tv.cells + i : tv.stash + (i - n_cells); c = *p; }
    const bool mine = c.key != kEmptyKey && meta_touched(c.meta);
    const unsigned mask = __ballot_sync(0xFFFFFFFFu, mine);
    if (!mask) continue;
    unsigned long long base = 0;
    const int leader = __ffs(mask) - 1;
    if (lane == leader) base = atomicAdd(&tv.st->export_n, (unsigned long long)__popc(mask));
    base = __shfl_sync(0xFFFFFFFFu, base, leader);
    if (!mine) continue;
    const long long k = (long long)(base + __popc(mask & ((1u << lane) - 1u)));
    if (k >= max_n) continue;
    ids[k] = c.key;
    p->meta = c.meta & ~(unsigned long long)kTouchedBit;
    const float4* src = reinterpret_cast<const float4*>(tv.w_row(meta_row(c.meta)));
    float4* dst = reinterpret_cast<float4*>(w + k * (long long)tv.dim);
    for (uint32_t c4 = 0; c4 < tv.dim / 4; ++c4) dst[c4] = src[c4];
  }
}

struct AuditCounters {
  unsigned long long occupied, misplaced, duplicate_keys, resident_cells, bad_rows, shared_rows, free_rows,
      unaccounted_rows, behind_records;
};

// row_marks: one bit per row, zeroed by the caller.
__global__ void __launch_bounds__(256)
audit_cells_kernel(TableView tv, unsigned long long n_cells, unsigned int* row_marks, AuditCounters* out) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  const unsigned long long total = n_cells + kStashCells;
  const unsigned stash_hw = tv.st->stash_hw;
  unsigned int n_occ = 0, n_res = 0;      // common counters: summed per warp at the end
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const bool in_stash = i >= n_cells;
    const Cell c = in_stash ? tv.stash[i - n_cells] : tv.cells[i];
    if (c.key == kEmptyKey) continue;
    ++n_occ;
    if (in_stash) {
      if (i - n_cells >= stash_hw) atomicAdd(&out->misplaced, 1ull);    // invisible to probes
    } else {
      const unsigned long long b = i / kCellsPerBucket;
      if (b != tv.bucket0(c.key) && b != tv.bucket1(c.key)) atomicAdd(&out->misplaced, 1ull);
      if (meta_time(c.meta) < tv.oldest[b]) atomicAdd(&out->behind_records, 1ull);   // the sweep could pass this entry by
    }
    // the key must occur exactly once among its two buckets and the stash
    unsigned copies = 0;
    const unsigned long long b0 = tv.bucket0(c.key), b1 = tv.bucket1(c.key);
    for (uint32_t k = 0; k < kCellsPerBucket; ++k) copies += tv.cells[b0 * kCellsPerBucket + k].key == c.key;
    if (b1 != b0)
      for (uint32_t k = 0; k < kCellsPerBucket; ++k) copies += tv.cells[b1 * kCellsPerBucket + k].key == c.key;
    for (unsigned s = 0; s < kStashCells; ++s) copies += tv.stash[s].key == c.key;
    if (copies != 1) atomicAdd(&out->duplicate_keys, 1ull);
    if (meta_resident(c.meta)) {
      ++n_res;
      const uint32_t row = meta_row(c.meta);
      if (row >= tv.capacity) { atomicAdd(&out->bad_rows, 1ull); continue; }
      const unsigned int bit = 1u << (row & 31);
      if (atomicOr(row_marks + (row >> 5), bit) & bit) atomicAdd(&out->shared_rows, 1ull);
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    n_occ += __shfl_down_sync(0xFFFFFFFFu, n_occ, o);
    n_res += __shfl_down_sync(0xFFFFFFFFu, n_res, o);
  }
  if ((threadIdx.x & 31) == 0) {
    if (n_occ) atomicAdd(&out->occupied, (unsigned long long)n_occ);
    if (n_res) atomicAdd(&out->resident_cells, (unsigned long long)n_res);
  }
}

__global__ void __launch_bounds__(256)
audit_free_kernel(TableView tv, unsigned int* row_marks, AuditCounters* out) {
  const long long n_free = tv.st->free_top;
  const long long stride = (long long)gridDim.x * blockDim.x;
  if (blockIdx.x == 0 && threadIdx.x == 0) out->free_rows = n_free > 0 ? (unsigned long long)n_free : 0ull;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_free; i += stride) {
    const uint32_t row = tv.free_rows[i];
    if (row >= tv.capacity) { atomicAdd(&out->bad_rows, 1ull); continue; }
    const unsigned int bit = 1u << (row & 31);
    if (atomicOr(row_marks + (row >> 5), bit) & bit) atomicAdd(&out->shared_rows, 1ull);
  }
}

__global__ void __launch_bounds__(256)
audit_rows_kernel(TableView tv, const unsigned int* row_marks, AuditCounters* out) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  for (unsigned long long r = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; r < tv.capacity; r += stride)
    if (!(row_marks[r >> 5] & (1u << (r & 31)))) atomicAdd(&out->unaccounted_rows, 1ull);
}

}  // namespace mono
