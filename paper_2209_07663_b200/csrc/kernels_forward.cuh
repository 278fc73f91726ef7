// Forward: cuckoo look-up of every ID of a batch, gather of the rows that
// exist, sum per bag in ID order (the HashTable look-up operation of Section 2.1 serving the
// parameter pull of Section 2.2; sum pooling per bag).
#pragma once

#include "kernels_dedup.cuh"
#include "table_layout.cuh"

namespace mono {

// Read-only look-up by one thread.  An insertion tries the cell named by the
// top bits of the hash first, so that cell is read first and alone; the other
// three cells of the bucket, the second bucket and the stash follow only on a
// miss.  Returns true and the metadata when the ID is tracked.
__device__ inline bool thread_lookup(const TableView& tv, unsigned long long id, unsigned stash_hw,
                                     unsigned long long* meta) {
  const unsigned long long h0 = tv.hash0(id);
  const Cell* b = tv.cells + (h0 & tv.bucket_mask) * kCellsPerBucket;
  const uint32_t first = (uint32_t)(h0 >> 62);
  const Cell c0 = load_cell_ro(b + first);
  if (c0.key == id) { *meta = c0.meta; return true; }
  // the other three cells of the bucket, requested together (named values, not an array: an
  // indexed array here ends up in local memory)
  const Cell c1 = load_cell_ro(b + ((first + 1u) & 3u));
  const Cell c2 = load_cell_ro(b + ((first + 2u) & 3u));
  const Cell c3 = load_cell_ro(b + ((first + 3u) & 3u));
  if (c1.key == id) { *meta = c1.meta; return true; }
  if (c2.key == id) { *meta = c2.meta; return true; }
  if (c3.key == id) { *meta = c3.meta; return true; }
  b = tv.cells + tv.bucket1(id) * kCellsPerBucket;
  const Cell d0 = load_cell_ro(b), d1 = load_cell_ro(b + 1), d2 = load_cell_ro(b + 2), d3 = load_cell_ro(b + 3);
  if (d0.key == id) { *meta = d0.meta; return true; }
  if (d1.key == id) { *meta = d1.meta; return true; }
  if (d2.key == id) { *meta = d2.meta; return true; }
  if (d3.key == id) { *meta = d3.meta; return true; }
  for (unsigned i = 0; i < stash_hw; ++i) {
    const Cell s = load_cell_ro(tv.stash + i);
    if (s.key == id) { *meta = s.meta; return true; }
  }
  return false;
}

// The same look-up for a caller that goes on to modify the entry: it also returns where
// the entry is (index into cells[], or n_cells + i for stash cell i; kNoCell if nowhere).
// Its kernel stores metadata into the cells it reads, so the loads are ordinary (coherent)
// 16-byte loads, not the read-only path.
constexpr unsigned long long kNoCell = 0xFFFFFFFFFFFFFFFFull;

__device__ inline unsigned long long thread_locate(const TableView& tv, unsigned long long id, unsigned stash_hw,
                                                   unsigned long long* meta) {
  const unsigned long long h0 = tv.hash0(id);
  const unsigned long long base0 = (h0 & tv.bucket_mask) * kCellsPerBucket;
  const uint32_t first = (uint32_t)(h0 >> 62);
  const Cell c0 = load_cell_whole(tv.cells + base0 + first);
  if (c0.key == id) { *meta = c0.meta; return base0 + first; }
#pragma unroll
  for (uint32_t k = 1; k < kCellsPerBucket; ++k) {
    const Cell c = load_cell_whole(tv.cells + base0 + ((first + k) & 3u));
    if (c.key == id) { *meta = c.meta; return base0 + ((first + k) & 3u); }
  }
  const unsigned long long base1 = tv.bucket1(id) * kCellsPerBucket;
#pragma unroll
  for (uint32_t k = 0; k < kCellsPerBucket; ++k) {
    const Cell c = load_cell_whole(tv.cells + base1 + k);
    if (c.key == id) { *meta = c.meta; return base1 + k; }
  }
  for (unsigned i = 0; i < stash_hw; ++i) {
    const Cell s = load_cell_whole(tv.stash + i);
    if (s.key == id) { *meta = s.meta; return (tv.bucket_mask + 1) * kCellsPerBucket + i; }
  }
  return kNoCell;
}

// Forward, step 1, for a batch that was not announced: one thread per ID occurrence resolves
// the ID to its row index; an ID without a row gets the index of the table's all-zero row (one
// past the capacity), so that step 2 can add rows without asking.  Every occurrence is
// independent, so the random bucket reads of a whole batch are in flight together.  (Measured
// against quad-cooperative variants: the shuffles those need cost more issue slots than the
// extra L1 wavefronts of four 16-byte loads per thread.  Measured against doing the look-ups
// inside step 2, one per lane of the bag's group: 0.50 ms against 0.15 + 0.27 ms for the two
// kernels on the largest configuration.)  For a batch that was announced, file_segments_kernel
// writes the same array from the look-up that was done once per distinct ID.
__device__ inline void probe_rows_body(const TableView& tv, const unsigned long long* __restrict__ ids, long long n_ids,
                                       uint32_t* __restrict__ occ_row, uint32_t vblock, uint32_t vgrid) {
  const unsigned stash_hw = tv.st->stash_hw;
  const uint32_t zero_row = (uint32_t)tv.capacity;
  const long long stride = (long long)vgrid * blockDim.x;
  for (long long j = (long long)vblock * blockDim.x + threadIdx.x; j < n_ids; j += stride) {
    const unsigned long long id = ids[j];
    unsigned long long meta = 0;
    uint32_t row = zero_row;
    if (id != kEmptyKey && thread_lookup(tv, id, stash_hw, &meta) && meta_resident(meta)) row = meta_row(meta);
    occ_row[j] = row;
  }
}
__global__ void __launch_bounds__(256)
probe_rows_kernel(TableView tv, const unsigned long long* __restrict__ ids, long long n_ids,
                  uint32_t* __restrict__ occ_row) { after_previous_kernel();
  probe_rows_body(tv, ids, n_ids, occ_row, blockIdx.x, gridDim.x);
}

// sum += rows idx[0..K), in that order; all K loads are issued before the first add.
template <int K, int G, int NV>
__device__ inline void add_rows(const TableView& tv, const uint32_t* __restrict__ idx, int gl, float4 (&sum)[NV]) {
  uint32_t row[K];
#pragma unroll
  for (int k = 0; k < K; ++k) row[k] = __ldg(idx + k);
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const uint32_t c4 = gl + v * G;
    if (c4 * 4u < tv.dim) {
      float4 x[K];
#pragma unroll
      for (int k = 0; k < K; ++k) x[k] = __ldg(reinterpret_cast<const float4*>(tv.w_row(row[k])) + c4);
#pragma unroll
      for (int k = 0; k < K; ++k) { sum[v].x += x[k].x; sum[v].y += x[k].y; sum[v].z += x[k].z; sum[v].w += x[k].w; }
    }
  }
}

// Forward, step 2: one group of G lanes per bag (G = 4, 8, 16 or 32 chosen from
// dim so that a lane owns NV 16-byte column vectors) adds up the rows of the
// bag's IDs, in ID order, so the fp32 sum has one fixed order.  The row
// indices are known, so the loads of up to eight rows are issued together (the
// compiler keeps the kernel at 32 registers and full occupancy, which matters
// more here than the depth: with room for all eight in flight, 45 registers, it
// ran 3 % of a step slower); what is left of the bag after the batches of eight
// is added in one batch of its exact size.  The kernel is bound by instruction issue, not by memory, so there are
// no per-row validity tests (step 1 points an ID without a row at the zero row)
// and no loads or adds for padding (measured: batches padded with the zero row
// 0.31 ms on the largest configuration, exact tails 0.26 ms).  Every lane of the
// group reads the row indices itself: the loads of a group hit one cache line.
// Three other shapes of this loop were measured slower on the largest configuration
// (0.26 - 0.28 ms as it stands): the indices read once per group and passed round by
// shuffle, 0.33 ms; a software pipeline over three bags (offsets, indices and rows of
// successive bags in flight together), 0.41 ms; and a walk over each group's run of
// occurrences in uniform batches of four with only the end of a bag depending on the
// offsets, 0.33 ms -- the last two need half as many registers again; and lane groups that
// take consecutive bags instead of bags a grid apart, so that offsets and indices of a
// group's next bag are cache hits (1.3 % of a step slower).
template <int G, int NV>
__device__ inline void gather_pool_body(const TableView& tv, const uint32_t* __restrict__ occ_row, long long n_ids,
                                        const long long* __restrict__ offsets, long long n_bags, float* __restrict__ out,
                                        uint32_t vblock, uint32_t vgrid) {
  const int gl = threadIdx.x % G;
  const uint32_t dim = tv.dim;
  const long long groups_per_block = blockDim.x / G;
  const long long stride = (long long)vgrid * groups_per_block;
  for (long long bag = (long long)vblock * groups_per_block + threadIdx.x / G; bag < n_bags; bag += stride) {
    long long lo = offsets[bag], hi = offsets[bag + 1];
    if (lo < 0 || hi < lo || hi > n_ids) {                 // not a well-formed bag: flagged and treated as empty
      if (gl == 0) atomicOr(&tv.st->error_bits, 4u /* MONO_DEV_BAD_OFFSETS */);
      lo = hi = 0;
    }
    float4 sum[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) sum[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    const uint32_t* idx = occ_row + lo;
    const uint32_t n = (uint32_t)(hi - lo);              // a call has fewer than 2^31 IDs
    uint32_t i = 0;
    for (; i + 8 <= n; i += 8) add_rows<8, G, NV>(tv, idx + i, gl, sum);
    switch (n - i) {
      case 7: add_rows<7, G, NV>(tv, idx + i, gl, sum); break;
      case 6: add_rows<6, G, NV>(tv, idx + i, gl, sum); break;
      case 5: add_rows<5, G, NV>(tv, idx + i, gl, sum); break;
      case 4: add_rows<4, G, NV>(tv, idx + i, gl, sum); break;
      case 3: add_rows<3, G, NV>(tv, idx + i, gl, sum); break;
      case 2: add_rows<2, G, NV>(tv, idx + i, gl, sum); break;
      case 1: add_rows<1, G, NV>(tv, idx + i, gl, sum); break;
      default: break;
    }
    float4* dst = reinterpret_cast<float4*>(out + bag * (long long)dim);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const uint32_t c4 = gl + v * G;
      if (c4 * 4u < dim) dst[c4] = sum[v];
    }
  }
}

template <int G, int NV>
__global__ void __launch_bounds__(256)
gather_pool_kernel(TableView tv, const uint32_t* __restrict__ occ_row, long long n_ids,
                   const long long* __restrict__ offsets, long long n_bags, float* __restrict__ out) { after_previous_kernel();
  gather_pool_body<G, NV>(tv, occ_row, n_ids, offsets, n_bags, out, blockIdx.x, gridDim.x);
}

}  // namespace mono
