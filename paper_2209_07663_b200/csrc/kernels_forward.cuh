// Forward: cuckoo look-up of every ID of a bag, gather of the rows that exist,
// sum in ID order (the HashTable look-up operation of Section 2.1 serving the
// parameter pull of Section 2.2; sum pooling per bag).
#pragma once

#include "table_layout.cuh"

namespace mono {

// Find `id` in its two candidate buckets (and the stash when it is in use) with
// the four lanes `sub` = 0..3 of a quad reading one cell each.  Returns, on the
// lane that saw the key, hit = true and the cell's metadata.  `quad_mask` names
// the four lanes; all four must call together.
__device__ inline bool quad_find(const TableView& tv, unsigned long long id, bool active, int sub,
                                 unsigned quad_mask, unsigned stash_hw, unsigned long long* meta_out) {
  bool hit = false;
  unsigned long long meta = 0;
  if (active) {
    const Cell c = load_cell_ro(tv.cells + tv.bucket0(id) * kCellsPerBucket + sub);
    hit = c.key == id;
    meta = c.meta;
  }
  bool found = (__ballot_sync(quad_mask, hit) & quad_mask) != 0;
  if (!found) {
    if (active) {
      const Cell c = load_cell_ro(tv.cells + tv.bucket1(id) * kCellsPerBucket + sub);
      hit = c.key == id;
      meta = c.meta;
    }
    found = (__ballot_sync(quad_mask, hit) & quad_mask) != 0;
    if (!found && stash_hw != 0 && active) {
      for (unsigned i = sub; i < stash_hw; i += kCellsPerBucket) {
        const Cell c = load_cell_ro(tv.stash + i);
        if (c.key == id) { hit = true; meta = c.meta; break; }
      }
    }
  }
  *meta_out = meta;
  return hit;
}

// One group of G lanes per bag (G = 4, 8, 16 or 32 chosen from dim so that a
// lane owns NV 16-byte column vectors).  Per round the group resolves G/4 IDs
// at once -- each quad probes one ID -- then every lane adds its columns of
// the rows found, in ID order, so the fp32 sum has one fixed order.
template <int G, int NV>
__global__ void __launch_bounds__(256)
lookup_pool_kernel(TableView tv, const unsigned long long* __restrict__ ids, long long n_ids,
                   const long long* __restrict__ offsets, long long n_bags, float* __restrict__ out) {
  constexpr int kIdsPerRound = G / 4;
  const int lane = threadIdx.x & 31;
  const int gl = lane % G;
  const int sub = gl & 3;
  const int quad = gl >> 2;
  const unsigned group_mask = (G == 32) ? 0xFFFFFFFFu : (((1u << G) - 1u) << (lane - gl));
  const unsigned quad_mask = 0xFu << (lane - sub);
  const unsigned stash_hw = tv.st->stash_hw;
  const uint32_t dim = tv.dim;
  const long long groups_per_block = blockDim.x / G;
  const long long stride = (long long)gridDim.x * groups_per_block;

  for (long long bag = (long long)blockIdx.x * groups_per_block + threadIdx.x / G; bag < n_bags; bag += stride) {
    long long lo = offsets[bag], hi = offsets[bag + 1];
    if (lo < 0 || hi < lo || hi > n_ids) {
      if (gl == 0) atomicOr(&tv.st->error_bits, 4u /* MONO_DEV_BAD_OFFSETS */);
      lo = hi = 0;
    }
    float4 sum[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) sum[v] = make_float4(0.f, 0.f, 0.f, 0.f);

    for (long long base = lo; base < hi; base += kIdsPerRound) {
      const long long j = base + quad;
      unsigned long long id = kEmptyKey;
      if (j < hi) id = ids[j];
      const bool active = id != kEmptyKey;
      unsigned long long meta;
      const bool hit = quad_find(tv, id, active, sub, quad_mask, stash_hw, &meta);
      const uint32_t my_row = (hit && meta_resident(meta)) ? meta_row(meta) : kNoRow;
      // lanes that hold a row, as a bit per lane of the group
      const unsigned holders = (__ballot_sync(group_mask, my_row != kNoRow) & group_mask) >> (lane - gl);
      uint32_t row_of[kIdsPerRound];
#pragma unroll
      for (int i = 0; i < kIdsPerRound; ++i) {
        const unsigned nib = (holders >> (4 * i)) & 0xFu;
        const int src = 4 * i + (nib ? (__ffs(nib) - 1) : 0);
        const uint32_t r = __shfl_sync(group_mask, my_row, src, G);
        row_of[i] = nib ? r : kNoRow;
      }
#pragma unroll
      for (int i = 0; i < kIdsPerRound; ++i) {
        if (row_of[i] != kNoRow) {
          const float4* src = reinterpret_cast<const float4*>(tv.w_row(row_of[i]));
#pragma unroll
          for (int v = 0; v < NV; ++v) {
            const uint32_t c4 = gl + v * G;
            if (c4 * 4u < dim) {
              const float4 x = __ldg(src + c4);
              sum[v].x += x.x; sum[v].y += x.y; sum[v].z += x.z; sum[v].w += x.w;
            }
          }
        }
      }
    }
    float4* dst = reinterpret_cast<float4*>(out + bag * (long long)dim);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const uint32_t c4 = gl + v * G;
      if (c4 * 4u < dim) dst[c4] = sum[v];
    }
  }
}

}  // namespace mono
