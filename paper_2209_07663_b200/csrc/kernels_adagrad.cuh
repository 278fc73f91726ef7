// Backward, last phase: per distinct ID that owns a row, sum the pooled
// gradients of its occurrences' bags (fp64 accumulation, one rounding to fp32)
// and apply one Adagrad step to the row, in place.  This is the parameter push
// of Section 2.2 for the sparse rows; the optimizer itself is not named in the
// paper.
//
// Three cases, by how often the ID occurs in the batch:
// Every repeated ID has a segment of bag_of_sorted[] that lists the bags of its
// occurrences (filed by file_segments_kernel: inside the lookup when the batch was
// announced, else inside the push).
//  - once (most distinct IDs of a long-tailed batch): its gradient is the
//    pooled gradient of its one bag, so update_singletons_kernel updates the
//    row straight from that bag's gradient row;
//  - 2 .. kSegChunk times: one lane group of reduce_adagrad_kernel gathers
//    the gradient rows of the segment's bags;
//  - more (the head of the Zipf distribution: one ID can own several percent of
//    a batch): the segment is cut into parts of kSegChunk that separate groups
//    reduce into fp64 partial sums, combined by one block per ID in a fixed
//    order.
#pragma once

#include "kernels_dedup.cuh"

namespace mono {

struct D4 { double x, y, z, w; };

__device__ inline void add4(D4& a, const float4 v) { a.x += (double)v.x; a.y += (double)v.y; a.z += (double)v.z; a.w += (double)v.w; }

// acc += G*G;  w -= lr*G/(sqrt(acc)+eps), each operation rounded to fp32 on its
// own (no fused multiply-add), so the result does not depend on contraction.
__device__ inline void adagrad4(float4& w, float4& a, const D4& g, float lr, float eps) {
  const float gx = (float)g.x, gy = (float)g.y, gz = (float)g.z, gw = (float)g.w;
  a.x = __fadd_rn(a.x, __fmul_rn(gx, gx));
  a.y = __fadd_rn(a.y, __fmul_rn(gy, gy));
  a.z = __fadd_rn(a.z, __fmul_rn(gz, gz));
  a.w = __fadd_rn(a.w, __fmul_rn(gw, gw));
  w.x = __fsub_rn(w.x, __fdiv_rn(__fmul_rn(lr, gx), __fadd_rn(__fsqrt_rn(a.x), eps)));
  w.y = __fsub_rn(w.y, __fdiv_rn(__fmul_rn(lr, gy), __fadd_rn(__fsqrt_rn(a.y), eps)));
  w.z = __fsub_rn(w.z, __fdiv_rn(__fmul_rn(lr, gz), __fadd_rn(__fsqrt_rn(a.z), eps)));
  w.w = __fsub_rn(w.w, __fdiv_rn(__fmul_rn(lr, gw), __fadd_rn(__fsqrt_rn(a.w), eps)));
}

// Load (or, for a row admitted in this call, create) the row, update, store.
__device__ inline void update_row(const TableView& tv, uint32_t row_word, unsigned long long id,
                                  uint32_t c4, const D4& g) {
  const uint32_t row = row_word & ~kFreshBit;
  float4* pw = reinterpret_cast<float4*>(tv.w_row(row)) + c4;
  float4* pa = reinterpret_cast<float4*>(tv.acc_row(row)) + c4;
  float4 w, a;
  if (row_word & kFreshBit) {
    w = init_vec(tv, id, c4);
    a = make_float4(tv.init_acc, tv.init_acc, tv.init_acc, tv.init_acc);
  } else {
    w = *pw;
    a = *pa;
  }
  adagrad4(w, a, g, tv.lr, tv.eps);
  *pw = w;
  *pa = a;
}

// The per-call set must be empty again when the push ends.  Its primary tier is wiped as a whole
// (clear_primary_kernel: a streaming write costs less than one scattered store per ID); an ID
// that overflowed into the secondary tier, which is far larger and almost empty, has its slot
// emptied by the kernel that updates its row.
__device__ inline void clear_overflow_slot(const Work& wk, uint32_t slot) {
  if (slot > wk.primary_mask) {
    BatchSlot e; e.key = kEmptyKey; e.a = 0; e.b = 0;
    wk.bset[slot] = e;
  }
}

__device__ inline void clear_primary_body(const Work& wk, uint32_t vblock, uint32_t vgrid) {
  const uint32_t n = wk.primary_mask + 1u;
  ulonglong2 e; e.x = kEmptyKey; e.y = 0ull;
  for (uint32_t i = vblock * blockDim.x + threadIdx.x; i < n; i += vgrid * blockDim.x)
    *reinterpret_cast<ulonglong2*>(wk.bset + i) = e;
}
__global__ void __launch_bounds__(256)
clear_primary_kernel(Work wk) { after_previous_kernel(); clear_primary_body(wk, blockIdx.x, gridDim.x); }

// Sum of grad rows of bags bag_of_sorted[begin .. end) for the NV column
// vectors this lane owns.  Eight independent row loads in flight per step.
template <int G, int NV>
__device__ inline void reduce_segment(const Work& wk, const float* __restrict__ grad, long long n_bags,
                                      uint32_t dim, int gl, uint32_t begin, uint32_t end, D4 (&s)[NV]) {
  constexpr int kDepth = NV == 1 ? 8 : 4;
  uint32_t i = begin;
  for (; i + kDepth <= end; i += kDepth) {
    uint32_t b[kDepth];
#pragma unroll
    for (int k = 0; k < kDepth; ++k) b[k] = wk.bag_of_sorted[i + k];
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const uint32_t c4 = gl + v * G;
      if (c4 * 4u < dim) {
        float4 x[kDepth];
#pragma unroll
        for (int k = 0; k < kDepth; ++k)
          x[k] = b[k] < n_bags ? __ldg(reinterpret_cast<const float4*>(grad + (size_t)b[k] * dim) + c4)
                               : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < kDepth; ++k) add4(s[v], x[k]);
      }
    }
  }
  if (i < end) {
    // the ragged tail, again with all its loads issued before the adds
    uint32_t b[kDepth];
#pragma unroll
    for (int k = 0; k < kDepth; ++k) b[k] = i + k < end ? wk.bag_of_sorted[i + k] : 0xFFFFFFFFu;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const uint32_t c4 = gl + v * G;
      if (c4 * 4u < dim) {
        float4 x[kDepth];
#pragma unroll
        for (int k = 0; k < kDepth; ++k)
          x[k] = b[k] < n_bags ? __ldg(reinterpret_cast<const float4*>(grad + (size_t)b[k] * dim) + c4)
                               : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < kDepth; ++k) add4(s[v], x[k]);
      }
    }
  }
}

// One pass over the occurrences once the distinct IDs have been looked up: every
// occurrence of a repeated ID reads its ID's slot of the per-call set and is filed under
// its ID -- its bag goes into the ID's segment of bag_of_sorted[], at the occurrence's rank -- and, when
// occ_row is given (the lookup of a batch that was announced), leaves there the row its ID
// owns, or the table's all-zero row, for the pooling kernel.
__device__ inline void file_segments_body(const Work& wk, long long n_ids, long long n_bags, uint32_t* __restrict__ occ_row,
                                          uint32_t zero_row, uint32_t vblock, uint32_t vgrid) {
  const long long stride = (long long)vgrid * blockDim.x;
  for (long long j = (long long)vblock * blockDim.x + threadIdx.x; j < n_ids; j += stride) {
    const uint2 o = wk.occ[j];
    uint32_t row = zero_row;
    if (o.x != kNoSlot && MONO_INDEX_OK(wk.error_bits, o.x, wk.n_slots)) {
      const uint4 bs = __ldg(reinterpret_cast<const uint4*>(wk.bset + o.x));     // key (x, y), segment start, row
      if (bs.w != kNoRow) row = bs.w;
      if (bs.z != kNoSegment) {                                                   // (an ID that occurs once has no segment)
        const uint32_t bag = wk.occ_bag[j];
        if (bag < n_bags && MONO_INDEX_OK(wk.error_bits, (unsigned long long)bs.z + o.y, wk.max_ids)) wk.bag_of_sorted[bs.z + o.y] = bag;
      }
    }
    if (occ_row) occ_row[j] = row;
  }
}
__global__ void __launch_bounds__(256)
file_segments_kernel(Work wk, long long n_ids, long long n_bags, uint32_t* __restrict__ occ_row, uint32_t zero_row) { after_previous_kernel();
  file_segments_body(wk, n_ids, n_bags, occ_row, zero_row, blockIdx.x, gridDim.x);
}

// The IDs that occur once in the batch (most distinct IDs of a long-tailed batch): the
// gradient of such an ID is the pooled gradient of its one bag, so its row is updated
// straight from there.  One warp per 32 consecutive distinct IDs, which are numbered in
// the order the batch first shows them, so the gradient rows are read roughly in order;
// the lanes whose ID occurs once and has a row are served in turn by lane groups of G,
// which read the bag's gradient row, the table row and its accumulator, and write both
// back updated.
template <int G, int NV>
__device__ inline void update_singletons_body(const TableView& tv, const Work& wk, const float* __restrict__ grad,
                                              long long n_bags, uint32_t vblock, uint32_t vgrid) {
  constexpr int kGroups = 32 / G;
  const int lane = threadIdx.x & 31;
  const int gl = lane % G, grp = lane / G;
  const uint32_t n = tv.st->n_unique;
  const uint32_t n_warps = (vgrid * blockDim.x) >> 5;
  const uint32_t n_rounds = (n + 31) / 32;
  unsigned int n_single = 0;
  for (uint32_t r = (vblock * blockDim.x + threadIdx.x) >> 5; r < n_rounds; r += n_warps) {
    const uint32_t u = r * 32 + lane;
    uint32_t row_word = kNoRow, bag = 0;
    unsigned long long id = 0;
    bool single = false;
    if (u < n && wk.ulen[u] == 1u) {
      const uint32_t slot = wk.uslot[u];
      row_word = wk.urow[u];
      if (row_word != kNoRow && MONO_INDEX_OK(wk.error_bits, wk.uocc[u], wk.max_ids)) {
        bag = wk.occ_bag[wk.uocc[u]];
        single = bag < n_bags;
        if (row_word & kFreshBit) id = wk.uid[u];
      }
      clear_overflow_slot(wk, slot);                     // (after the loads: a store in between would hold them back)
    }
    unsigned todo = __ballot_sync(0xFFFFFFFFu, single);
    n_single += __popc(todo);
    while (todo) {
      // the next kGroups flagged lanes, one per lane group
      int src = -1;
      unsigned rest = todo;
#pragma unroll
      for (int g = 0; g < kGroups; ++g) {
        const int l = rest ? __ffs(rest) - 1 : -1;
        if (l >= 0) rest &= rest - 1;
        if (g == grp) src = l;
      }
      todo = rest;
      const int from = src < 0 ? 0 : src;
      const uint32_t rw = __shfl_sync(0xFFFFFFFFu, row_word, from);
      const uint32_t bg = __shfl_sync(0xFFFFFFFFu, bag, from);
      const unsigned long long key = __shfl_sync(0xFFFFFFFFu, id, from);
      if (src >= 0) {
        const float4* g4 = reinterpret_cast<const float4*>(grad + (size_t)bg * tv.dim);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
          const uint32_t c4 = gl + v * G;
          if (c4 * 4u < tv.dim) {
            const float4 x = __ldg(g4 + c4);
            const D4 g = D4{(double)x.x, (double)x.y, (double)x.z, (double)x.w};
            update_row(tv, rw, key, c4, g);
          }
        }
      }
    }
  }
  if (lane == 0 && n_single) atomicAdd(&tv.st->sum_single_resident, (unsigned long long)n_single);
}
template <int G, int NV>
__global__ void __launch_bounds__(256)
update_singletons_kernel(TableView tv, Work wk, const float* __restrict__ grad, long long n_bags) { after_previous_kernel();
  update_singletons_body<G, NV>(tv, wk, grad, n_bags, blockIdx.x, gridDim.x);
}

// One lane group per work item.  Items [0, n_parts) are the parts of the long
// segments (the heaviest items, so they are started first): a group reduces
// one part into fp64 partial sums in scratch, which combine_adagrad_kernel adds
// up afterwards.  Items [n_parts, n_parts + n_multi) are the repeated IDs: a
// group empties the ID's slot of the per-call set (every occurrence has been
// filed by now), and when the segment is short reduces it and updates the row.
// `which` selects the items of one launch: kReduceParts, kReduceShort (the repeated IDs need
// nothing from the kernels that order the parts, so they can run beside them), or both.
enum : int { kReduceParts = 1, kReduceShort = 2 };

template <int G, int NV>
__device__ inline void reduce_adagrad_body(const TableView& tv, const Work& wk, const float* __restrict__ grad,
                                           long long n_bags, int which, uint32_t vblock, uint32_t vgrid) {
  const uint32_t n = tv.st->n_multi;
  uint32_t n_parts = tv.st->n_parts;
  if (n_parts > wk.max_parts) n_parts = wk.max_parts;
  const uint32_t first_item = (which & kReduceParts) ? 0u : n_parts;
  const uint32_t n_items = (which & kReduceShort) ? n + n_parts : n_parts;
  const int gl = threadIdx.x % G;
  const uint32_t groups = (vgrid * blockDim.x) / G;
  for (uint32_t item = first_item + (vblock * blockDim.x + threadIdx.x) / G; item < n_items; item += groups) {
    D4 s[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) s[v] = D4{0.0, 0.0, 0.0, 0.0};
    if (item >= n_parts) {
      // (measured against one packed record per repeated ID, read a trip ahead: these separate
      // arrays were 2 % of a step faster on the largest configuration)
      const uint32_t u = wk.multi_list[item - n_parts];
      if (gl == 0) clear_overflow_slot(wk, wk.uslot[u]);
      const uint32_t m = wk.ulen[u];
      const uint32_t row_word = wk.urow[u];
      if (row_word == kNoRow || m > kSegChunk) continue;      // no row: gradient dropped; long: in parts
      const uint32_t begin = wk.useg[u];
      reduce_segment<G, NV>(wk, grad, n_bags, tv.dim, gl, begin, begin + m, s);
      const unsigned long long id = wk.uid[u];
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const uint32_t c4 = gl + v * G;
        if (c4 * 4u < tv.dim) update_row(tv, row_word, id, c4, s[v]);
      }
    } else {
      const uint32_t p = wk.part_order[item];
      if (!MONO_INDEX_OK(wk.error_bits, p, wk.max_parts)) continue;
      const uint32_t li = wk.part_u[p];
      if (!MONO_INDEX_OK(wk.error_bits, li, wk.max_long)) continue;
      const uint32_t u = wk.long_u[li];
      const uint32_t k = p - wk.long_part0[li];
      const uint32_t seg_end = wk.useg[u] + wk.ulen[u];
      const uint32_t begin = wk.useg[u] + k * kSegChunk;
      const uint32_t end = begin + kSegChunk < seg_end ? begin + kSegChunk : seg_end;
      if (!MONO_INDEX_OK(wk.error_bits, (unsigned long long)end - 1, wk.max_ids)) continue;
      reduce_segment<G, NV>(wk, grad, n_bags, tv.dim, gl, begin, end, s);
      double* dst = wk.partials + (size_t)p * tv.dim;
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const uint32_t c4 = gl + v * G;
        if (c4 * 4u < tv.dim) {
          reinterpret_cast<double2*>(dst)[c4 * 2] = make_double2(s[v].x, s[v].y);
          reinterpret_cast<double2*>(dst)[c4 * 2 + 1] = make_double2(s[v].z, s[v].w);
        }
      }
    }
  }
}

template <int G, int NV>
__global__ void __launch_bounds__(256)
reduce_adagrad_kernel(TableView tv, Work wk, const float* __restrict__ grad, long long n_bags, int which) { after_previous_kernel();
  reduce_adagrad_body<G, NV>(tv, wk, grad, n_bags, which, blockIdx.x, gridDim.x);
}

// First level of the combination for very long segments: one block adds up one
// group of kFoldWidth consecutive parts of one ID, column by column, and leaves
// the sum in the group's first part.  Fixed order within the block.
__device__ inline void fold_partials_body(const TableView& tv, const Work& wk, uint32_t vblock, uint32_t vgrid) {
  __shared__ double s_sum[8][256];
  uint32_t n_folds = tv.st->n_folds;
  if (n_folds > wk.max_folds) n_folds = wk.max_folds;
  const uint32_t dim = tv.dim;
  for (uint32_t fi = vblock; fi < n_folds; fi += vgrid) {
    const uint32_t li = wk.fold_li[fi], f = wk.fold_idx[fi];
    const uint32_t u = wk.long_u[li];
    if (wk.urow[u] == kNoRow) continue;               // block-uniform
    const uint32_t parts = (wk.ulen[u] + kSegChunk - 1) / kSegChunk;
    const uint32_t p_begin = f * kFoldWidth;
    const uint32_t p_end = p_begin + kFoldWidth < parts ? p_begin + kFoldWidth : parts;
    double* base = wk.partials + ((size_t)wk.long_part0[li] + p_begin) * dim;
    for (uint32_t cbase = 0; cbase < dim; cbase += 256) {
      const uint32_t width = dim - cbase < 256 ? dim - cbase : 256;
      uint32_t slices = 256 / width;
      if (slices > 8) slices = 8;
      const uint32_t col = threadIdx.x % width, slice = threadIdx.x / width;
      const uint32_t n = p_end - p_begin;
      if (slice < slices) {
        const uint32_t per = (n + slices - 1) / slices;
        const uint32_t lo = slice * per, hi = lo + per < n ? lo + per : n;
        double a0 = 0.0, a1 = 0.0;
        uint32_t p = lo;
        for (; p + 2 <= hi; p += 2) { a0 += base[(size_t)p * dim + cbase + col]; a1 += base[(size_t)(p + 1) * dim + cbase + col]; }
        if (p < hi) a0 += base[(size_t)p * dim + cbase + col];
        s_sum[slice][col] = a0 + a1;
      }
      __syncthreads();                                // every read of this group's parts is done
      if (threadIdx.x < width) {
        double g = 0.0;
        for (uint32_t s = 0; s < slices; ++s) g += s_sum[s][threadIdx.x];
        base[cbase + threadIdx.x] = g;
      }
      __syncthreads();
    }
  }
}

__global__ void __launch_bounds__(256)
fold_partials_kernel(TableView tv, Work wk) { after_previous_kernel(); fold_partials_body(tv, wk, blockIdx.x, gridDim.x); }

// One block per long ID: the block's threads split into slices of the parts
// (or, for a very long segment, of the group sums fold_partials_kernel left),
// one column each; the slices' sums are added in increasing order, so the
// combination order is fixed.
constexpr int kCombineThreads = 256;
__device__ inline void combine_adagrad_body(const TableView& tv, const Work& wk, uint32_t vblock, uint32_t vgrid) {
  constexpr int kMaxSlices = 8;
  __shared__ double s_sum[kMaxSlices][256];
  uint32_t n_long = tv.st->n_long;
  if (n_long > wk.max_long) n_long = wk.max_long;
  const uint32_t dim = tv.dim;
  for (uint32_t li = vblock; li < n_long; li += vgrid) {
    const uint32_t u = wk.long_u[li];
    const uint32_t row_word = wk.urow[u];
    if (row_word == kNoRow) continue;                 // block-uniform
    const uint32_t m = wk.ulen[u];
    uint32_t parts = (m + kSegChunk - 1) / kSegChunk;
    size_t stride = dim;                              // distance between the sums to add
    if (parts > kFoldWidth) { parts = (parts + kFoldWidth - 1) / kFoldWidth; stride = (size_t)kFoldWidth * dim; }
    const double* src = wk.partials + (size_t)wk.long_part0[li] * dim;
    const unsigned long long id = wk.uid[u];
    for (uint32_t cbase = 0; cbase < dim; cbase += 256) {
      const uint32_t width = dim - cbase < 256 ? dim - cbase : 256;      // multiple of 4
      uint32_t slices = kCombineThreads / width;
      if (slices > kMaxSlices) slices = kMaxSlices;
      const uint32_t col = threadIdx.x % width, slice = threadIdx.x / width;
      if (slice < slices) {
        const uint32_t per = (parts + slices - 1) / slices;
        const uint32_t p_lo = slice * per, p_hi = p_lo + per < parts ? p_lo + per : parts;
        double a0 = 0.0, a1 = 0.0;
        uint32_t p = p_lo;
        for (; p + 2 <= p_hi; p += 2) { a0 += src[p * stride + cbase + col]; a1 += src[(p + 1) * stride + cbase + col]; }
        if (p < p_hi) a0 += src[p * stride + cbase + col];
        s_sum[slice][col] = a0 + a1;
      }
      __syncthreads();
      if (threadIdx.x < width / 4) {
        D4 g = D4{0.0, 0.0, 0.0, 0.0};
        for (uint32_t s = 0; s < slices; ++s) {
          g.x += s_sum[s][threadIdx.x * 4 + 0];
          g.y += s_sum[s][threadIdx.x * 4 + 1];
          g.z += s_sum[s][threadIdx.x * 4 + 2];
          g.w += s_sum[s][threadIdx.x * 4 + 3];
        }
        update_row(tv, row_word, id, cbase / 4 + threadIdx.x, g);
      }
      __syncthreads();
    }
  }
}

__global__ void __launch_bounds__(kCombineThreads)
combine_adagrad_kernel(TableView tv, Work wk) { after_previous_kernel(); combine_adagrad_body(tv, wk, blockIdx.x, gridDim.x); }

}  // namespace mono
