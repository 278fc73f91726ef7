// Backward, phase 1: group the batch's ID occurrences by ID.
//
// The paper does not describe this step; it is what turns the parameter push
// of Section 2.2, for a batch with repeated IDs, into one update per distinct
// ID.  Output: the distinct IDs uid[0..U), their segment offsets
// useg[0..U] into bag_of_sorted[], which lists, ID by ID, the bag of every
// occurrence of that ID.
//
// Method: a per-call open-addressing set of the batch's IDs in scratch memory
// (linear probing, 64-bit compare-and-swap on the key).  Inserting an
// occurrence yields its ID's slot and, from a fetch-add on the slot's counter,
// the occurrence's rank inside its ID's segment; a prefix sum over the
// multiplicities then gives every occurrence its final position directly, so
// no sort pass over the occurrences is needed.
#pragma once

#include "table_layout.cuh"

namespace mono {

struct __align__(16) BatchSlot {
  unsigned long long key;
  unsigned int count;     // multiplicity while counting, segment start after the scan
  unsigned int spare;
};

constexpr uint32_t kNoSlot = 0xFFFFFFFFu;
constexpr uint32_t kSegChunk = 256;       // longest segment one lane group reduces alone
constexpr int kScanBlocks = 592;          // 4 per SM on 148 SMs
constexpr int kScanThreads = 256;

// Scratch of one mono_apply_grads call.
struct Work {
  BatchSlot* bset;           // [bset_mask + 1], all keys empty between calls
  unsigned long long bset_mask;
  uint32_t* occ_slot;        // [max_ids] slot of each occurrence, kNoSlot if padding / outside bags
  uint32_t* occ_rank;        // [max_ids] rank of the occurrence among those of its ID
  uint32_t* occ_bag;         // [max_ids] bag of each occurrence
  uint32_t* bag_of_sorted;   // [max_ids] bags, grouped by ID
  unsigned long long* uid;   // [max_ids] distinct IDs
  uint32_t* uslot;           // [max_ids] slot of each distinct ID
  uint32_t* useg;            // [max_ids + 1] segment offsets
  uint32_t* urow;            // [max_ids] row word per distinct ID (kNoRow / row | kFreshBit)
  uint32_t* ins_list;        // [max_ids] distinct IDs that were not in the key store
  uint32_t* block_sums;      // [kScanBlocks + 1]
  uint32_t* long_u;          // [max_long] distinct IDs whose segment is split
  uint32_t* long_part0;      // [max_long] first part of each
  uint32_t* part_u;          // [max_parts] owner (index into long_u) of each part
  double* partials;          // [max_parts][dim]
  uint32_t max_long, max_parts;
};

// bag -> occurrences: every occurrence learns which bag it belongs to.
__global__ void __launch_bounds__(256)
fill_occ_bag_kernel(const long long* __restrict__ offsets, long long n_bags, long long n_ids,
                    uint32_t* __restrict__ occ_bag, DevState* st) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long b = (long long)blockIdx.x * blockDim.x + threadIdx.x; b < n_bags; b += stride) {
    const long long lo = offsets[b], hi = offsets[b + 1];
    if (lo < 0 || hi < lo || hi > n_ids) { atomicOr(&st->error_bits, 4u); continue; }
    for (long long j = lo; j < hi; ++j) occ_bag[j] = (uint32_t)b;
  }
}

// One thread per occurrence.  Lanes of a warp that hold the same ID elect a
// leader that touches the set once for all of them.
__global__ void __launch_bounds__(256)
dedup_insert_kernel(Work wk, const unsigned long long* __restrict__ ids, long long n_ids,
                    const long long* __restrict__ offsets, long long n_bags, DevState* st,
                    unsigned long long seed) {
  __shared__ unsigned int s_new[8];
  __shared__ unsigned int s_base;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  long long first = offsets[0], last = offsets[n_bags];
  if (first < 0) first = 0;
  if (last > n_ids) last = n_ids;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long n_round = (n_ids + stride - 1) / stride;   // same trip count for every thread
  unsigned int valid_total = 0;

  for (long long it = 0; it < n_round; ++it) {
    const long long j = it * stride + (long long)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned long long id = kEmptyKey;
    if (j >= first && j < last) id = ids[j];
    const bool valid = id != kEmptyKey;
    const unsigned peers = __match_any_sync(0xFFFFFFFFu, id);
    const int leader = __ffs(peers) - 1;
    const unsigned my_rank = __popc(peers & ((1u << lane) - 1u));
    unsigned long long slot = 0;
    unsigned int base = 0;
    bool is_new = false;
    if (valid && lane == leader) {
      slot = mix_b(id ^ seed) >> 20 & wk.bset_mask;
      // the set has at least twice as many slots as a call has IDs, so an empty
      // slot is always reached; the bound only guards against misuse
      for (unsigned long long probe = 0; probe <= wk.bset_mask; ++probe) {
        unsigned long long k = *reinterpret_cast<volatile unsigned long long*>(&wk.bset[slot].key);
        if (k == kEmptyKey) {
          k = atomicCAS(&wk.bset[slot].key, kEmptyKey, id);
          if (k == kEmptyKey) { is_new = true; break; }
        }
        if (k == id) break;
        slot = (slot + 1) & wk.bset_mask;
      }
      base = atomicAdd(&wk.bset[slot].count, (unsigned)__popc(peers));
    }
    // block-wide numbering of the IDs seen for the first time
    const unsigned new_mask = __ballot_sync(0xFFFFFFFFu, is_new);
    if (lane == 0) s_new[warp] = __popc(new_mask);
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned tot = 0;
      for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { const unsigned c = s_new[w]; s_new[w] = tot; tot += c; }
      s_base = tot ? atomicAdd(&st->n_unique, tot) : 0u;
    }
    __syncthreads();
    if (is_new) {
      const unsigned u = s_base + s_new[warp] + __popc(new_mask & ((1u << lane) - 1u));
      wk.uid[u] = id;
      wk.uslot[u] = (uint32_t)slot;
    }
    __syncthreads();   // s_new / s_base are rewritten next round
    const uint32_t slot32 = (uint32_t)__shfl_sync(0xFFFFFFFFu, (unsigned)slot, leader);
    base = __shfl_sync(0xFFFFFFFFu, base, leader);
    if (j < n_ids) {
      wk.occ_slot[j] = valid ? slot32 : kNoSlot;
      wk.occ_rank[j] = base + my_rank;
    }
    valid_total += valid;
  }
  // one counter update per warp
  for (int o = 16; o > 0; o >>= 1) valid_total += __shfl_down_sync(0xFFFFFFFFu, valid_total, o);
  if (lane == 0 && valid_total) atomicAdd(&st->n_valid_ids, valid_total);
}

// ---- exclusive prefix sum of the multiplicities: three small launches -------

__device__ inline uint32_t scan_range_begin(uint32_t n, int b) {
  const uint32_t per = (n + kScanBlocks - 1) / kScanBlocks;
  const unsigned long long s = (unsigned long long)per * b;
  return s < n ? (uint32_t)s : n;
}

__global__ void __launch_bounds__(kScanThreads)
seg_count_kernel(Work wk, const DevState* st) {
  __shared__ uint32_t s_part[kScanThreads / 32];
  const uint32_t n = st->n_unique;
  const uint32_t lo = scan_range_begin(n, blockIdx.x), hi = scan_range_begin(n, blockIdx.x + 1);
  uint32_t sum = 0;
  for (uint32_t u = lo + threadIdx.x; u < hi; u += kScanThreads) sum += wk.bset[wk.uslot[u]].count;
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_down_sync(0xFFFFFFFFu, sum, o);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t t = 0;
    for (int w = 0; w < kScanThreads / 32; ++w) t += s_part[w];
    wk.block_sums[blockIdx.x] = t;
  }
}

__global__ void seg_scan_blocks_kernel(Work wk) {
  // kScanBlocks values: one thread is enough
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    uint32_t run = 0;
    for (int b = 0; b < kScanBlocks; ++b) { const uint32_t c = wk.block_sums[b]; wk.block_sums[b] = run; run += c; }
    wk.block_sums[kScanBlocks] = run;
  }
}

// Writes useg[], turns every slot's counter into its segment start, and lists
// the IDs whose segments are long enough to be reduced in parts.
__global__ void __launch_bounds__(kScanThreads)
seg_offsets_kernel(Work wk, DevState* st) {
  __shared__ uint32_t s_warp[kScanThreads / 32];
  __shared__ uint32_t s_run;
  const uint32_t n = st->n_unique;
  const uint32_t lo = scan_range_begin(n, blockIdx.x), hi = scan_range_begin(n, blockIdx.x + 1);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) s_run = wk.block_sums[blockIdx.x];
  __syncthreads();
  for (uint32_t base = lo; base < hi; base += kScanThreads) {
    const uint32_t u = base + threadIdx.x;
    uint32_t slot = 0, m = 0;
    if (u < hi) { slot = wk.uslot[u]; m = wk.bset[slot].count; }
    uint32_t incl = m;
    for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += t; }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    uint32_t before = s_run;
    for (int w = 0; w < warp; ++w) before += s_warp[w];
    const uint32_t start = before + incl - m;
    if (u < hi) {
      wk.useg[u] = start;
      wk.bset[slot].count = start;
      if (m > kSegChunk) {
        const uint32_t parts = (m + kSegChunk - 1) / kSegChunk;
        const uint32_t li = atomicAdd(&st->n_long, 1u);
        const uint32_t p0 = atomicAdd(&st->n_parts, parts);
        if (li < wk.max_long && p0 + parts <= wk.max_parts) {
          wk.long_u[li] = u;
          wk.long_part0[li] = p0;
          for (uint32_t p = 0; p < parts; ++p) wk.part_u[p0 + p] = li;
        }
      }
    }
    __syncthreads();
    if (threadIdx.x == kScanThreads - 1) s_run = before + incl;
    __syncthreads();
  }
  if (blockIdx.x == kScanBlocks - 1 && threadIdx.x == 0) wk.useg[n] = wk.block_sums[kScanBlocks];
}

// Every occurrence drops its bag at (segment start of its ID) + (its rank).
__global__ void __launch_bounds__(256)
place_kernel(Work wk, long long n_ids) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < n_ids; j += stride) {
    const uint32_t s = wk.occ_slot[j];
    if (s == kNoSlot) continue;
    wk.bag_of_sorted[wk.bset[s].count + wk.occ_rank[j]] = wk.occ_bag[j];
  }
}

// Empty the set again (only the slots that were used) for the next call.
__global__ void __launch_bounds__(256)
dedup_reset_kernel(Work wk, const DevState* st) {
  const uint32_t n = st->n_unique;
  const uint32_t stride = gridDim.x * blockDim.x;
  for (uint32_t u = blockIdx.x * blockDim.x + threadIdx.x; u < n; u += stride) {
    BatchSlot e; e.key = kEmptyKey; e.count = 0; e.spare = 0;
    wk.bset[wk.uslot[u]] = e;
  }
}

}  // namespace mono
