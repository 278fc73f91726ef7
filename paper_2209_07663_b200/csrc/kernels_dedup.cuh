// Backward, phase 1: group the batch's ID occurrences by ID.
//
// The paper does not describe this step; it is what turns the parameter push
// of Section 2.2, for a batch with repeated IDs, into one update per distinct
// ID.  Output: the distinct IDs uid[0..U) with their slot in a per-call set,
// and for every occurrence its ID's slot and its rank among the occurrences of
// that ID.
//
// Method: a per-call open-addressing set of the batch's IDs in scratch memory
// (linear probing, 64-bit compare-and-swap on the key).  A block first groups
// its tile of occurrences in a shared-memory table, so that an ID that fills
// several percent of a batch (the head of a Zipf distribution) costs one
// global atomic per tile instead of one per occurrence; then it touches the
// global set once per distinct ID of the tile.  The fetch-add on the slot's
// counter returns the tile's base rank for that ID, so no sort pass over the
// occurrences is needed.
#pragma once

#include "table_layout.cuh"

namespace mono {

// One slot of the per-call set.  `a` is the ID's multiplicity while the batch
// is being counted.  Once the distinct IDs have been looked up in the key store
// (table_update_kernel), `a` is the start of the ID's segment in bag_of_sorted[]
// (kNoSegment for an ID that occurs once: its bag is found through uocc[]) and
// `b` the row the ID owned before this push (kNoRow if none): what an
// occurrence needs to pool the row and to file its bag.  The kernels that
// update the rows empty the slots again for the next call.
struct __align__(16) BatchSlot {
  unsigned long long key;
  unsigned int a;
  unsigned int b;
};

constexpr uint32_t kNoSlot = 0xFFFFFFFFu;
constexpr uint32_t kNoSegment = 0xFFFFFFFFu;
constexpr uint32_t kSegChunk = 64;             // longest segment one lane group reduces alone
constexpr uint32_t kFoldWidth = 64;           // parts added up by one block of fold_partials_kernel
constexpr int kTileIds = 512;                  // occurrences per block of dedup_tile_kernel
constexpr int kTileSlots = 1024;               // shared-memory table of one tile
constexpr int kTileThreads = 256;              // block size of dedup_tile_kernel
constexpr int kPrimaryProbes = 16;             // positions tried in the primary tier of the per-call set
constexpr uint32_t kWindows = 1024;            // the parts of long segments are scheduled by position in the batch, this finely

// Scratch of one mono_apply_grads call.
struct Work {
  // The per-call set has two tiers, both empty between calls.  The primary tier
  // is small enough to stay in L2 for a batch with the usual share of repeats;
  // an ID that finds no free slot among its first kPrimaryProbes positions there
  // goes to the secondary tier, which alone can hold a batch of all-distinct IDs.
  BatchSlot* bset;           // [primary_mask + 1 + secondary_mask + 1]
  uint32_t primary_mask;     // primary tier: slots [0, primary_mask]
  uint32_t secondary_mask;   // secondary tier: slots primary_mask + 1 + [0, secondary_mask]
  uint2* occ;                // [max_ids] per occurrence: x = slot of its ID (kNoSlot if padding / outside bags),
                             //           y = rank of the occurrence among those of its ID
  uint32_t* occ_bag;         // [max_ids] bag of each occurrence
  uint32_t* bag_of_sorted;   // [max_ids] bags of the occurrences of repeated IDs, grouped by ID
  unsigned long long* uid;   // [max_ids] distinct IDs
  uint32_t* uslot;           // [max_ids] slot of each distinct ID
  uint32_t* uocc;            // [max_ids] one occurrence of each distinct ID (the occurrence, if there is only one)
  uint32_t* useg;            // [max_ids] start of the ID's segment in bag_of_sorted
  uint32_t* ulen;            // [max_ids] multiplicity of the ID in this batch
  uint32_t* urow;            // [max_ids] row word per distinct ID (kNoRow / row | kFreshBit)
  unsigned long long* ucell; // [max_ids] where the key store holds the ID (kNoCell: nowhere) and
  unsigned long long* umeta; // [max_ids] the metadata found there, from the look-up that mono_prepare_push does
                             //           ahead of the push
  uint32_t* ins_list;        // [max_ids] distinct IDs that are not in the key store yet
  uint32_t* multi_list;         // [max_ids / 2 + 1] the distinct IDs that occur more than once, in one record each:
                             //           x = its number u, y = multiplicity, z = segment start, w = slot
  uint32_t* long_u;          // [max_long] distinct IDs whose segment is reduced in parts
  uint32_t* long_part0;      // [max_long] first part of each
  uint32_t* part_u;          // [max_parts] owner (index into long_u) of each part
  uint32_t* part_order;      // [max_parts] the parts in the order they are reduced in: by window of the batch
  uint32_t* win_count;       // [2 * kWindows] parts per window, then a cursor per window; zero between calls
  double* partials;          // [max_parts][dim]
  uint32_t* fold_li;         // [max_folds] owner (index into long_u) of each fold
  uint32_t* fold_idx;        // [max_folds] which group of kFoldWidth parts of that owner
  uint32_t max_long, max_parts, max_folds;
  uint32_t max_ids;          // entries of the per-occurrence and per-distinct-ID arrays
  uint32_t n_slots;          // slots of bset, both tiers
  unsigned int* error_bits;  // the table's sticky condition bits (the checked build reports through them)
};

// A bag is well formed when 0 <= offsets[b] <= offsets[b+1] <= n_ids; any other bag is
// treated as empty by every kernel.
__device__ inline bool bag_ok(long long lo, long long hi, long long n_ids) { return lo >= 0 && hi >= lo && hi <= n_ids; }

// bag -> occurrences: every occurrence learns which bag it belongs to.  A malformed bag
// writes nothing, sets the sticky condition bit and marks the call, so that the grouping
// pass checks every occurrence against the bag it claims (occurrence_covered).
__device__ inline void fill_occ_bag_body(const long long* __restrict__ offsets, long long n_bags, long long n_ids,
                                         uint32_t* __restrict__ occ_bag, DevState* st, uint32_t vblock, uint32_t vgrid) {
  const long long stride = (long long)vgrid * blockDim.x;
  for (long long b = (long long)vblock * blockDim.x + threadIdx.x; b < n_bags; b += stride) {
    const long long lo = offsets[b], hi = offsets[b + 1];
    if (!bag_ok(lo, hi, n_ids)) { atomicOr(&st->error_bits, 4u /* MONO_DEV_BAD_OFFSETS */); st->call_bad_offsets = 1u; continue; }
    for (long long j = lo; j < hi; ++j) occ_bag[j] = (uint32_t)b;
  }
}
__global__ void __launch_bounds__(256)
fill_occ_bag_kernel(const long long* __restrict__ offsets, long long n_bags, long long n_ids,
                    uint32_t* __restrict__ occ_bag, DevState* st) { after_previous_kernel();
  fill_occ_bag_body(offsets, n_bags, n_ids, occ_bag, st, blockIdx.x, gridDim.x);
}

// Only used when the call's offsets are malformed: does a well-formed bag cover occurrence j,
// and is it the one occ_bag[j] names?  (occ_bag[j] may be left over from an earlier call where
// no bag of this call covers j; the test against this call's offsets settles it either way.)
__device__ inline bool occurrence_covered(const uint32_t* __restrict__ occ_bag, const long long* __restrict__ offsets,
                                          long long n_bags, long long n_ids, long long j) {
  const uint32_t b = occ_bag[j];
  if ((long long)b >= n_bags) return false;
  const long long lo = offsets[b], hi = offsets[b + 1];
  return bag_ok(lo, hi, n_ids) && j >= lo && j < hi;
}

// Sum of `v` over the block and this thread's exclusive prefix, with two
// barriers.  s_warp needs one word per warp.  All threads must call.
__device__ inline unsigned long long block_exclusive_scan(unsigned long long v, unsigned long long* s_warp,
                                                          unsigned long long* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = (blockDim.x + 31) >> 5;
  unsigned long long incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();                       // s_warp may still be read from a previous call
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  unsigned long long before = 0, all = 0;
  for (int w = 0; w < n_warps; ++w) {
    const unsigned long long c = s_warp[w];
    if (w < warp) before += c;
    all += c;
  }
  *total = all;
  return before + incl - v;
}

// One block per tile of kTileIds consecutive occurrences.
// (eight blocks per SM: measured 0.207 ms on the largest configuration against 0.234 ms with six)
__device__ inline void dedup_tile_body(const Work& wk, const unsigned long long* __restrict__ ids, long long n_ids,
                                       const long long* __restrict__ offsets, long long n_bags, DevState* st,
                                       unsigned long long seed, uint32_t vblock) {
  constexpr int kPerThread = kTileIds / kTileThreads;
  __shared__ unsigned long long s_key[kTileSlots];
  __shared__ unsigned int s_cnt[kTileSlots];     // multiplicity in the tile, then base rank
  __shared__ unsigned int s_gslot[kTileSlots];   // the ID's slot in the global set
  __shared__ unsigned long long s_warp[kTileThreads / 32];
  __shared__ unsigned int s_ubase;

  for (int i = threadIdx.x; i < kTileSlots; i += kTileThreads) { s_key[i] = kEmptyKey; s_cnt[i] = 0; }
  long long first = offsets[0], last = offsets[n_bags];
  if (first < 0) first = 0;
  if (last > n_ids) last = n_ids;
  const bool check_each = st->call_bad_offsets != 0u;     // set by fill_occ_bag_kernel, earlier on this stream
  if (check_each) { first = 0; last = n_ids; }
  __syncthreads();

  // 1. group the tile's occurrences in shared memory.  The thread whose occurrence puts an ID
  //    into the tile's table owns that ID for the rest of the kernel.
  const long long tile0 = (long long)vblock * kTileIds;
  unsigned long long my_id[kPerThread];
  uint32_t my_slot[kPerThread], my_rank[kPerThread];
  bool own[kPerThread];
  unsigned int n_valid = 0;
#pragma unroll
  for (int k = 0; k < kPerThread; ++k) {
    const long long j = tile0 + k * kTileThreads + threadIdx.x;
    unsigned long long id = kEmptyKey;
    if (j >= first && j < last) id = ids[j];
    // malformed offsets: an occurrence that no well-formed bag covers is padding, as in the lookup
    if (check_each && id != kEmptyKey && !occurrence_covered(wk.occ_bag, offsets, n_bags, n_ids, j)) id = kEmptyKey;
    my_id[k] = id;
    my_slot[k] = kNoSlot;
    my_rank[k] = 0;
    own[k] = false;
    if (id != kEmptyKey) {
      ++n_valid;
      uint32_t s = (uint32_t)(mix_a(id ^ seed) >> 40) & (kTileSlots - 1);
      for (int probe = 0; probe < kTileSlots; ++probe) {      // at most kTileIds keys in kTileSlots slots
        const unsigned long long old = atomicCAS(&s_key[s], kEmptyKey, id);
        if (old == kEmptyKey) { own[k] = true; break; }
        if (old == id) break;
        s = (s + 1) & (kTileSlots - 1);
      }
      my_slot[k] = s;
      my_rank[k] = atomicAdd(&s_cnt[s], 1u);
    }
  }
  __syncthreads();

  // 2. one visit of the global set per distinct ID of the tile, by the ID's owner.  The first
  //    probes of a thread's IDs are issued together, then resolved, then the counter updates
  //    are issued together, so their latencies overlap.
  unsigned long long seen[kPerThread];
  uint32_t g[kPerThread], base_rank[kPerThread];
  bool is_new[kPerThread];
#pragma unroll
  for (int k = 0; k < kPerThread; ++k) {
    g[k] = (uint32_t)(mix_b(my_id[k] ^ seed) >> 20) & wk.primary_mask;
    seen[k] = own[k] ? *reinterpret_cast<volatile unsigned long long*>(&wk.bset[g[k]].key) : 0ull;
  }
  unsigned int n_new = 0;
#pragma unroll
  for (int k = 0; k < kPerThread; ++k) {
    is_new[k] = false;
    if (!own[k]) continue;
    const unsigned long long id = my_id[k];
    unsigned long long kk = seen[k];
    bool placed = false;
    // primary tier: a short window of consecutive positions
    for (int probe = 0; probe < kPrimaryProbes; ++probe) {
      if (kk == kEmptyKey) {
        kk = atomicCAS(&wk.bset[g[k]].key, kEmptyKey, id);
        if (kk == kEmptyKey) { is_new[k] = true; placed = true; break; }
      }
      if (kk == id) { placed = true; break; }
      g[k] = (g[k] + 1) & wk.primary_mask;
      kk = *reinterpret_cast<volatile unsigned long long*>(&wk.bset[g[k]].key);
    }
    if (!placed) {
      // secondary tier: it has at least twice as many slots as a call has IDs, so
      // an empty slot is always reached; the bound only guards against misuse
      const uint32_t base2 = wk.primary_mask + 1u;
      uint32_t q = (uint32_t)(mix_a(id ^ seed) >> 24) & wk.secondary_mask;
      for (uint32_t probe = 0; probe <= wk.secondary_mask; ++probe) {
        kk = *reinterpret_cast<volatile unsigned long long*>(&wk.bset[base2 + q].key);
        if (kk == kEmptyKey) {
          kk = atomicCAS(&wk.bset[base2 + q].key, kEmptyKey, id);
          if (kk == kEmptyKey) { is_new[k] = true; break; }
        }
        if (kk == id) break;
        q = (q + 1) & wk.secondary_mask;
      }
      g[k] = base2 + q;
    }
    n_new += is_new[k];
  }
#pragma unroll
  for (int k = 0; k < kPerThread; ++k)
    base_rank[k] = own[k] ? atomicAdd(&wk.bset[g[k]].a, s_cnt[my_slot[k]]) : 0u;
#pragma unroll
  for (int k = 0; k < kPerThread; ++k) {
    if (!own[k]) continue;
    s_cnt[my_slot[k]] = base_rank[k];
    s_gslot[my_slot[k]] = g[k];
  }
  // number the IDs this tile saw first: one counter update per tile
  // (new IDs in the low word, valid occurrences in the high word of one scan)
  unsigned long long total = 0;
  unsigned int my_u = (unsigned int)block_exclusive_scan(((unsigned long long)n_valid << 32) | n_new, s_warp, &total);
  if (threadIdx.x == 0) {
    const unsigned int total_new = (unsigned int)total, total_valid = (unsigned int)(total >> 32);
    s_ubase = total_new ? atomicAdd(&st->n_unique, total_new) : 0u;
    if (total_valid) atomicAdd(&st->n_valid_ids, total_valid);
  }
  __syncthreads();
  my_u += s_ubase;
#pragma unroll
  for (int k = 0; k < kPerThread; ++k) {
    if (is_new[k]) {
      if (MONO_INDEX_OK(wk.error_bits, my_u, wk.max_ids)) {
        wk.uid[my_u] = my_id[k];
        wk.uslot[my_u] = g[k];
        wk.uocc[my_u] = (uint32_t)(tile0 + k * kTileThreads + threadIdx.x);     // the owner's own occurrence
      }
      ++my_u;
    }
  }

  // 3. every occurrence learns its ID's slot and its rank
#pragma unroll
  for (int k = 0; k < kPerThread; ++k) {
    const long long j = tile0 + k * kTileThreads + threadIdx.x;
    if (j < n_ids) {
      const uint32_t s = my_slot[k];
      wk.occ[j] = s == kNoSlot ? make_uint2(kNoSlot, 0u) : make_uint2(s_gslot[s], s_cnt[s] + my_rank[k]);
    }
  }
}

__global__ void __launch_bounds__(kTileThreads, 8)
dedup_tile_kernel(Work wk, const unsigned long long* __restrict__ ids, long long n_ids,
                  const long long* __restrict__ offsets, long long n_bags, DevState* st,
                  unsigned long long seed) { after_previous_kernel();
  dedup_tile_body(wk, ids, n_ids, offsets, n_bags, st, seed, blockIdx.x);
}

}  // namespace mono
