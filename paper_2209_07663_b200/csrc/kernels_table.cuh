// Mutating table kernels: count / stamp / admit for IDs that are already
// tracked, cuckoo insertion of new IDs (Section 2.1: place at h0, displace the
// occupant to its other bucket, repeat), the expiry sweep, and bulk import.
#pragma once

#include "kernels_dedup.cuh"
#include "kernels_forward.cuh"

namespace mono {

// Take a free row (one at a time: the bulk-import path).  Returns kNoRow (and
// records the refusal) when none is left.
__device__ inline uint32_t alloc_row(const TableView& tv) {
  const long long old = (long long)atomicAdd(reinterpret_cast<unsigned long long*>(&tv.st->free_top),
                                              (unsigned long long)(-1LL));
  if (old <= 0) {
    atomicAdd(reinterpret_cast<unsigned long long*>(&tv.st->free_top), 1ull);
    atomicOr(&tv.st->error_bits, 1u /* MONO_DEV_ROWS_FULL */);
    atomicAdd(&tv.st->n_rows_refused, 1ull);
    return kNoRow;
  }
  atomicAdd(&tv.st->n_resident, 1ull);
  atomicAdd(&tv.st->n_admitted_total, 1ull);
  return tv.free_rows[old - 1];
}

// Block-wide reservation for the batch path: every thread states whether its
// ID needs a row, whether it must be inserted into the key store (it then gets
// a place in ins_list[]), whether it occurs more than once in the batch (a
// place in multi_list[]) and how many entries of bag_of_sorted[] its segment
// takes (its multiplicity); one thread does the counter updates for the whole block, so counters
// that every admission would otherwise hit are touched once per block and
// round.  All threads of the block must call.
struct BlockAlloc {
  unsigned long long warp_sums[8];
  long long row_base;       // free_top before this block's reservation
  unsigned int rows_granted;
  unsigned int seg_base;
  unsigned int multi_base;
  unsigned int ins_base;
};

struct Reservation {
  uint32_t row;             // kNoRow if refused or not asked for
  uint32_t seg_start;
  uint32_t multi_pos;
  uint32_t ins_pos;
};

__device__ inline Reservation block_reserve(const TableView& tv, BlockAlloc* sh, bool need_row, bool is_multi,
                                            bool need_insert, uint32_t seg_len) {
  // segment entries in bits 0..31, repeated IDs in 32..41, inserts in 42..51, rows in 52..61
  unsigned long long total = 0;
  const unsigned long long mine = ((unsigned long long)(need_row ? 1u : 0u) << 52) |
                                  ((unsigned long long)(need_insert ? 1u : 0u) << 42) |
                                  ((unsigned long long)(is_multi ? 1u : 0u) << 32) | seg_len;
  const unsigned long long before = block_exclusive_scan(mine, sh->warp_sums, &total);
  // the four counters are updated by the first lanes of four different warps, so that their round
  // trips to memory overlap instead of following one another (blocks have at least four warps)
  const unsigned int rows_wanted = (unsigned int)(total >> 52) & 0x3FFu, ins_total = (unsigned int)(total >> 42) & 0x3FFu,
                     multi_total = (unsigned int)(total >> 32) & 0x3FFu, seg_total = (unsigned int)total;
  const unsigned int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31u) == 0u && warp < 4u) {
    if (warp == 0u) {
      unsigned int granted = 0;
      long long old = 0;
      if (rows_wanted) {
        old = (long long)atomicAdd(reinterpret_cast<unsigned long long*>(&tv.st->free_top),
                                   (unsigned long long)(-(long long)rows_wanted));
        const long long avail = old > 0 ? old : 0;
        granted = avail >= (long long)rows_wanted ? rows_wanted : (unsigned int)avail;
        if (granted < rows_wanted) {
          atomicAdd(reinterpret_cast<unsigned long long*>(&tv.st->free_top), (unsigned long long)(rows_wanted - granted));
          atomicOr(&tv.st->error_bits, 1u /* MONO_DEV_ROWS_FULL */);
          atomicAdd(&tv.st->n_rows_refused, (unsigned long long)(rows_wanted - granted));
        }
        if (granted) {
          atomicAdd(&tv.st->n_resident, (unsigned long long)granted);
          atomicAdd(&tv.st->n_admitted_total, (unsigned long long)granted);
        }
      }
      sh->row_base = old;
      sh->rows_granted = granted;
    } else if (warp == 1u) {
      sh->seg_base = seg_total ? atomicAdd(&tv.st->seg_cursor, seg_total) : 0u;
    } else if (warp == 2u) {
      sh->multi_base = multi_total ? atomicAdd(&tv.st->n_multi, multi_total) : 0u;
    } else {
      sh->ins_base = ins_total ? atomicAdd(&tv.st->n_insert, ins_total) : 0u;
    }
  }
  __syncthreads();
  Reservation r;
  r.seg_start = sh->seg_base + (unsigned int)before;
  r.multi_pos = sh->multi_base + ((unsigned int)(before >> 32) & 0x3FFu);
  r.ins_pos = sh->ins_base + ((unsigned int)(before >> 42) & 0x3FFu);
  const unsigned int my_row_index = (unsigned int)(before >> 52) & 0x3FFu;
  r.row = kNoRow;
  if (need_row && my_row_index < sh->rows_granted &&
      MONO_INDEX_OK(&tv.st->error_bits, sh->row_base - 1 - (long long)my_row_index, tv.capacity))
    r.row = tv.free_rows[sh->row_base - 1 - my_row_index];
  return r;
}

// A distinct ID whose segment is longer than kSegChunk is reduced in parts:
// register it and its parts.  Rare (the few hottest IDs of a batch).
__device__ inline void register_long(const TableView& tv, const Work& wk, uint32_t u, uint32_t m) {
  const uint32_t parts = (m + kSegChunk - 1) / kSegChunk;
  const uint32_t li = atomicAdd(&tv.st->n_long, 1u);
  const uint32_t p0 = atomicAdd(&tv.st->n_parts, parts);
  if (li < wk.max_long && p0 + parts <= wk.max_parts) {
    wk.long_u[li] = u;
    wk.long_part0[li] = p0;
    // (part_u[] is filled by expand_parts_kernel: a segment can have thousands of parts)
    if (parts > kFoldWidth) {
      // very long segment: its parts are first added up in groups of kFoldWidth
      const uint32_t nf = (parts + kFoldWidth - 1) / kFoldWidth;
      const uint32_t f0 = atomicAdd(&tv.st->n_folds, nf);
      if (f0 + nf <= wk.max_folds)
        for (uint32_t f = 0; f < nf; ++f) { wk.fold_li[f0 + f] = li; wk.fold_idx[f0 + f] = f; }
    }
  }
}

// Phase 2 of a push: one thread per distinct ID, in up to two halves.
//
//  kLookUp  (can run ahead of the push, when mono_prepare_push announced the batch: it changes
//           nothing in the table) -- the ID's multiplicity is read from the per-call set, the ID is
//           looked up in the key store (the cell an insertion prefers first), an ID that occurs more
//           than once is given its segment of bag_of_sorted[] and its place in multi_list[];
//           the ID's slot of the per-call set is rewritten to (segment start, row owned so far),
//           which is what the occurrences need, and the cell is remembered in ucell[].
//  kCommit  (the push itself) -- a tracked ID gets count += multiplicity (saturating at the
//           threshold), last_seen = now, and a row if the count has reached the threshold; an ID
//           the key store does not hold is queued for insertion.  With kLookUp in an earlier
//           kernel, the cell and its metadata are the remembered ones: the kernel reads its
//           inputs in order and only scatters the new metadata words.
//
// Both halves in one kernel is the push that was not announced.  No cell moves during either
// half, so the thread whose ID sits in a cell owns it.
enum : int { kLookUp = 1, kCommit = 2 };

__device__ inline Cell* cell_address(const TableView& tv, unsigned long long cell, unsigned long long n_cells) {
  return cell < n_cells ? tv.cells + cell : tv.stash + (cell - n_cells);
}

template <int MODE>
__device__ inline void table_update_body(const TableView& tv, const Work& wk, uint32_t now, uint32_t vblock, uint32_t vgrid) {
  __shared__ BlockAlloc sh;
  const uint32_t n = tv.st->n_unique;
  const unsigned stash_hw = tv.st->stash_hw;
  const unsigned long long n_cells = (tv.bucket_mask + 1) * kCellsPerBucket;
  const int lane = threadIdx.x & 31;
  unsigned int n_res = 0;
  for (uint32_t base = vblock * blockDim.x; base < n; base += vgrid * blockDim.x) {   // block-uniform
    const uint32_t u = base + threadIdx.x;
    const bool active = u < n;
    unsigned long long id = kEmptyKey, meta = 0, cell = kNoCell;
    uint32_t m = 0, slot = 0;
    if (active) {
      id = wk.uid[u];
      if (MODE & kLookUp) {
        slot = wk.uslot[u];
        if (!MONO_INDEX_OK(wk.error_bits, slot, wk.n_slots)) slot = 0;
        m = wk.bset[slot].a;
        cell = thread_locate(tv, id, stash_hw, &meta);
      } else {
        // nothing has changed the table since the look-up (every call that could forgets the
        // announcement), so the cell and its metadata are as remembered
        m = wk.ulen[u];
        cell = wk.ucell[u];
        meta = wk.umeta[u];
#ifdef MONO_DEBUG
        if (cell != kNoCell) {
          const Cell c = load_cell_whole(cell_address(tv, cell, n_cells));
          if (c.key != id || c.meta != meta) { atomicOr(&tv.st->error_bits, 16u /* MONO_DEV_INTERNAL */); cell = thread_locate(tv, id, stash_hw, &meta); }
        }
#endif
      }
    }
    const bool hit = cell != kNoCell;
    uint32_t low = meta_low(meta);
    const bool resident = hit && (low & kResidentBit) != 0;
    bool need_row = false;
    if ((MODE & kCommit) && hit && !resident) {
      const unsigned long long c = (unsigned long long)low + m;
      low = c < tv.threshold ? (uint32_t)c : tv.threshold;
      need_row = low >= tv.threshold;
    }
    // exact filter: a new ID that this batch alone takes to the threshold gets its row here too, so
    // that the insertion that follows has nothing to tell the kernels that update rows
    const bool exact = tv.sketch_depth == 0;
    if ((MODE & kCommit) && exact && active && !hit && m >= tv.threshold) need_row = true;
    const Reservation rv = block_reserve(tv, &sh, need_row, (MODE & kLookUp) && m > 1, (MODE & kCommit) && active && !hit,
                                         ((MODE & kLookUp) && m > 1) ? m : 0u);
    if (!active) continue;
    if (MODE & kLookUp) {
      wk.ulen[u] = m;
      wk.useg[u] = rv.seg_start;
      if (!(MODE & kCommit)) { wk.ucell[u] = cell; wk.umeta[u] = meta; }
      BatchSlot bs; bs.key = id; bs.a = m > 1 ? rv.seg_start : kNoSegment; bs.b = resident ? (low & kRowMask) : kNoRow;
      wk.bset[slot] = bs;
      (void)MONO_INDEX_OK(wk.error_bits, (unsigned long long)rv.seg_start + m - 1, wk.max_ids);
      if (m > 1 && MONO_INDEX_OK(wk.error_bits, rv.multi_pos, wk.max_ids / 2 + 1)) wk.multi_list[rv.multi_pos] = u;
    }
    if (MODE & kCommit) {
      if (hit) {
        uint32_t row_word = kNoRow;
        // every ID of the batch that has a row is trained in this call: mark it for the next sync
        if (resident) { row_word = low & kRowMask; low |= kTouchedBit; }
        else if (rv.row != kNoRow) { low = kResidentBit | kTouchedBit | rv.row; row_word = rv.row | kFreshBit; }
        cell_address(tv, cell, n_cells)->meta = make_meta(now, low);
        wk.urow[u] = row_word;
        if (row_word != kNoRow) {
          ++n_res;
          if (m > kSegChunk) register_long(tv, wk, u, m);
        }
      } else {
        if (exact) {
          const uint32_t row_word = rv.row != kNoRow ? (rv.row | kFreshBit) : kNoRow;
          wk.urow[u] = row_word;
          if (row_word != kNoRow) {
            ++n_res;
            if (m > kSegChunk) register_long(tv, wk, u, m);
          }
        }
        if (MONO_INDEX_OK(wk.error_bits, rv.ins_pos, wk.max_ids)) wk.ins_list[rv.ins_pos] = u;
      }
    }
  }
  if (MODE & kCommit) {
    for (int o = 16; o > 0; o >>= 1) n_res += __shfl_down_sync(0xFFFFFFFFu, n_res, o);
    if (lane == 0 && n_res) atomicAdd(&tv.st->sum_unique_resident, (unsigned long long)n_res);
  }
}

// (six blocks per SM: measured 0.210 ms on the largest configuration for both halves in one kernel, against
// 0.222 ms for look-ups shared within quads, which need twice the registers)
template <int MODE>
__global__ void __launch_bounds__(256, 6)
table_update_kernel(TableView tv, Work wk, uint32_t now) { after_previous_kernel();
  table_update_body<MODE>(tv, wk, now, blockIdx.x, gridDim.x);
}

// An entry whose metadata is `meta` has just been written into a cell of bucket `bkt`: the
// bucket's record of its oldest stamp may not stay above that entry's.  (Entries that leave a
// bucket, and stamps that are renewed, leave the record as it is: it only has to be a lower
// bound, and the sweep makes it exact again whenever it visits the bucket.)  `rec` is the
// record as read before the write; records only fall while entries are being inserted, so a
// value read earlier is at or above the present one and the test errs on the safe side.
__device__ inline void note_stamp(const TableView& tv, unsigned long long bkt, unsigned long long meta, uint32_t rec) {
  if (rec > meta_time(meta)) atomicMin(tv.oldest + bkt, meta_time(meta));
}

// Put `item` (a key that is in no cell) into the key store.  Lock-free against
// other inserters: an empty cell is claimed, and an occupant displaced, with a
// single 16-byte atomic, so every entry is at all times either in exactly one
// cell or carried by exactly one thread.  The displacement chain is bounded;
// what is still carried at the end goes to the stash, and if that is full the
// entry is dropped and the condition recorded.
__device__ inline void cuckoo_insert(const TableView& tv, Cell item) {
  const Cell empty = empty_cell();
  unsigned long long h0 = tv.hash0(item.key), h1 = tv.hash1(item.key);
  unsigned long long bkt = h0 & tv.bucket_mask;
  uint32_t first = (uint32_t)(h0 >> 62);            // the cell of this bucket the entry prefers
  uint32_t rnd = (uint32_t)(item.key >> 17) * 2654435761u + 0x9E3779B9u;
  uint32_t chain = 0;
  bool placed = false;
  for (;;) {
    Cell* base = tv.cells + bkt * kCellsPerBucket;
    const uint32_t rec = __ldcg(tv.oldest + bkt);
    for (uint32_t c = 0; c < kCellsPerBucket && !placed; ++c) {
      Cell* p = base + ((c + first) & 3u);
      if (*reinterpret_cast<volatile unsigned long long*>(&p->key) == kEmptyKey) {
        const Cell old = atomicCAS(p, empty, item);
        placed = old.key == kEmptyKey;
      }
    }
    if (placed) { note_stamp(tv, bkt, item.meta, rec); break; }
    if (chain == 0) {
      // a new ID may take an empty cell of its second bucket before displacing anyone
      const unsigned long long alt = h1 & tv.bucket_mask;
      Cell* abase = tv.cells + alt * kCellsPerBucket;
      for (uint32_t c = 0; c < kCellsPerBucket && !placed && alt != bkt; ++c) {
        Cell* p = abase + ((c + (uint32_t)(h1 >> 62)) & 3u);
        if (*reinterpret_cast<volatile unsigned long long*>(&p->key) == kEmptyKey) {
          const Cell old = atomicCAS(p, empty, item);
          placed = old.key == kEmptyKey;
        }
      }
      if (placed) { note_stamp(tv, alt, item.meta, __ldcg(tv.oldest + alt)); break; }
    }
    if (chain >= kMaxChain) break;
    ++chain;
    rnd = rnd * 1664525u + 1013904223u;
    const Cell old = atomicExch(base + (rnd >> 30), item);
    note_stamp(tv, bkt, item.meta, rec);
    if (old.key == kEmptyKey) { placed = true; break; }
    item = old;
    h0 = tv.hash0(item.key);
    h1 = tv.hash1(item.key);
    const bool to_second = (h0 & tv.bucket_mask) == bkt;
    bkt = (to_second ? h1 : h0) & tv.bucket_mask;
    first = (uint32_t)((to_second ? h1 : h0) >> 62);
  }
  if (chain) {
    atomicAdd(&tv.st->n_evictions_total, (unsigned long long)chain);
    atomicMax(&tv.st->max_chain, chain);
  }
  if (placed) return;
  for (uint32_t i = 0; i < kStashCells; ++i) {
    if (*reinterpret_cast<volatile unsigned long long*>(&tv.stash[i].key) == kEmptyKey) {
      const Cell old = atomicCAS(tv.stash + i, empty, item);
      if (old.key == kEmptyKey) { atomicMax(&tv.st->stash_hw, i + 1u); return; }
    }
  }
  // nowhere to go: the carried entry is lost (its row, if any, stays allocated)
  atomicOr(&tv.st->error_bits, 2u /* MONO_DEV_KEYS_FULL */);
  atomicAdd(&tv.st->n_keys_dropped, 1ull);
  atomicAdd(&tv.st->n_tracked, (unsigned long long)(-1LL));
  if (meta_resident(item.meta)) atomicAdd(&tv.st->n_resident, (unsigned long long)(-1LL));
}

// Probabilistic filter, between phases 2 and 3: every distinct ID that is not in the key
// store adds its multiplicity to one counter per sketch row.  All additions of a batch are
// done before any estimate is read (next kernel), so the outcome does not depend on order.
__device__ inline void sketch_add_body(const TableView& tv, const Work& wk, uint32_t vblock, uint32_t vgrid) {
  const uint32_t n = tv.st->n_insert;
  const uint32_t stride = vgrid * blockDim.x;
  for (uint32_t i = vblock * blockDim.x + threadIdx.x; i < n; i += stride) {
    const uint32_t u = wk.ins_list[i];
    const unsigned long long id = wk.uid[u];
    const uint32_t m = wk.ulen[u];
    for (uint32_t r = 0; r < tv.sketch_depth; ++r) atomicAdd(tv.sketch_counter(r, id), m);
  }
}
__global__ void __launch_bounds__(256)
sketch_add_kernel(TableView tv, Work wk) { after_previous_kernel(); sketch_add_body(tv, wk, blockIdx.x, gridDim.x); }

// Phase 3 of a push: one thread per ID that phase 2 found unknown to the key store.
// Exact filter: it is inserted; whether it has a row straight away (the batch alone reached
// the threshold) was settled in phase 2, which left the row in urow[], so nothing that
// updates rows waits for this kernel.  Probabilistic filter: it is inserted, with a row,
// only if its sketch estimate has reached the threshold; otherwise nothing is stored for it.
__device__ inline void table_insert_body(const TableView& tv, const Work& wk, uint32_t now, uint32_t vblock, uint32_t vgrid) {
  __shared__ BlockAlloc sh;
  const uint32_t n = tv.st->n_insert;
  const int lane = threadIdx.x & 31;
  const bool sketch = tv.sketch_depth != 0;
  unsigned int n_res = 0, n_done = 0;
  for (uint32_t base = vblock * blockDim.x; base < n; base += vgrid * blockDim.x) {   // block-uniform
    const bool todo = base + threadIdx.x < n;
    uint32_t u = 0, m = 0;
    if (todo) { u = wk.ins_list[base + threadIdx.x]; m = wk.ulen[u]; }
    uint32_t count = m < tv.threshold ? m : tv.threshold;
    uint32_t row_word = kNoRow;
    if (sketch) {
      if (todo) {
        const unsigned int est = tv.sketch_estimate(wk.uid[u]);
        count = est < tv.threshold ? est : tv.threshold;
      }
      const bool need_row = todo && count >= tv.threshold;
      const Reservation rv = block_reserve(tv, &sh, need_row, false, false, 0u);
      if (!todo) continue;
      if (rv.row != kNoRow) row_word = rv.row | kFreshBit;
      wk.urow[u] = row_word;
      if (row_word != kNoRow) {
        ++n_res;
        if (m > kSegChunk) register_long(tv, wk, u, m);
      }
      if (row_word == kNoRow) continue;                // below the estimate (or no row left): not stored
    } else {
      if (!todo) continue;
      row_word = wk.urow[u];
    }
    const uint32_t low = row_word != kNoRow ? (kResidentBit | kTouchedBit | (row_word & ~kFreshBit)) : count;
    Cell item; item.key = wk.uid[u]; item.meta = make_meta(now, low);
    cuckoo_insert(tv, item);
    ++n_done;
  }
  for (int o = 16; o > 0; o >>= 1) {
    n_res += __shfl_down_sync(0xFFFFFFFFu, n_res, o);
    n_done += __shfl_down_sync(0xFFFFFFFFu, n_done, o);
  }
  if (lane == 0) {
    if (n_res) atomicAdd(&tv.st->sum_unique_resident, (unsigned long long)n_res);
    if (n_done) {
      atomicAdd(&tv.st->n_tracked, (unsigned long long)n_done);
      atomicAdd(&tv.st->n_inserted_total, (unsigned long long)n_done);
    }
  }
}
__global__ void __launch_bounds__(256)
table_insert_kernel(TableView tv, Work wk, uint32_t now) { after_previous_kernel();
  table_insert_body(tv, wk, now, blockIdx.x, gridDim.x);
}

// Window of the batch that part k of a segment of `parts` parts falls into.  A segment lists
// its occurrences roughly in batch order (tile by tile), so part k of n covers roughly the
// k-th n-th of the bags.
__device__ inline uint32_t part_window(uint32_t k, uint32_t parts) {
  return (uint32_t)(((unsigned long long)k * kWindows) / parts);
}

// After phases 2 and 3: every part of a long segment learns which ID it belongs to
// (one block per long ID, its threads share the parts), and the parts are counted by window.
__device__ inline void expand_parts_body(const TableView& tv, const Work& wk, uint32_t vblock, uint32_t vgrid) {
  uint32_t n_long = tv.st->n_long;
  if (n_long > wk.max_long) n_long = wk.max_long;
  for (uint32_t li = vblock; li < n_long; li += vgrid) {
    const uint32_t parts = (wk.ulen[wk.long_u[li]] + kSegChunk - 1) / kSegChunk;
    const uint32_t p0 = wk.long_part0[li];
    if (p0 + parts > wk.max_parts) continue;
    for (uint32_t p = threadIdx.x; p < parts; p += blockDim.x) {
      wk.part_u[p0 + p] = li;
      atomicAdd(&wk.win_count[part_window(p, parts)], 1u);
    }
  }
}
__global__ void __launch_bounds__(128)
expand_parts_kernel(TableView tv, Work wk) { after_previous_kernel(); expand_parts_body(tv, wk, blockIdx.x, gridDim.x); }

// The order the parts are reduced in: window by window, so that the parts in flight at any
// time -- of different IDs -- gather gradient rows of the same stretch of bags, and a row
// that several hot IDs need is fetched from DRAM once and found in L2 by the others.
// Every block scans the window counts for itself; positions inside a window are handed out
// by a per-window cursor (their order does not matter: each part has its own partial sum).
__device__ inline void order_parts_body(const TableView& tv, const Work& wk, uint32_t vblock, uint32_t vgrid) {
  __shared__ uint32_t s_start[kWindows];
  __shared__ uint32_t s_warp[kWindows / 32];
  uint32_t n_parts = tv.st->n_parts;
  if (n_parts > wk.max_parts) n_parts = wk.max_parts;
  if (n_parts == 0) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t c = wk.win_count[threadIdx.x];
  uint32_t incl = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  uint32_t before = 0;
  for (int w = 0; w < warp; ++w) before += s_warp[w];
  s_start[threadIdx.x] = before + incl - c;
  __syncthreads();
  uint32_t* cursor = wk.win_count + kWindows;
  for (uint32_t p = vblock * blockDim.x + threadIdx.x; p < n_parts; p += vgrid * blockDim.x) {
    const uint32_t li = wk.part_u[p];
    const uint32_t parts = (wk.ulen[wk.long_u[li]] + kSegChunk - 1) / kSegChunk;
    const uint32_t w = part_window(p - wk.long_part0[li], parts);
    const uint32_t at = s_start[w] + atomicAdd(&cursor[w], 1u);
    if (MONO_INDEX_OK(wk.error_bits, at, wk.max_parts)) wk.part_order[at] = p;
  }
}
__global__ void __launch_bounds__(kWindows)
order_parts_kernel(TableView tv, Work wk) { after_previous_kernel(); order_parts_body(tv, wk, blockIdx.x, gridDim.x); }

// End of a mono_apply_grads call: fold the per-call counters into the totals
// (commit = 0: a grouping that was prepared but never applied is only forgotten).
// (one block)
__device__ inline void finish_apply_body(DevState* st, uint32_t* win_count, int commit) {
  const bool had_parts = st->n_parts != 0;
  __syncthreads();                                   // everyone has read n_parts before it is reset
  if (had_parts)
    for (uint32_t i = threadIdx.x; i < 2 * kWindows; i += blockDim.x) win_count[i] = 0;
  if (threadIdx.x == 0) {
    if (commit) {
      st->sum_ids += st->n_valid_ids;
      st->sum_unique += st->n_unique;
      st->sum_new += st->n_insert;
    }
    st->n_unique = 0; st->n_insert = 0; st->n_long = 0; st->n_parts = 0; st->n_folds = 0; st->n_valid_ids = 0;
    st->seg_cursor = 0; st->n_multi = 0; st->call_bad_offsets = 0;
  }
}
__global__ void finish_apply_kernel(DevState* st, uint32_t* win_count, int commit) { after_previous_kernel();
  if (blockIdx.x == 0) finish_apply_body(st, win_count, commit);
}

// Expiry sweep (Section 2.1, heuristic 2): a streaming pass over the key
// store; a cell whose ID has been inactive for longer than ttl is emptied and
// its row, if it has one, goes back on the free list (one counter update per
// warp and round).
// Rows of expired entries go back on the free stack: one counter update per warp.  Every lane
// of the warp calls this.
__device__ inline void warp_free_row(const TableView& tv, bool frees_row, uint32_t row, int lane) {
  const unsigned mask = __ballot_sync(0xFFFFFFFFu, frees_row);
  if (mask == 0) return;
  unsigned long long pos = 0;
  const int leader = __ffs(mask) - 1;
  if (lane == leader)
    pos = atomicAdd(reinterpret_cast<unsigned long long*>(&tv.st->free_top), (unsigned long long)__popc(mask));
  pos = __shfl_sync(0xFFFFFFFFu, pos, leader);
  const unsigned long long at = pos + __popc(mask & ((1u << lane) - 1u));
  if (frees_row && MONO_INDEX_OK(&tv.st->error_bits, at, tv.capacity)) tv.free_rows[at] = row;
}

// Sweep of buckets [first_bkt, last_bkt) of the key store, and of the stash if `with_stash`.
// The sweep reads, per bucket, the record of its oldest stamp (4 bytes, in order) and opens only
// the buckets in which that stamp is past the expire time: an entry that has to go has a stamp at
// or above its bucket's record, so its bucket is always opened, and the outcome is that of a sweep
// over every cell.  A bucket that is opened gets an exact record again.  Nothing else touches the
// key store while this runs.
// A block lists the buckets to open in shared memory, then takes them one cell per thread, so that
// all their loads are in flight together and the four lanes of a bucket read its 64 bytes as one.
constexpr int kSweepDepth = 2;                                             // 16-byte loads of four records per thread and round
__device__ inline void expire_body(const TableView& tv, unsigned long long first_bkt, unsigned long long last_bkt,
                                   bool with_stash, long long now, uint32_t vblock, uint32_t vgrid) {
  // first_bkt and last_bkt are multiples of four
  __shared__ unsigned long long open_list[256 * kSweepDepth * 4];
  __shared__ unsigned int n_open;
  const unsigned long long stride = (unsigned long long)vgrid * blockDim.x * 4u;
  const unsigned long long rounds = (last_bkt - first_bkt + stride * kSweepDepth - 1) / (stride * kSweepDepth);  // same for every thread
  const int lane = threadIdx.x & 31;
  const long long ttl = (long long)tv.ttl;
  unsigned int n_gone = 0, n_rows = 0;
  for (unsigned long long r = 0; r < rounds; ++r) {
    if (threadIdx.x == 0) n_open = 0;
    __syncthreads();
    const unsigned long long b0 = first_bkt + r * kSweepDepth * stride + ((unsigned long long)vblock * blockDim.x + threadIdx.x) * 4u;
    uint4 rec[kSweepDepth];
#pragma unroll
    for (int k = 0; k < kSweepDepth; ++k) {
      const unsigned long long b = b0 + k * stride;
      rec[k] = make_uint4(kNoStamp, kNoStamp, kNoStamp, kNoStamp);
      if (b < last_bkt) rec[k] = *reinterpret_cast<const uint4*>(tv.oldest + b);
    }
#pragma unroll
    for (int k = 0; k < kSweepDepth; ++k) {
      const uint32_t four[4] = {rec[k].x, rec[k].y, rec[k].z, rec[k].w};
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (four[q] != kNoStamp && now - (long long)four[q] > ttl) open_list[atomicAdd(&n_open, 1u)] = b0 + k * stride + q;
    }
    __syncthreads();
    const unsigned int n_cells_open = n_open * kCellsPerBucket;
    for (unsigned int base = 0; base < n_cells_open; base += blockDim.x) {      // block-uniform
      const unsigned int idx = base + threadIdx.x;
      const bool valid = idx < n_cells_open;
      const unsigned long long b = valid ? open_list[idx / kCellsPerBucket] : 0ull;
      ulonglong2* cell = reinterpret_cast<ulonglong2*>(tv.cells + b * kCellsPerBucket + (idx % kCellsPerBucket));
      ulonglong2 v; v.x = kEmptyKey; v.y = 0ull;
      if (valid) v = *cell;
      bool frees_row = false;
      uint32_t row = 0, kept = kNoStamp;
      if (v.x != kEmptyKey) {
        const uint32_t seen = meta_time(v.y);
        if (now - (long long)seen > ttl) {
          ulonglong2 e; e.x = kEmptyKey; e.y = 0ull;
          *cell = e;
          ++n_gone;
          if (meta_resident(v.y)) { frees_row = true; row = meta_row(v.y); ++n_rows; }
        } else {
          kept = seen;
        }
      }
      // the oldest stamp that stays in the bucket: its four cells sit in four adjacent lanes
      kept = min(kept, __shfl_xor_sync(0xFFFFFFFFu, kept, 1));
      kept = min(kept, __shfl_xor_sync(0xFFFFFFFFu, kept, 2));
      if (valid && (idx % kCellsPerBucket) == 0) tv.oldest[b] = kept;
      warp_free_row(tv, frees_row, row, lane);
    }
    __syncthreads();                                       // everyone has read n_open before the next round resets it
  }
  if (with_stash) {
    for (uint32_t base = vblock * blockDim.x; base < kStashCells; base += vgrid * blockDim.x) {   // block-uniform
      const uint32_t i = base + threadIdx.x;
      bool frees_row = false;
      uint32_t row = 0;
      if (i < kStashCells) {
        const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(tv.stash + i);
        if (v.x != kEmptyKey && now - (long long)meta_time(v.y) > ttl) {
          ulonglong2 e; e.x = kEmptyKey; e.y = 0ull;
          *reinterpret_cast<ulonglong2*>(tv.stash + i) = e;
          ++n_gone;
          if (meta_resident(v.y)) { frees_row = true; row = meta_row(v.y); ++n_rows; }
        }
      }
      warp_free_row(tv, frees_row, row, lane);
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    n_gone += __shfl_down_sync(0xFFFFFFFFu, n_gone, o);
    n_rows += __shfl_down_sync(0xFFFFFFFFu, n_rows, o);
  }
  if (lane == 0 && n_gone) {
    atomicAdd(&tv.st->n_tracked, (unsigned long long)(-(long long)n_gone));
    atomicAdd(&tv.st->n_expired_total, (unsigned long long)n_gone);
    if (n_rows) atomicAdd(&tv.st->n_resident, (unsigned long long)(-(long long)n_rows));
  }
}
__global__ void __launch_bounds__(256)
expire_kernel(TableView tv, unsigned long long first_bkt, unsigned long long last_bkt, int with_stash, long long now) { after_previous_kernel();
  expire_body(tv, first_bkt, last_bkt, with_stash != 0, now, blockIdx.x, gridDim.x);
}

// A batch that was grouped beside the table's other work is taken over: the counters its
// grouping left in a block of their own become the call's counters.
__global__ void adopt_group_kernel(DevState* st, DevState* side) {
  after_previous_kernel();
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    st->n_unique = side->n_unique;
    st->n_valid_ids = side->n_valid_ids;
    st->call_bad_offsets = side->call_bad_offsets;
    if (side->error_bits) atomicOr(&st->error_bits, side->error_bits);
    side->n_unique = 0; side->n_valid_ids = 0; side->call_bad_offsets = 0; side->error_bits = 0;
  }
}

// After a sweep: if the stash has become empty, probes may skip it again.
__global__ void stash_trim_kernel(TableView tv) { after_previous_kernel();
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    unsigned hw = tv.st->stash_hw;
    while (hw > 0 && tv.stash[hw - 1].key == kEmptyKey) --hw;
    tv.st->stash_hw = hw;
  }
}

__global__ void __launch_bounds__(256)
init_table_kernel(TableView tv, unsigned long long n_cells) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  ulonglong2 e; e.x = kEmptyKey; e.y = 0ull;
  for (unsigned long long i = tid; i < n_cells; i += stride) *reinterpret_cast<ulonglong2*>(tv.cells + i) = e;
  for (unsigned long long i = tid; i < kStashCells; i += stride) *reinterpret_cast<ulonglong2*>(tv.stash + i) = e;
  for (unsigned long long i = tid; i < n_cells / kCellsPerBucket; i += stride) tv.oldest[i] = kNoStamp;
  // rows are handed out in increasing order from a fresh table
  for (unsigned long long i = tid; i < tv.capacity; i += stride) tv.free_rows[i] = (uint32_t)(tv.capacity - 1 - i);
}

__global__ void __launch_bounds__(256)
init_bset_kernel(BatchSlot* bset, unsigned long long n) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  BatchSlot e; e.key = kEmptyKey; e.a = 0; e.b = 0;
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) bset[i] = e;
}

// Rehash (Section 2.1: cuckoo hashing rehashes when an insertion runs into a cycle; here the
// caller asks for it, between batches): every entry of the old key store is inserted into a
// new, empty one that has its own size and hash seeds.
__global__ void __launch_bounds__(256)
rehash_kernel(TableView fresh, const Cell* __restrict__ old_cells, unsigned long long n_old_cells,
              const Cell* __restrict__ old_stash) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  const unsigned long long total = n_old_cells + kStashCells;
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const Cell c = i < n_old_cells ? old_cells[i] : old_stash[i - n_old_cells];
    if (c.key != kEmptyKey) cuckoo_insert(fresh, c);
  }
}

// ---- bulk import -----------------------------------------------------------

// Import runs in two kernels, like the batch path: while an insertion is carrying a displaced
// entry that key sits in no cell, so the test "is this ID tracked already?" is made for all
// entries first, while nothing moves, and the insertions follow.
constexpr uint32_t kImportSkip = 0xFFFFFFFEu;

// One thread per entry: row_word[i] = kImportSkip for an ID that is already tracked (or is the
// padding value), kNoRow otherwise.
__global__ void __launch_bounds__(256)
import_check_kernel(TableView tv, const unsigned long long* __restrict__ ids, long long n, uint32_t* __restrict__ row_word) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  const unsigned stash_hw = tv.st->stash_hw;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const unsigned long long id = ids[i];
    if (id == kEmptyKey) { row_word[i] = kImportSkip; continue; }
    unsigned long long meta = 0;
    const bool present = thread_lookup(tv, id, stash_hw, &meta);
    if (present) atomicOr(&tv.st->error_bits, 8u /* MONO_DEV_IMPORT_DUP */);
    row_word[i] = present ? kImportSkip : kNoRow;
  }
}

// One thread per entry that passed the check: claim a row for resident entries, insert.
// row_word[i] tells import_rows_kernel where the entry's values go.
__global__ void __launch_bounds__(256)
import_insert_kernel(TableView tv, const unsigned long long* __restrict__ ids, const uint32_t* __restrict__ count,
                     const long long* __restrict__ last_seen, const uint8_t* __restrict__ resident,
                     long long n, uint32_t* __restrict__ row_word) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const unsigned long long id = ids[i];
    if (row_word[i] == kImportSkip) { row_word[i] = kNoRow; continue; }
    if (tv.sketch_depth != 0 && !resident[i]) continue;     // probabilistic filter: IDs without a row have no entry
    long long seen = last_seen[i];
    if (seen < 0) seen = 0;
    if (seen > 0xFFFFFFFELL) seen = 0xFFFFFFFELL;
    // an entry without a row keeps its count, up to the threshold: at the threshold it is an ID whose
    // admission was refused for lack of a row, and the batch path retries it at its next occurrence
    uint32_t low = count[i] < tv.threshold ? count[i] : tv.threshold;
    if (resident[i]) {
      const uint32_t row = alloc_row(tv);
      if (row != kNoRow) { low = kResidentBit | row; row_word[i] = row; }
      else low = tv.threshold;
    }
    Cell item; item.key = id; item.meta = make_meta((uint32_t)seen, low);
    atomicAdd(&tv.st->n_tracked, 1ull);
    atomicAdd(&tv.st->n_inserted_total, 1ull);
    cuckoo_insert(tv, item);
  }
}

// One lane group of 8 per entry copies (or initialises) the row and accumulator.
__global__ void __launch_bounds__(256)
import_rows_kernel(TableView tv, const unsigned long long* __restrict__ ids, const float* __restrict__ w,
                   const float* __restrict__ acc, long long n, const uint32_t* __restrict__ row_word) {
  const int gl = threadIdx.x & 7;
  const long long groups = ((long long)gridDim.x * blockDim.x) >> 3;
  const uint32_t dim4 = tv.dim / 4;
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 3; i < n; i += groups) {
    const uint32_t row = row_word[i];
    if (row == kNoRow) continue;
    float4* dw = reinterpret_cast<float4*>(tv.w_row(row));
    float4* da = reinterpret_cast<float4*>(tv.acc_row(row));
    for (uint32_t c4 = gl; c4 < dim4; c4 += 8) {
      dw[c4] = w ? reinterpret_cast<const float4*>(w + i * (long long)tv.dim)[c4] : init_vec(tv, ids[i], c4);
      da[c4] = acc ? reinterpret_cast<const float4*>(acc + i * (long long)tv.dim)[c4]
                   : make_float4(tv.init_acc, tv.init_acc, tv.init_acc, tv.init_acc);
    }
  }
}

}  // namespace mono
