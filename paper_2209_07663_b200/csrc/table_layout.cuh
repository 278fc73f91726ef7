// Device-side layout of the collisionless table and the small helpers every
// kernel shares: the key cell, the two bucket hash functions (h0, h1 of the
// cuckoo scheme in Section 2.1 of the Monolith paper), the counters block and
// the row-initialisation generator.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace mono {

// ---------------------------------------------------------------------------
// Key store.  One cell = one tracked ID: 8-byte key + 8-byte metadata, moved
// and claimed as a single 16-byte word (128-bit atomicCAS / atomicExch), so a
// cuckoo displacement never exposes a half-written entry.  A bucket is four
// consecutive cells = 64 bytes, 64-byte aligned: a probe reads it with four
// 16-byte loads from adjacent lanes (one 64-byte request, two DRAM sectors).
//
// meta, high 32 bits: last_seen (time of the last mono_apply_grads that held
//                     the ID);
// meta, low 32 bits : bit 31 set   -> the ID owns row (low 30 bits); bit 30 then marks a row
//                     trained since the last mono_export_touched;
//                     bit 31 clear -> still filtered, low 31 bits = occurrences
//                     so far (< threshold unless no row was free).
// ---------------------------------------------------------------------------
struct __align__(16) Cell {
  unsigned long long key;
  unsigned long long meta;
};

constexpr unsigned long long kEmptyKey = 0xFFFFFFFFFFFFFFFFull;
constexpr uint32_t kResidentBit = 0x80000000u;
constexpr uint32_t kTouchedBit = 0x40000000u;    // set with kResidentBit only
constexpr uint32_t kRowMask = 0x3FFFFFFFu;
constexpr uint32_t kCellsPerBucket = 4;
constexpr uint32_t kStashCells = 256;      // overflow area scanned only when non-empty
constexpr uint32_t kMaxChain = 96;         // bound on one insertion's displacement chain
constexpr uint32_t kNoStamp = 0xFFFFFFFFu; // a bucket's record of its oldest stamp: nothing was put there since the sweep found it empty

// Per-unique "row word" passed from the table phases to the Adagrad phase.
constexpr uint32_t kNoRow = 0xFFFFFFFFu;
constexpr uint32_t kFreshBit = 0x80000000u;  // row admitted in this call: init instead of load

__host__ __device__ inline Cell empty_cell() { Cell c; c.key = kEmptyKey; c.meta = 0ull; return c; }
__host__ __device__ inline uint32_t meta_low(unsigned long long m) { return (uint32_t)m; }
__host__ __device__ inline uint32_t meta_time(unsigned long long m) { return (uint32_t)(m >> 32); }
__host__ __device__ inline unsigned long long make_meta(uint32_t time, uint32_t low) {
  return ((unsigned long long)time << 32) | low;
}
__host__ __device__ inline bool meta_resident(unsigned long long m) { return (meta_low(m) & kResidentBit) != 0; }
__host__ __device__ inline uint32_t meta_row(unsigned long long m) { return meta_low(m) & kRowMask; }
__host__ __device__ inline bool meta_touched(unsigned long long m) { return (meta_low(m) & (kResidentBit | kTouchedBit)) == (kResidentBit | kTouchedBit); }

// Two unrelated 64-bit finalisers (multiply / xor-shift).  Both differ from the
// mixer the workload generator uses for IDs, so structured inputs of one do not
// line up with the other.
__host__ __device__ inline unsigned long long mix_a(unsigned long long x) {
  x ^= x >> 33; x *= 0xFF51AFD7ED558CCDull;
  x ^= x >> 33; x *= 0xC4CEB9FE1A85EC53ull;
  x ^= x >> 33;
  return x;
}
__host__ __device__ inline unsigned long long mix_b(unsigned long long x) {
  x ^= x >> 27; x *= 0x3C79AC492BA7B653ull;
  x ^= x >> 33; x *= 0x1C69B3F74AC4AE35ull;
  x ^= x >> 27;
  return x;
}

// SplitMix64 output function (Steele, Lea, Flood 2014): the sketch's row hashes are
// defined through it in the ABI header, so the CPU oracle indexes the same counters.
__host__ __device__ inline unsigned long long splitmix64_mix(unsigned long long z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Counters and sticky condition bits, one block per table in device memory.
struct DevState {
  unsigned int error_bits;
  unsigned int max_chain;
  unsigned int stash_hw;                 // cells [0, stash_hw) of the stash may be occupied
  unsigned int pad0;
  long long free_top;                    // free_rows[0 .. free_top) hold unused row indices
  unsigned long long n_tracked;
  unsigned long long n_resident;
  unsigned long long n_admitted_total;
  unsigned long long n_expired_total;
  unsigned long long n_inserted_total;
  unsigned long long n_rows_refused;
  unsigned long long n_keys_dropped;
  unsigned long long n_evictions_total;
  unsigned long long sum_ids;
  unsigned long long sum_unique;
  unsigned long long sum_unique_resident;
  unsigned long long sum_new;
  unsigned long long sum_single_resident;
  // per-call work counters, reset at the end of every mono_apply_grads
  unsigned int n_unique;
  unsigned int n_insert;
  unsigned int n_long;                   // distinct IDs whose segment is split into parts
  unsigned int n_parts;
  unsigned int n_folds;                  // groups of kFoldWidth parts that are added up before the final combine
  unsigned int call_bad_offsets;         // this call's offsets were malformed: occurrences are checked one by one
  unsigned int n_valid_ids;
  unsigned int seg_cursor;               // entries of bag_of_sorted[] handed out so far
  unsigned int n_multi;                  // distinct IDs that occur more than once in the batch
  unsigned int pad1;
  // export / audit scratch
  unsigned long long export_n;
};

// Checked build (-DMONO_DEBUG): every index the library computes for itself -- a segment
// position, a place in one of the per-call lists, a slot of the per-call set, a position of
// the free-row stack -- is tested against the size of its array before it is used; one that
// falls outside sets the sticky MONO_DEV_INTERNAL bit and the access is skipped.  The release
// build compiles the tests away.  (Indices that come from the caller, the bag offsets, are
// checked in every build.)
#ifdef MONO_DEBUG
#define MONO_INDEX_OK(error_bits, i, n) \
  ((unsigned long long)(i) < (unsigned long long)(n) ? true : (atomicOr((error_bits), 16u /* MONO_DEV_INTERNAL */), false))
#else
#define MONO_INDEX_OK(error_bits, i, n) true
#endif

// First statement of every kernel of the hot path.  These kernels are launched with programmatic
// stream serialisation, which lets the launch of a kernel be prepared while the kernel before it
// on the stream is still running; the kernel waits here until that one has completed and its
// writes are visible, and reads or writes nothing before.  Launched in the ordinary way this is
// a no-op.  (No kernel releases its successor early: with the successor's blocks placed beside a
// kernel's last wave, and idle there, the largest configuration measured 0.5 % slower than with
// ordinary launches; with the wait alone it is 1.2 % faster, and 6-9 % on the configurations
// whose kernels are short.)
__device__ __forceinline__ void after_previous_kernel() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Everything a kernel needs to know about a table; passed by value.
struct TableView {
  Cell* cells;                 // [n_buckets * 4]
  Cell* stash;                 // [kStashCells]
  uint32_t* oldest;            // [n_buckets]: no entry of the bucket was last seen before this time (kNoStamp:
                               // none can be there); what the expiry sweep reads instead of the cells
  float* rows;                 // [capacity][2][dim]: weights then accumulator
  uint32_t* free_rows;         // [capacity]
  DevState* st;
  unsigned long long bucket_mask;   // n_buckets - 1
  unsigned long long seed0, seed1;  // hash seeds
  unsigned long long capacity;
  uint32_t dim;
  uint32_t threshold;          // effective, >= 1
  uint32_t ttl;
  float lr, eps, init_acc, init_scale;
  uint32_t init_key0, init_key1;    // Philox key = table seed
  // probabilistic admission filter (count-min sketch); sketch_depth 0 = exact counters
  unsigned int* sketch;             // [sketch_depth][sketch_mask + 1]
  unsigned long long sketch_mask;
  unsigned long long sketch_seed;
  uint32_t sketch_depth;

  // h0 / h1: the low bits pick the bucket, the top two bits the cell of that bucket an
  // insertion tries first, so a look-up that reads that one cell first usually needs no more
  __device__ inline unsigned long long hash0(unsigned long long id) const { return mix_a(id ^ seed0); }
  __device__ inline unsigned long long hash1(unsigned long long id) const { return mix_b(id ^ seed1); }
  __device__ inline unsigned long long bucket0(unsigned long long id) const { return hash0(id) & bucket_mask; }
  __device__ inline unsigned long long bucket1(unsigned long long id) const { return hash1(id) & bucket_mask; }
  // counter of sketch row r that `id` maps to
  __device__ inline unsigned int* sketch_counter(uint32_t r, unsigned long long id) const {
    const unsigned long long i = splitmix64_mix(id ^ (sketch_seed + (unsigned long long)(r + 1) * 0x9E3779B97F4A7C15ull)) & sketch_mask;
    return sketch + (size_t)r * (sketch_mask + 1) + i;
  }
  // count-min estimate of the occurrences of `id`: the smallest of its counters
  __device__ inline unsigned int sketch_estimate(unsigned long long id) const {
    unsigned int est = 0xFFFFFFFFu;
    for (uint32_t r = 0; r < sketch_depth; ++r) {
      const unsigned int c = *reinterpret_cast<const volatile unsigned int*>(sketch_counter(r, id));
      est = c < est ? c : est;
    }
    return est;
  }
  __device__ inline float* w_row(uint32_t row) const { return rows + (size_t)row * 2u * dim; }
  __device__ inline float* acc_row(uint32_t row) const { return rows + (size_t)row * 2u * dim + dim; }
};

// ---------------------------------------------------------------------------
// Row initialisation: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) on the
// counter (id low, id high, column block, 0), keyed by the table seed.  One
// call yields the four columns of one 16-byte vector.
// ---------------------------------------------------------------------------
__device__ inline uint4 philox4x32_10(uint4 ctr, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, ctr.x), lo0 = 0xD2511F53u * ctr.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, ctr.z), lo1 = 0xCD9E8D57u * ctr.z;
    ctr = make_uint4(hi1 ^ ctr.y ^ k0, lo1, hi0 ^ ctr.w ^ k1, lo0);
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return ctr;
}

__device__ inline float unit_from_bits(uint32_t r) {
  // top 24 bits -> multiple of 2^-23 in [-1, 1); exact in fp32
  return __fsub_rn(__fmul_rn((float)(r >> 8), 1.0f / 8388608.0f), 1.0f);
}

__device__ inline float4 init_vec(const TableView& tv, unsigned long long id, uint32_t col4) {
  if (tv.init_scale == 0.0f) return make_float4(0.f, 0.f, 0.f, 0.f);
  const uint4 r = philox4x32_10(make_uint4((uint32_t)id, (uint32_t)(id >> 32), col4, 0u),
                                tv.init_key0, tv.init_key1);
  return make_float4(__fmul_rn(unit_from_bits(r.x), tv.init_scale), __fmul_rn(unit_from_bits(r.y), tv.init_scale),
                     __fmul_rn(unit_from_bits(r.z), tv.init_scale), __fmul_rn(unit_from_bits(r.w), tv.init_scale));
}

// Cell load that the compiler may not cache in registers across the bounded
// retry loops of the insert path (two 8-byte reads: only used where a torn
// pair is harmless because a 16-byte atomic validates it afterwards).
__device__ inline Cell load_cell(const Cell* p) {
  Cell c;
  c.key = *reinterpret_cast<const volatile unsigned long long*>(&p->key);
  c.meta = *reinterpret_cast<const volatile unsigned long long*>(&p->meta);
  return c;
}
// One ordinary 16-byte load: for kernels that also write cells (no key moves while they run).
__device__ inline Cell load_cell_whole(const Cell* p) {
  const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(p);
  Cell c; c.key = v.x; c.meta = v.y; return c;
}
// The same through the read-only data path: only for kernels that write no cell.
__device__ inline Cell load_cell_ro(const Cell* p) {
  const ulonglong2 v = __ldg(reinterpret_cast<const ulonglong2*>(p));
  Cell c; c.key = v.x; c.meta = v.y; return c;
}


}  // namespace mono
