/*
 * mono.h -- C ABI of the collisionless embedding table for one NVIDIA B200.
 *
 * The table is the sparse-parameter store of Monolith (arXiv 2209.07663):
 * a key-value HashTable from 64-bit feature IDs to fp32 embedding rows that
 * never lets two IDs share a row (Section 2.1), admits an ID only after it has
 * occurred a threshold number of times (Section 2.1, filtering heuristic 1),
 * stamps every ID with its last access so that inactive IDs can be expired
 * (heuristic 2), and serves the sparse half of a training step (Section 2.2:
 * pull the parameters, forward, backward, push the updated parameters back).
 * Sum pooling per bag, gradient de-duplication and the Adagrad row update are
 * not described in the paper; their definitions are stated at each call.
 *
 * Conventions
 *  - Every call returns an int: MONO_OK or a negative MONO_ERR_* code that the
 *    host detected before any work was enqueued.  No exception crosses the ABI.
 *  - Unless a parameter is marked HOST, data pointers are DEVICE pointers owned
 *    by the caller; the library reads or writes them only through work enqueued
 *    by the call and never frees or keeps them.
 *  - All work of a table is enqueued on the CUDA stream given at creation.  The
 *    hot calls (mono_lookup_pool, mono_apply_grads, mono_expire) return without
 *    synchronising.  Calls on one table must not overlap on the GPU: issue them
 *    from one thread, on that stream.  (A call may run some of its kernels on
 *    streams of the table's own; they start after everything issued on the
 *    table's stream so far, and whatever is issued on it next waits for them,
 *    so a caller sees the order of one stream.)
 *  - Conditions that only the device can see (no free row, key store full,
 *    malformed offsets) never trap or hang: every device loop is bounded, the
 *    condition sets a sticky bit and a counter, and mono_status reports them.
 *  - A "bag" is one (example, feature slot) pair.  Bags are given CSR style:
 *    bag b owns ids[slot_offsets[b] .. slot_offsets[b+1]).
 *  - IDs are arbitrary 64-bit patterns except MONO_RESERVED_ID, which is
 *    padding: it pools as zero and is neither counted nor inserted.
 *  - Time is the integer `now` the caller passes (a step counter, seconds,
 *    ...).  It must not decrease and must lie in [0, MONO_MAX_NOW].
 */
#ifndef MONO_H_
#define MONO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MONO_RESERVED_ID 0xFFFFFFFFFFFFFFFFull
#define MONO_MAX_NOW     0xFFFFFFFEll
#define MONO_MAX_DIM     1024u
#define MONO_MAX_CAPACITY (1ull << 30)

enum {
  MONO_OK = 0,
  MONO_ERR_ARG = -1,    /* null or misaligned pointer, size out of range, bad option */
  MONO_ERR_TIME = -2,   /* `now` decreased or is outside [0, MONO_MAX_NOW] */
  MONO_ERR_CUDA = -3,   /* a CUDA runtime call failed; see mono_last_cuda_error */
  MONO_ERR_NOMEM = -4,  /* device allocation failed */
  MONO_ERR_SIZE = -5,   /* caller buffer too small (mono_export) */
  MONO_ERR_LIMIT = -6   /* the call is larger than the fixed maximum of an entry point that
                           never allocates (mono_lookup_pool_noalloc) */
};

/* Sticky device-side condition bits reported in mono_status_t.error_bits. */
enum {
  MONO_DEV_ROWS_FULL = 1u,    /* an ID reached the threshold but no free row was left;
                                 it stays tracked without a row and is retried later */
  MONO_DEV_KEYS_FULL = 2u,    /* an insertion found no cell after the bounded eviction
                                 chain and the stash was full: one tracked key was lost */
  MONO_DEV_BAD_OFFSETS = 4u,  /* a bag with slot_offsets[b] < 0, slot_offsets[b+1] < slot_offsets[b]
                                 or slot_offsets[b+1] > n_ids: that bag was treated as empty, by
                                 the lookup (zeros) and by the push (its IDs are neither counted,
                                 stamped nor trained).  After a decrease in the offsets two
                                 well-formed bags can overlap; the lookup then pools the shared
                                 IDs in both, the push counts each of them once, for one of the
                                 two bags */
  MONO_DEV_IMPORT_DUP = 8u,   /* mono_import met an ID that was already tracked; skipped */
  MONO_DEV_INTERNAL = 16u     /* only in the checked build (-DMONO_DEBUG): an index the library computed
                                 for itself fell outside its array; the access was skipped */
};

enum { MONO_OPT_ADAGRAD = 1 };

typedef struct mono_table mono_table; /* opaque, owned by the library */

/*
 * Options of mono_table_create.  Zero-initialise, then set what is needed.
 *
 * Row initialisation (the paper does not give one): column c of a newly
 * admitted ID starts at  (u * 2^-23 - 1) * init_scale  with u the top 24 bits
 * of word (c mod 4) of Philox4x32-10 (Salmon et al., SC'11) keyed by
 * (seed low 32 bits, seed high 32 bits) on the counter
 * (id low 32 bits, id high 32 bits, c / 4, 0).  It depends on nothing but
 * (seed, id, c), so it is the same whatever the insertion order or row index.
 */
typedef struct {
  int32_t  kind;          /* MONO_OPT_ADAGRAD (0 selects it too) */
  float    lr;            /* Adagrad learning rate */
  float    eps;           /* added to sqrt(acc), outside the square root */
  float    init_acc;      /* initial value of every accumulator element */
  float    init_scale;    /* rows start uniform in [-init_scale, init_scale); 0 => zeros */
  uint64_t seed;          /* seeds row initialisation and the table's hash functions */
  uint64_t key_cells;     /* cells of the key store = how many IDs can be tracked (with or
                             without a row) at load 1.  Power of two, >= 64.
                             0 => 4 * capacity rounded up to a power of two. */
  uint64_t max_ids;       /* scratch is sized for this many IDs per call at creation;
                             larger calls grow it (an allocation, so not inside a timed
                             loop).  0 => grown on first use. */
  uint64_t max_bags;      /* same, for bags per call */
  uint64_t sketch_width;  /* counters per sketch row, power of two (see sketch_depth) */
  uint32_t sketch_depth;  /* 0: exact per-ID counters (default).  1..8: probabilistic filter, a
                             count-min sketch of sketch_depth rows; see below */
  uint32_t pad_;
} mono_opt;

/*
 * Probabilistic admission filter (Section 2.1, heuristic 1: besides filtering by occurrence
 * count the paper uses a probabilistic filter to save more memory; it does not say which).
 * With sketch_depth > 0 an ID without a row has no entry in the key store at all.  Instead,
 * per batch: (a) every distinct ID without a row adds its multiplicity to one 32-bit counter
 * in each sketch row -- row r (0-based) uses counter
 *     SplitMix64(id XOR (seed + (r + 1) * 0x9E3779B97F4A7C15)) AND (sketch_width - 1),
 * SplitMix64 being the output function of Steele, Lea and Flood's generator;  (b) once all
 * additions of the batch are done, an ID whose smallest counter has reached filter_threshold
 * is given a row and enters the key store.  Collisions can only raise an estimate, so the
 * sketch never rejects an ID the exact filter would admit, but it may admit one early.
 * mono_expire clears the whole sketch when more than ttl has passed since it was last cleared
 * (time 0 at creation), and expires rows as usual.  mono_probe reports, for an ID without an
 * entry, count = min(estimate, filter_threshold).  Counters must not reach 2^32 between two
 * clearings.  mono_import skips entries that are not resident.
 */

typedef struct {
  uint32_t error_bits;          /* OR of MONO_DEV_* since creation */
  uint32_t dim;
  uint64_t capacity;            /* rows */
  uint64_t key_cells;
  uint64_t n_tracked;           /* IDs in the key store (with or without a row) */
  uint64_t n_resident;          /* IDs that own a row */
  uint64_t n_admitted_total;    /* rows handed out since creation */
  uint64_t n_expired_total;     /* IDs removed by mono_expire */
  uint64_t n_inserted_total;    /* IDs that entered the key store */
  uint64_t n_rows_refused;      /* admissions refused for lack of a row */
  uint64_t n_keys_dropped;      /* keys lost to MONO_DEV_KEYS_FULL */
  uint64_t n_evictions_total;   /* cuckoo displacements performed */
  uint32_t max_chain;           /* longest eviction chain seen */
  uint32_t stash_used;          /* occupied stash cells (high-water mark index) */
  /* totals over all mono_apply_grads calls (for traffic accounting) */
  uint64_t sum_ids;             /* non-padding ID occurrences */
  uint64_t sum_unique;          /* distinct IDs per call, summed */
  uint64_t sum_unique_resident; /* distinct IDs that had (or got) a row, summed */
  uint64_t sum_new;             /* distinct IDs that were new to the key store, summed */
  uint64_t sum_single_resident; /* distinct IDs with a row that occurred once in their batch, summed */
  uint64_t scratch_reallocs;    /* times a call had to grow the scratch (cudaMalloc + synchronise inside
                                   the call); stays 0 when max_ids / max_bags or mono_reserve were large enough */
} mono_status_t;

typedef struct {
  uint64_t occupied_cells;      /* occupied key cells incl. stash */
  uint64_t misplaced;           /* keys found in a bucket that is neither h0(key) nor h1(key) */
  uint64_t duplicate_keys;      /* keys present in more than one cell */
  uint64_t resident_cells;
  uint64_t bad_rows;            /* row index >= capacity */
  uint64_t shared_rows;         /* rows owned by two cells, or owned and also on the free list */
  uint64_t free_rows;
  uint64_t unaccounted_rows;    /* rows neither owned nor free */
  uint32_t ok;                  /* 1 iff all of the above are consistent with the counters */
  uint32_t behind_records;      /* entries last seen before the time their bucket's sweep record holds
                                   (saturating); the expiry sweep would not find them */
} mono_audit_t;

/*
 * Create an empty table (Section 2.1: one HashTable per sparse feature group).
 *  out               HOST, receives the handle
 *  capacity          number of embedding rows, 1 .. MONO_MAX_CAPACITY
 *  dim               fp32 columns per row, multiple of 4, 4 .. MONO_MAX_DIM
 *  filter_threshold  an ID gets a row once its occurrences reach this (0 acts as 1);
 *                    a per-model hyperparameter in the paper, here set per table
 *  ttl               an ID unseen for MORE than ttl time units is removed by
 *                    mono_expire; 0 disables expiry (the paper tunes it per table)
 *  opt               HOST, may be NULL for defaults (lr 0.05, eps 1e-8, zeros)
 *  cuda_stream       a cudaStream_t (NULL = the default stream) on the current device
 * Allocates capacity * dim * 8 bytes of rows+accumulators, key_cells * 16 bytes
 * of keys, key_cells bytes of sweep records (below, mono_expire), capacity * 4
 * bytes of free-row bookkeeping and the scratch.
 */
int mono_table_create(mono_table** out, uint64_t capacity, uint32_t dim,
                      uint32_t filter_threshold, uint32_t ttl, const mono_opt* opt,
                      void* cuda_stream);

/* Synchronise the stream and free everything the table owns. */
int mono_table_destroy(mono_table* t);

/* Grow the scratch so that calls with up to max_ids IDs and max_bags bags
 * allocate nothing.  Synchronises if it has to reallocate. */
int mono_reserve(mono_table* t, int64_t max_ids, int64_t max_bags);

/*
 * Forward (the parameter pull of a training step, Section 2.2; the HashTable
 * look-up operation of Section 2.1): out[b, :] = sum over the IDs of bag b, in order, of the row of
 * each ID that owns one; an ID without a row (unknown, below the threshold,
 * expired) contributes zero; an empty bag gives zeros.  Read-only: counts and
 * last-access times do not change.
 *  ids           uint64 [n_ids], 8-byte aligned
 *  slot_offsets  int64 [n_bags + 1], non-decreasing, slot_offsets[0] >= 0,
 *                slot_offsets[n_bags] <= n_ids
 *  out           fp32 [n_bags, dim] row-major, 16-byte aligned, overwritten
 */
int mono_lookup_pool(mono_table* t, const uint64_t* ids, int64_t n_ids,
                     const int64_t* slot_offsets, int64_t n_bags, float* out);

/*
 * Backward + update (the parameter push of a training step, Section 2.2; the
 * HashTable update operation with the occurrence filter and the access stamp of Section 2.1).  For the
 * batch as a whole:
 *  1. every distinct ID u gets  count(u) += multiplicity of u in ids  (saturating
 *     at the threshold; the counter only gates admission) and last_seen(u) = now;
 *     IDs met for the first time enter the key store (cuckoo insertion);
 *  2. an ID whose count has reached the threshold and that has no row is given a
 *     free row, initialised as described at mono_opt;
 *  3. every distinct ID that owns a row takes ONE Adagrad step with
 *     G = sum over its occurrences j of grad_pooled[bag(j), :]  (summed in fp64,
 *     rounded once to fp32):   acc += G*G;   w -= lr * G / (sqrt(acc) + eps).
 *     The whole batch's G applies even when the row was admitted in this call.
 *     Gradients of IDs without a row are dropped.
 * Counts, times, admissions and the set of rows do not depend on the order of IDs or
 * bags.  The fp64 sum G is taken in an order that can differ from run to run (it follows
 * the order in which thread blocks reach an ID), so two runs on the same input can differ
 * in the last bit of an updated element: the results are order-independent to within one
 * fp32 rounding of G, not bitwise reproducible.
 *  grad_pooled   fp32 [n_bags, dim], 16-byte aligned
 *  now           time of this batch; MONO_ERR_TIME if it decreased
 */
int mono_apply_grads(mono_table* t, const uint64_t* ids, int64_t n_ids,
                     const int64_t* slot_offsets, int64_t n_bags,
                     const float* grad_pooled, int64_t now);

/*
 * Expiry sweep (Section 2.1, heuristic 2): remove every tracked ID, with or
 * without a row, for which  now - last_seen > ttl; free its row and forget its
 * count.  Expiry takes effect only here; a stale ID that re-occurs before a
 * sweep is refreshed.  No-op when ttl == 0.
 * The sweep does not read every cell: beside each 4-cell bucket the table keeps a
 * time that is not later than the last_seen of any entry in it, reads those (4
 * bytes per bucket) and opens only the buckets where that time is past the ttl.
 * The set of IDs removed is that of a sweep over all cells.
 */
int mono_expire(mono_table* t, int64_t now);

/*
 * Optional hint for a training loop that knows its batch before the pull (Section 2.2: a step
 * pulls the parameters of a batch and later pushes updates for the same batch).  Announces
 * the batch that the NEXT mono_lookup_pool and mono_apply_grads on this table will be given
 * -- the same device pointers and sizes, contents unchanged until the push -- and does the
 * work both calls share ahead of them: the occurrences are grouped by ID, and every distinct
 * ID is looked up in the key store once.  mono_lookup_pool called with exactly these `ids`,
 * `n_ids`, `slot_offsets`, `n_bags` then takes the rows from that look-up instead of probing
 * the key store once per occurrence, and mono_apply_grads called with them goes straight to
 * the cells the look-up found.  Called with anything else, either call works as if nothing
 * had been announced (a push then forgets the announcement, as does a second
 * mono_prepare_push).  Any call that changes the table between the announcement and the push
 * -- mono_expire*, mono_import, mono_rehash, mono_export_touched, mono_snapshot_restore --
 * forgets it too, so results are the same with or without the hint.  The table is not
 * changed by this call.  Errors: as mono_lookup_pool; malformed offsets raise
 * MONO_DEV_BAD_OFFSETS in the status, as they would in mono_apply_grads.
 */
int mono_prepare_push(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                      int64_t n_bags);

/*
 * Optional, one step further ahead: groups the occurrences of a batch by ID -- the part of
 * mono_prepare_push that needs nothing from the table -- on an internal stream, beside whatever
 * the table's stream is doing (typically the push of the batch before).  It starts once the work
 * the table's stream holds at the time of the call is done, so `ids` and `slot_offsets` may be
 * produced on that stream; like an announced batch they must stay unchanged until the push.  A
 * later mono_prepare_push with exactly these arguments takes the grouping over and only looks the
 * distinct IDs up; with other arguments it groups its batch itself and the grouping made ahead
 * stays for a later call.  One batch can be grouped ahead at a time: a second call forgets the
 * first.  Neither the table nor a batch that was announced is touched, and results are the same
 * with or without this call.  The first call allocates a second copy of the scratch the grouping
 * fills (about 70 bytes per ID of max_ids).  Errors: as mono_prepare_push; malformed offsets show
 * in the status once the batch is taken over.
 */
int mono_group_ahead(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                     int64_t n_bags);

/*
 * Grouped calls: one call, and one kernel launch per step of the path, for several tables
 * (Section 3.1: a production model holds many embedding tables of very uneven size, most of
 * them far too small to fill a GPU on their own).  Table i gets batch i: `tables`, `ids`,
 * `n_ids`, `slot_offsets`, `n_bags`, `out` / `grad_pooled` are HOST arrays of `n_tables`
 * entries whose elements are what the single-table call takes (device pointers, sizes).  The
 * grid of every kernel is the concatenation of the grids the tables would launch one by one;
 * tables of different dims share a launch (rows wider than 128 columns get a second one).
 * The group's work runs on `group_stream`: it starts after everything issued so far on
 * `group_stream` and on the tables' own streams, and whatever is issued next on any of them
 * waits for it.  Tables created on `group_stream` itself need no such ordering and are the
 * cheapest to group.  All tables must live on the current device; the same table must not
 * appear twice; successive grouped calls that share tables[0] must use the same
 * `group_stream`.  Results are those of the n_tables single calls.  Errors: the first one met
 * while checking the arguments, before anything is enqueued; MONO_ERR_ARG for n_tables < 0
 * or a null array.
 *
 * mono_group_prepare_push announces every table's next batch, as mono_prepare_push does for
 * one table.  mono_group_apply_grads uses the announcements if every table of the group (with
 * a batch that is not empty) is given exactly the batch it was announced; otherwise it
 * forgets them all and groups and looks up the batches itself.
 */
int mono_group_prepare_push(int32_t n_tables, mono_table* const* tables, const uint64_t* const* ids,
                            const int64_t* n_ids, const int64_t* const* slot_offsets, const int64_t* n_bags,
                            void* group_stream);
int mono_group_lookup_pool(int32_t n_tables, mono_table* const* tables, const uint64_t* const* ids,
                           const int64_t* n_ids, const int64_t* const* slot_offsets, const int64_t* n_bags,
                           float* const* out, void* group_stream);
int mono_group_apply_grads(int32_t n_tables, mono_table* const* tables, const uint64_t* const* ids,
                           const int64_t* n_ids, const int64_t* const* slot_offsets, const int64_t* n_bags,
                           const float* const* grad_pooled, int64_t now, void* group_stream);

/*
 * Incremental form of mono_expire: sweeps slice `slice` of `n_slices` equal parts of the key
 * store (multiples of 16 cells; the last slice also covers the remainder and the overflow stash), so that the cost of a full sweep can
 * be spread over n_slices training steps.  Calling it for slice = 0 .. n_slices-1 with the
 * same `now` (and no other call in between) has exactly the effect of mono_expire(now).
 * 1 <= n_slices <= 65536, slice < n_slices.  With the probabilistic filter, slice 0 is the
 * one that clears the sketch when its window has passed.
 */
int mono_expire_slice(mono_table* t, int64_t now, uint32_t slice, uint32_t n_slices);

/*
 * Host-buffer forms of the two hot calls, for callers whose batches live in host memory
 * (pinned memory makes the copies asynchronous).  Same kernels as the device-pointer forms;
 * the library copies the inputs into staging buffers of its own and the pooled rows back out,
 * on two copy streams of the table's own (one per direction), so that the gradients of a step
 * come in while its pooled rows still go out and both run beside the kernels.
 *  - Neither call synchronises.  `out` holds the result, and the host input buffers may be
 *    reused, once the table's stream has passed a mono_fence issued after the calls
 *    (mono_fence, then synchronise the stream or wait for an event recorded on it).
 *  - mono_lookup_pool_host stages `ids` and `slot_offsets` on the device and treats the staged
 *    batch as announced (see mono_prepare_push).  mono_apply_grads_host given the same host
 *    pointers and sizes as the mono_lookup_pool_host call directly before it reuses that copy
 *    and that announcement -- the contents must not have changed in between; given anything
 *    else it copies its own.
 *  - The two bag-by-dim staging matrices are allocated by the first host-buffer call.
 * All pointers HOST.
 */
int mono_lookup_pool_host(mono_table* t, const uint64_t* ids, int64_t n_ids,
                          const int64_t* slot_offsets, int64_t n_bags, float* out);
int mono_apply_grads_host(mono_table* t, const uint64_t* ids, int64_t n_ids,
                          const int64_t* slot_offsets, int64_t n_bags,
                          const float* grad_pooled, int64_t now);

/*
 * mono_lookup_pool for callers that must not allocate device memory.  (The
 * paper has no counterpart; this is a deployment variant of the forward call.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a
 * serving loop whose memory budget was fixed at start-up, under an allocator
 * that owns the whole device, or in a process that has handed every spare
 * byte to other tenants.  mono_lookup_pool keeps its per-ID scratch (the row
 * index of every ID of the batch) in a buffer it grows with cudaMalloc when a
 * larger batch arrives; this entry point keeps the same scratch in a fixed
 * array that is part of the library image instead, so it never calls
 * cudaMalloc, cudaFree or anything else that allocates.
 *
 *  - Same arguments, same result and same error codes as mono_lookup_pool.
 *  - n_ids may be at most MONO_NOALLOC_MAX_IDS; a larger batch is refused with
 *    MONO_ERR_LIMIT before anything is enqueued (split it into several calls).
 *  - The array (MONO_NOALLOC_MAX_IDS * 4 bytes = 4 MiB) is reserved on every
 *    GPU that loads the library, from load until the process exits.
 *  - The first call on a device looks up the array's device address once
 *    (no allocation, but a runtime query): make that first call before any
 *    CUDA stream capture begins on that device.  The address is remembered for
 *    the life of the process; a cudaDeviceReset in between invalidates it.
 *  - The table's device must be the current device (MONO_ERR_ARG otherwise:
 *    another device's copy of the array would be the wrong memory).
 *  - With mono_timing_enable switched on, the call creates CUDA events for its
 *    two launches like every other hot call; leave timing off where even that
 *    is unwelcome.
 *  - All tables and all calls on a device share the one array, and it keeps
 *    whatever the previous call left in it.  Nothing in it needs clearing --
 *    each call overwrites the entries it reads -- but two calls that are in
 *    flight on the GPU at the same time (different streams, different tables)
 *    would overwrite each other's entries: serialise them.
 */
#define MONO_NOALLOC_MAX_IDS (1u << 20)
int mono_lookup_pool_noalloc(mono_table* t, const uint64_t* ids, int64_t n_ids,
                             const int64_t* slot_offsets, int64_t n_bags, float* out);

/*
 * Order point for the table's internal streams (the paper has no counterpart).  A hot call may
 * leave work running on streams of the table's own (the sweep of mono_expire*, the grouping of
 * mono_group_ahead);
 * the next call on the table waits for it by itself.  mono_fence makes the table's stream wait
 * for all of it now, without synchronising the host, so that an event the caller records on
 * the table's stream afterwards marks the end of everything issued so far.
 */
int mono_fence(mono_table* t);

/*
 * Device-resident snapshot (Section 2.3: the parameter servers snapshot their state so that
 * training can go back to it; here the copy stays in device memory, for callers that want to
 * return to a state quickly -- benchmarks that repeat a timed region from the same state,
 * what-if runs).  mono_snapshot_save copies the key store, the rows and accumulators, the
 * free-row list, the counters and the sketch into a second set of buffers owned by the table
 * (allocated on the first save: as much memory again as the table itself; MONO_ERR_NOMEM if
 * that does not fit) and remembers the table's clock.  mono_snapshot_restore copies them back
 * and resets the clock, so calls may again use any `now` >= the saved one; a batch announced
 * with mono_prepare_push is forgotten.  Both are asynchronous device-to-device copies on the
 * table's stream.  A table that was rehashed since the save cannot be restored
 * (MONO_ERR_ARG), nor one that has no snapshot.  mono_snapshot_drop frees the copy.
 */
int mono_snapshot_save(mono_table* t);
int mono_snapshot_restore(mono_table* t);
int mono_snapshot_drop(mono_table* t);

/* ---- inspection and fixtures: not on the hot path, all synchronise ---- */

/* Counters and sticky error bits.  host_out HOST. */
int mono_status(mono_table* t, mono_status_t* host_out);

/* Clear the sticky error bits (counters are kept). */
int mono_clear_errors(mono_table* t);

/*
 * State of n IDs: resident[i] 1/0, count[i] (0 if untracked; equals the
 * threshold once resident), last_seen[i] (-1 if untracked).  Any output
 * pointer may be NULL.
 */
int mono_probe(mono_table* t, const uint64_t* ids, int64_t n, uint8_t* resident,
               uint32_t* count, int64_t* last_seen);

/* Rows and accumulators of n IDs, fp32 [n, dim] each; zeros where the ID has
 * no row.  Either output may be NULL. */
int mono_read_rows(mono_table* t, const uint64_t* ids, int64_t n, float* w, float* acc);

/*
 * Dump every tracked ID (any order) into caller buffers of max_n entries:
 * ids, count, last_seen, resident, and fp32 [max_n, dim] w / acc (zeros for IDs
 * without a row; w and acc may be NULL).  n_out HOST receives the number
 * written.  MONO_ERR_SIZE (and *n_out = needed) if max_n is too small.
 * This is the table's snapshot (Section 2.3) in its simplest form.
 */
int mono_export(mono_table* t, uint64_t* ids, uint32_t* count, int64_t* last_seen,
                uint8_t* resident, float* w, float* acc, int64_t max_n, int64_t* n_out);

/*
 * Rebuild the key store with new hash functions and, optionally, a new size (Section 2.1:
 * cuckoo hashing rehashes when an insertion runs into a cycle; on a fixed-size device table
 * that moment is reported as MONO_DEV_KEYS_FULL or a filling stash, and the caller rehashes
 * between batches).  Every tracked ID keeps its count, last-access time and row; only its
 * position changes.  new_key_cells: power of two >= 64, 0 keeps the size.  new_seed seeds the
 * two bucket hash functions (row initialisation keeps the seed given at creation).
 * Allocates the new store before freeing the old one; synchronises.  Keys that were dropped
 * earlier are not brought back; if the new store is too small the usual overflow bits are set.
 */
int mono_rehash(mono_table* t, uint64_t new_key_cells, uint64_t new_seed);

/*
 * Incremental export for parameter synchronisation (Section 2.2.3: the training side keeps
 * the set of touched keys -- IDs whose embeddings were trained since the last
 * synchronisation -- and pushes only those rows to the serving side).  Every ID whose row
 * mono_apply_grads has updated since the previous call is written to ids / w (fp32
 * [max_n, dim], any order) and leaves the set.  n_out HOST receives how many touched IDs
 * there were.  If that is more than max_n, the first max_n found are exported, the rest stay
 * in the set for the next call, and the return code is MONO_ERR_SIZE.  An ID that expired
 * before the call is not exported.  One pass over the key store; synchronises.
 */
int mono_export_touched(mono_table* t, uint64_t* ids, float* w, int64_t max_n, int64_t* n_out);

/*
 * Insert n entries given as (id, count, last_seen, resident[, w, acc]).  An ID
 * that is already tracked is skipped and MONO_DEV_IMPORT_DUP is set.  The IDs of
 * one call must be distinct: this is not checked, and a repeated ID ends up in
 * two cells (mono_audit reports it as a duplicate key).  resident[i] != 0 claims a row; its values come
 * from w/acc, or from the initialisation rule (and init_acc) when w or acc is
 * NULL.  count is clamped to the threshold; an entry without a row whose count
 * is at the threshold (an admission that was refused for lack of a row) is admitted
 * at its next occurrence.  Restores a snapshot, or pre-fills a table to a chosen load.
 */
int mono_import(mono_table* t, const uint64_t* ids, const uint32_t* count,
                const int64_t* last_seen, const uint8_t* resident, const float* w,
                const float* acc, int64_t n);

/*
 * Structural audit of the cuckoo table (Section 2.1: an element lives in
 * exactly one of its two candidate positions): every key sits in one of its
 * two buckets or the stash, no key twice, row indices distinct and disjoint
 * from the free rows, rows owned + free = capacity.  host_out HOST.
 */
int mono_audit(mono_table* t, mono_audit_t* host_out);

/*
 * Launch accounting for benchmarks (the paper has no counterpart).  Every
 * kernel the hot calls launch is counted per kernel.  With timing enabled,
 * each launch is also bracketed by two CUDA events on the table's stream and
 * mono_timing_read (which synchronises) adds up the elapsed device time per
 * kernel; the events cost a few microseconds per launch, so leave timing off
 * when measuring whole-step throughput.  ms is 0 for launches made with timing
 * off.  reset != 0 zeroes the counts and times after reading.  host_out HOST.
 */
#define MONO_MAX_KERNELS 24
typedef struct {
  char     name[32];
  uint64_t launches;
  double   ms;
} mono_kernel_time_t;
typedef struct {
  uint32_t n_kernels;
  uint32_t pad_;
  uint64_t launches_total;
  mono_kernel_time_t kernel[MONO_MAX_KERNELS];
} mono_timing_t;
int mono_timing_enable(mono_table* t, int on);
int mono_timing_read(mono_table* t, mono_timing_t* host_out, int reset);

/* Text of the last CUDA error seen by this table (HOST string, library-owned). */
const char* mono_last_cuda_error(mono_table* t);

/* Name of a MONO_* return code. */
const char* mono_error_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* MONO_H_ */
