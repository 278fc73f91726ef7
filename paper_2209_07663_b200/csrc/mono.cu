// Host side of the C ABI declared in include/mono.h: argument checks, memory
// ownership, and the launch sequence of each call.  Every step of the hot path
// runs in the kernels included below; nothing here computes on the host.
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include <cuda_runtime.h>

#include "../../include/mono.h"
#include "kernels_adagrad.cuh"
#include "kernels_dedup.cuh"
#include "kernels_forward.cuh"
#include "kernels_inspect.cuh"
#include "kernels_table.cuh"
#include "table_layout.cuh"

using namespace mono;

// Scratch of mono_lookup_pool_noalloc: part of the library image, so the entry
// point never allocates.  In host code this name is only a handle for
// cudaGetSymbolAddress; kernels get the device address that call returns.
static __device__ __align__(256) uint32_t g_noalloc_occ_row[MONO_NOALLOC_MAX_IDS];

enum KernelId {
  K_PROBE, K_GATHER, K_FILL_BAG, K_DEDUP, K_UPDATE, K_SKETCH, K_INSERT, K_EXPAND, K_ORDER, K_FILE, K_SINGLES, K_REDUCE, K_FOLD, K_COMBINE, K_FINISH, K_EXPIRE,
  K_STASH_TRIM, K_COUNT
};
static const char* const kKernelNames[K_COUNT] = {
  "probe_rows", "gather_pool", "fill_occ_bag", "dedup_tile", "table_update", "sketch_add", "table_insert", "expand_parts", "order_parts",
  "file_segments", "update_singletons", "reduce_adagrad", "fold_partials", "combine_adagrad",
  "finish_apply", "expire", "stash_trim"
};

struct mono_table {
  // per-kernel launch counts, and (when timing is on) CUDA-event durations
  uint64_t launches[K_COUNT] = {};
  double kernel_ms[K_COUNT] = {};
  bool timing = false;
  std::vector<cudaEvent_t> spare_events;
  std::vector<std::pair<int, std::pair<cudaEvent_t, cudaEvent_t>>> pending;
  cudaEvent_t open_event = nullptr;
  TableView tv{};
  Work wk{};
  cudaStream_t stream = nullptr;
  // Two internal streams, ordered against `stream` with events only: one runs the
  // ID-only part of a push that mono_prepare_push announced, the other the sweep.
  cudaStream_t prep_stream = nullptr, sweep_stream = nullptr;
  // A third one runs the small kernels that serve only the few hottest IDs of a push beside
  // the large ones (see launch_apply).
  cudaStream_t aux_stream = nullptr;
  cudaEvent_t ev_parts = nullptr, ev_reduced = nullptr, ev_aux = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_prepared = nullptr, ev_keys = nullptr, ev_swept = nullptr;
  cudaEvent_t ev_group = nullptr;  // grouped calls: the group's start (first table's), this table's end
  bool sweep_pending = false;     // the sweep stream has work `stream` has not waited for yet
  bool keys_idle = false;         // nothing launched on `stream` after ev_keys touches the key store
  struct { const void* ids; int64_t n_ids; const void* off; int64_t n_bags; bool valid; } prep = {nullptr, 0, nullptr, 0, false};
  uint32_t* occ_row = nullptr;    // scratch of the lookup: row of every occurrence
  int sm_count = 148;
  uint64_t key_cells = 0;
  int64_t last_now = -1;
  int64_t sketch_epoch = 0;       // time the sketch was last cleared
  int64_t max_ids = 0, max_bags = 0;
  // device staging for the host-buffer calls
  unsigned long long* stage_ids = nullptr;
  long long* stage_off = nullptr;
  float* stage_vec = nullptr;
  std::string last_err;
};

namespace {

#define CUDA_TRY(t, expr)                                                         \
  do {                                                                            \
    cudaError_t e__ = (expr);                                                     \
    if (e__ != cudaSuccess) {                                                     \
      (t)->last_err = std::string(#expr) + ": " + cudaGetErrorString(e__);        \
      return e__ == cudaErrorMemoryAllocation ? MONO_ERR_NOMEM : MONO_ERR_CUDA;   \
    }                                                                             \
  } while (0)

inline bool is_pow2(uint64_t x) { return x && !(x & (x - 1)); }
inline uint64_t next_pow2(uint64_t x) { uint64_t p = 1; while (p < x) p <<= 1; return p; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

template <typename T>
int dev_alloc(mono_table* t, T** p, size_t n) {
  *p = nullptr;
  CUDA_TRY(t, cudaMalloc(reinterpret_cast<void**>(p), (n ? n : 1) * sizeof(T)));
  return MONO_OK;
}

template <typename T>
void dev_free(T*& p) { if (p) { cudaFree(p); p = nullptr; } }

void free_scratch(mono_table* t) {
  Work& w = t->wk;
  dev_free(w.bset); dev_free(w.occ_slot); dev_free(w.occ_rank); dev_free(w.occ_bag); dev_free(w.bag_of_sorted);
  dev_free(w.uid); dev_free(w.uslot); dev_free(w.uocc); dev_free(w.useg); dev_free(w.ulen); dev_free(w.urow);
  dev_free(w.multi_list); dev_free(w.ins_list); dev_free(w.long_u); dev_free(w.long_part0); dev_free(w.part_u); dev_free(w.part_order); dev_free(w.win_count); dev_free(w.partials); dev_free(w.fold_li); dev_free(w.fold_idx);
  dev_free(t->stage_ids); dev_free(t->stage_off); dev_free(t->stage_vec); dev_free(t->occ_row);
  t->max_ids = t->max_bags = 0;
}

int grid_for(const mono_table* t, int per_sm) { return t->sm_count * per_sm; }

cudaEvent_t take_event(mono_table* t) {
  if (!t->spare_events.empty()) { cudaEvent_t e = t->spare_events.back(); t->spare_events.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}
void launch_begin(mono_table* t, int kid, cudaStream_t s) {
  ++t->launches[kid];
  if (t->timing) { t->open_event = take_event(t); cudaEventRecord(t->open_event, s); }
}
void launch_end(mono_table* t, int kid, cudaStream_t s) {
  if (t->timing) {
    cudaEvent_t stop = take_event(t);
    cudaEventRecord(stop, s);
    t->pending.push_back({kid, {t->open_event, stop}});
    t->open_event = nullptr;
  }
}
// Every kernel of the hot calls is launched through this, so that launches can
// be counted and, on request, timed one by one on the stream it runs on.
#define LAUNCH_ON(t, s, kid, ...) do { launch_begin((t), (kid), (s)); __VA_ARGS__; launch_end((t), (kid), (s)); } while (0)
#define LAUNCH(t, kid, ...) LAUNCH_ON(t, (t)->stream, kid, __VA_ARGS__)

// The table's stream waits for whatever the sweep stream still has in flight.
// Called by every entry point before it launches on, or synchronises, `stream`.
void join_sweep(mono_table* t) {
  if (t->sweep_pending) { cudaStreamWaitEvent(t->stream, t->ev_swept, 0); t->sweep_pending = false; }
  t->keys_idle = false;
}

int reserve(mono_table* t, int64_t max_ids, int64_t max_bags) {
  if (max_ids <= t->max_ids && max_bags <= t->max_bags) return MONO_OK;
  if (max_ids < t->max_ids) max_ids = t->max_ids;
  if (max_bags < t->max_bags) max_bags = t->max_bags;
  if (max_ids < 1024) max_ids = 1024;
  if (max_bags < 1024) max_bags = 1024;
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  CUDA_TRY(t, cudaStreamSynchronize(t->prep_stream));     // a prepared grouping is lost with the scratch it lives in
  if (t->prep.valid) { t->prep.valid = false; finish_apply_kernel<<<1, 256, 0, t->stream>>>(t->tv.st, t->wk.win_count, 0); }
  free_scratch(t);
  Work& w = t->wk;
  const size_t n = (size_t)max_ids;
  uint64_t primary = next_pow2(((uint64_t)max_ids * 2) / 5);
  if (primary < 1024) primary = 1024;
  const uint64_t secondary = next_pow2(2 * (uint64_t)max_ids);
  const uint64_t slots = primary + secondary;
  int rc;
#define ALLOC(p, cnt) if ((rc = dev_alloc(t, &(p), (cnt))) != MONO_OK) { free_scratch(t); return rc; }
  ALLOC(w.bset, slots);
  ALLOC(w.occ_slot, n); ALLOC(w.occ_rank, n); ALLOC(w.occ_bag, n); ALLOC(w.bag_of_sorted, n);
  ALLOC(w.uid, n); ALLOC(w.uslot, n); ALLOC(w.uocc, n); ALLOC(w.useg, n); ALLOC(w.ulen, n); ALLOC(w.urow, n);
  ALLOC(w.multi_list, n / 2 + 1); ALLOC(w.ins_list, n);
  w.max_long = (uint32_t)(n / kSegChunk + 1);
  w.max_parts = (uint32_t)(2 * (n / kSegChunk) + 2);
  ALLOC(w.long_u, w.max_long); ALLOC(w.long_part0, w.max_long); ALLOC(w.part_u, w.max_parts); ALLOC(w.part_order, w.max_parts); ALLOC(w.win_count, 2 * kWindows);
  ALLOC(w.partials, (size_t)w.max_parts * t->tv.dim);
  w.max_folds = w.max_parts / kFoldWidth + w.max_long + 1;
  ALLOC(w.fold_li, w.max_folds); ALLOC(w.fold_idx, w.max_folds);
  ALLOC(t->stage_ids, n); ALLOC(t->stage_off, (size_t)max_bags + 1);
  ALLOC(t->stage_vec, (size_t)max_bags * t->tv.dim);
  ALLOC(t->occ_row, n);
#undef ALLOC
  w.primary_mask = (uint32_t)(primary - 1);
  w.secondary_mask = (uint32_t)(secondary - 1);
  init_bset_kernel<<<grid_for(t, 4), 256, 0, t->stream>>>(w.bset, slots);
  CUDA_TRY(t, cudaGetLastError());
  CUDA_TRY(t, cudaMemsetAsync(w.win_count, 0, 2 * kWindows * sizeof(uint32_t), t->stream));
  t->max_ids = max_ids;
  t->max_bags = max_bags;
  return MONO_OK;
}

int check_batch(const mono_table* t, const void* ids, int64_t n_ids, const void* off, int64_t n_bags) {
  if (!t || n_ids < 0 || n_bags < 0) return MONO_ERR_ARG;
  if (n_ids >= (1ll << 31) || n_bags >= (1ll << 31)) return MONO_ERR_ARG;
  if (!off || !aligned(off, 8)) return MONO_ERR_ARG;
  if (n_ids > 0 && (!ids || !aligned(ids, 8))) return MONO_ERR_ARG;
  return MONO_OK;
}

// lane-group width and column vectors per lane for a given dim
template <typename F>
int dispatch_dim(uint32_t dim, F&& f) {
  if (dim <= 16) return f(std::integral_constant<int, 4>{}, std::integral_constant<int, 1>{});
  if (dim <= 32) return f(std::integral_constant<int, 8>{}, std::integral_constant<int, 1>{});
  if (dim <= 64) return f(std::integral_constant<int, 16>{}, std::integral_constant<int, 1>{});
  if (dim <= 128) return f(std::integral_constant<int, 32>{}, std::integral_constant<int, 1>{});
  if (dim <= 256) return f(std::integral_constant<int, 32>{}, std::integral_constant<int, 2>{});
  if (dim <= 512) return f(std::integral_constant<int, 32>{}, std::integral_constant<int, 4>{});
  return f(std::integral_constant<int, 32>{}, std::integral_constant<int, 8>{});
}

int launch_lookup(mono_table* t, const unsigned long long* ids, int64_t n_ids, const long long* off,
                  int64_t n_bags, float* out) {
  if (n_bags == 0) return MONO_OK;
  uint32_t* occ_row = t->occ_row;
  if (n_ids > 0) {
    int64_t blocks = (n_ids + 255) / 256;
    const int64_t cap = (int64_t)grid_for(t, 8) * 8;
    if (blocks > cap) blocks = cap;
    LAUNCH(t, K_PROBE, probe_rows_kernel<<<(int)blocks, 256, 0, t->stream>>>(t->tv, ids, n_ids, occ_row));
  }
  return dispatch_dim(t->tv.dim, [&](auto g, auto nv) -> int {
    constexpr int G = decltype(g)::value, NV = decltype(nv)::value;
    const int64_t groups_per_block = 256 / G;
    int64_t blocks = (n_bags + groups_per_block - 1) / groups_per_block;
    const int64_t cap = (int64_t)grid_for(t, 8) * 8;
    if (blocks > cap) blocks = cap;
    LAUNCH(t, K_GATHER, gather_pool_kernel<G, NV><<<(int)blocks, 256, 0, t->stream>>>(t->tv, occ_row, n_ids, off,
                                                                                    n_bags, out));
    CUDA_TRY(t, cudaGetLastError());
    return (int)MONO_OK;
  });
}

// The part of a push that depends on the IDs alone: bag of every occurrence, and the
// occurrences grouped by ID in the per-call set.
int launch_group(mono_table* t, cudaStream_t s, const unsigned long long* ids, int64_t n_ids, const long long* off,
                 int64_t n_bags) {
  const TableView& tv = t->tv;
  const Work& wk = t->wk;
  LAUNCH_ON(t, s, K_FILL_BAG, fill_occ_bag_kernel<<<grid_for(t, 8), 256, 0, s>>>(off, n_bags, n_ids, wk.occ_bag, tv.st));
  const int tiles = (int)((n_ids + kTileIds - 1) / kTileIds);
  LAUNCH_ON(t, s, K_DEDUP, dedup_tile_kernel<<<tiles, kTileThreads, 0, s>>>(wk, ids, n_ids, off, n_bags, tv.st,
                                                                          tv.seed0 ^ 0xA5A5A5A55A5A5A5Aull));
  CUDA_TRY(t, cudaGetLastError());
  return MONO_OK;
}

// Forget a prepared grouping: wait for it, then empty the per-call set and the per-call counters.
int discard_prepared(mono_table* t) {
  if (!t->prep.valid) return MONO_OK;
  t->prep.valid = false;
  CUDA_TRY(t, cudaStreamWaitEvent(t->stream, t->ev_prepared, 0));
  const uint64_t slots = (uint64_t)t->wk.primary_mask + 1 + (uint64_t)t->wk.secondary_mask + 1;
  init_bset_kernel<<<grid_for(t, 4), 256, 0, t->stream>>>(t->wk.bset, slots);
  finish_apply_kernel<<<1, 256, 0, t->stream>>>(t->tv.st, t->wk.win_count, 0);
  CUDA_TRY(t, cudaGetLastError());
  return MONO_OK;
}

int launch_apply(mono_table* t, const unsigned long long* ids, int64_t n_ids, const long long* off,
                 int64_t n_bags, const float* grad, uint32_t now) {
  int rc0 = MONO_OK;
  if (t->prep.valid && t->prep.ids == ids && t->prep.n_ids == n_ids && t->prep.off == off && t->prep.n_bags == n_bags) {
    // the grouping of exactly this batch is ready, or in flight on the preparation stream
    t->prep.valid = false;
    CUDA_TRY(t, cudaStreamWaitEvent(t->stream, t->ev_prepared, 0));
  } else {
    if ((rc0 = discard_prepared(t)) != MONO_OK) return rc0;
    if (n_ids == 0 || n_bags == 0) return MONO_OK;
    if ((rc0 = launch_group(t, t->stream, ids, n_ids, off, n_bags)) != MONO_OK) return rc0;
  }
  cudaStream_t s = t->stream;
  const TableView& tv = t->tv;
  const Work& wk = t->wk;
  // grids of the grid-stride kernels: several waves of blocks per SM where that measured faster
  // (shorter tails), one wave elsewhere
  const int g4 = grid_for(t, 4), g8 = grid_for(t, 8);
  LAUNCH(t, K_UPDATE, table_update_kernel<<<g8 * 4, 256, 0, s>>>(tv, wk, now));
  if (tv.sketch_depth) LAUNCH(t, K_SKETCH, sketch_add_kernel<<<g8, 256, 0, s>>>(tv, wk));
  LAUNCH(t, K_INSERT, table_insert_kernel<<<g8, 256, 0, s>>>(tv, wk, now));
  CUDA_TRY(t, cudaGetLastError());
  // the rest of the call touches rows and scratch only: a sweep may run beside it
  CUDA_TRY(t, cudaEventRecord(t->ev_keys, s));
  // The kernels that prepare and finish the reduction of the long segments (the few hottest
  // IDs) keep only a few blocks busy each, so they run on a stream of their own beside the
  // kernels that work through the whole batch: expand/order beside file_segments, and
  // fold/combine, which need only what reduce_adagrad left, beside update_singletons.  While
  // kernels are being timed one by one, everything stays on the table's stream.
  cudaStream_t a = t->timing ? s : t->aux_stream;
  if (a != s) CUDA_TRY(t, cudaStreamWaitEvent(a, t->ev_keys, 0));
  LAUNCH_ON(t, a, K_EXPAND, expand_parts_kernel<<<g8 * 4, 128, 0, a>>>(tv, wk));
  LAUNCH_ON(t, a, K_ORDER, order_parts_kernel<<<64, kWindows, 0, a>>>(tv, wk));
  CUDA_TRY(t, cudaGetLastError());
  if (a != s) CUDA_TRY(t, cudaEventRecord(t->ev_parts, a));
  const int rc = dispatch_dim(tv.dim, [&](auto g, auto nv) -> int {
    constexpr int G = decltype(g)::value, NV = decltype(nv)::value;
    LAUNCH(t, K_FILE, file_segments_kernel<<<g8, 256, 0, s>>>(wk, n_ids, n_bags));
    if (a != s) CUDA_TRY(t, cudaStreamWaitEvent(s, t->ev_parts, 0));
    LAUNCH(t, K_REDUCE, reduce_adagrad_kernel<G, NV><<<g8 * 8, 128, 0, s>>>(tv, wk, grad, n_bags));
    if (a != s) {
      CUDA_TRY(t, cudaEventRecord(t->ev_reduced, s));
      CUDA_TRY(t, cudaStreamWaitEvent(a, t->ev_reduced, 0));
    }
    LAUNCH(t, K_SINGLES, update_singletons_kernel<G, NV><<<g8 * 8, 128, 0, s>>>(tv, wk, grad, n_bags));
    return (int)MONO_OK;
  });
  if (rc != MONO_OK) return rc;
  LAUNCH_ON(t, a, K_FOLD, fold_partials_kernel<<<g4, 256, 0, a>>>(tv, wk));
  LAUNCH_ON(t, a, K_COMBINE, combine_adagrad_kernel<<<g8, kCombineThreads, 0, a>>>(tv, wk));
  if (a != s) {
    CUDA_TRY(t, cudaEventRecord(t->ev_aux, a));
    CUDA_TRY(t, cudaStreamWaitEvent(s, t->ev_aux, 0));
  }
  LAUNCH(t, K_FINISH, finish_apply_kernel<<<1, 256, 0, s>>>(tv.st, wk.win_count, 1));
  CUDA_TRY(t, cudaGetLastError());
  t->keys_idle = true;
  return MONO_OK;
}

int check_now(mono_table* t, int64_t now) {
  if (now < 0 || now > MONO_MAX_NOW || now < t->last_now) return MONO_ERR_TIME;
  return MONO_OK;
}

// Fork/join of a grouped call around `one(i)`, the single-table call of table i.
template <typename F>
int group_call(int32_t n_tables, mono_table* const* tables, void* group_stream, F&& one) {
  if (n_tables < 0 || (n_tables > 0 && !tables)) return MONO_ERR_ARG;
  if (n_tables == 0) return MONO_OK;
  for (int32_t i = 0; i < n_tables; ++i) {
    if (!tables[i]) return MONO_ERR_ARG;
    for (int32_t j = 0; j < i; ++j) if (tables[j] == tables[i]) return MONO_ERR_ARG;
  }
  cudaStream_t gs = static_cast<cudaStream_t>(group_stream);
  mono_table* t0 = tables[0];
  CUDA_TRY(t0, cudaEventRecord(t0->ev_fork, gs));              // (ev_fork is re-recorded by whoever uses it next)
  int rc = MONO_OK;
  int32_t started = 0;
  for (; started < n_tables && rc == MONO_OK; ++started) {
    mono_table* t = tables[started];
    if (t->stream != gs) CUDA_TRY(t, cudaStreamWaitEvent(t->stream, t0->ev_fork, 0));
    rc = one(started);
  }
  // join what was started, also after an error
  for (int32_t i = 0; i < started; ++i) {
    mono_table* t = tables[i];
    if (t->stream == gs) continue;
    CUDA_TRY(t, cudaEventRecord(t->ev_group, t->stream));
    CUDA_TRY(t, cudaStreamWaitEvent(gs, t->ev_group, 0));
  }
  return rc;
}

}  // namespace

extern "C" {

int mono_table_create(mono_table** out, uint64_t capacity, uint32_t dim, uint32_t filter_threshold,
                      uint32_t ttl, const mono_opt* opt, void* cuda_stream) {
  if (!out) return MONO_ERR_ARG;
  *out = nullptr;
  if (capacity == 0 || capacity > MONO_MAX_CAPACITY) return MONO_ERR_ARG;
  if (dim < 4 || dim > MONO_MAX_DIM || (dim & 3u)) return MONO_ERR_ARG;
  if (filter_threshold >= 0x7FFFFFFFu) return MONO_ERR_ARG;
  mono_opt o;
  std::memset(&o, 0, sizeof(o));
  if (opt) o = *opt; else { o.lr = 0.05f; o.eps = 1e-8f; }
  if (o.kind != 0 && o.kind != MONO_OPT_ADAGRAD) return MONO_ERR_ARG;
  uint64_t key_cells = o.key_cells ? o.key_cells : next_pow2(4 * capacity);
  if (!is_pow2(key_cells) || key_cells < 64 || key_cells > (1ull << 34)) return MONO_ERR_ARG;
  if (o.max_ids >= (1ull << 31) || o.max_bags >= (1ull << 31)) return MONO_ERR_ARG;
  if (o.sketch_depth > 8 || (o.sketch_depth && (!is_pow2(o.sketch_width) || o.sketch_width > (1ull << 32)))) return MONO_ERR_ARG;

  mono_table* t = new (std::nothrow) mono_table();
  if (!t) return MONO_ERR_NOMEM;
  t->stream = static_cast<cudaStream_t>(cuda_stream);
  t->key_cells = key_cells;
  int dev = 0, rc = MONO_OK;
  auto fail = [&](int code) { mono_table_destroy(t); return code; };
  if (cudaGetDevice(&dev) != cudaSuccess) return fail(MONO_ERR_CUDA);
  if (cudaDeviceGetAttribute(&t->sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || t->sm_count < 1)
    return fail(MONO_ERR_CUDA);
  if (cudaStreamCreateWithFlags(&t->prep_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaStreamCreateWithFlags(&t->sweep_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaStreamCreateWithFlags(&t->aux_stream, cudaStreamNonBlocking) != cudaSuccess)
    return fail(MONO_ERR_CUDA);
  for (cudaEvent_t* e : {&t->ev_fork, &t->ev_prepared, &t->ev_keys, &t->ev_swept, &t->ev_group, &t->ev_parts,
                         &t->ev_reduced, &t->ev_aux})
    if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return fail(MONO_ERR_CUDA);

  TableView& tv = t->tv;
  tv.bucket_mask = key_cells / kCellsPerBucket - 1;
  tv.seed0 = mix_a(o.seed + 0x1234567ull);
  tv.seed1 = mix_b(o.seed + 0x89ABCDEFull);
  tv.capacity = capacity;
  tv.dim = dim;
  tv.threshold = filter_threshold ? filter_threshold : 1u;
  tv.ttl = ttl;
  tv.lr = o.lr; tv.eps = o.eps; tv.init_acc = o.init_acc; tv.init_scale = o.init_scale;
  tv.init_key0 = (uint32_t)o.seed;
  tv.init_key1 = (uint32_t)(o.seed >> 32);
  if ((rc = dev_alloc(t, &tv.cells, key_cells)) != MONO_OK) return fail(rc);
  if ((rc = dev_alloc(t, &tv.stash, kStashCells)) != MONO_OK) return fail(rc);
  // one row more than the capacity: row index `capacity` is never handed out and stays all zero
  // (the lookup adds it for an ID that has no row)
  if ((rc = dev_alloc(t, &tv.rows, ((size_t)capacity + 1) * 2 * dim)) != MONO_OK) return fail(rc);
  if (cudaMemsetAsync(tv.rows + (size_t)capacity * 2 * dim, 0, (size_t)2 * dim * sizeof(float), t->stream) != cudaSuccess)
    return fail(MONO_ERR_CUDA);
  if ((rc = dev_alloc(t, &tv.free_rows, capacity)) != MONO_OK) return fail(rc);
  if ((rc = dev_alloc(t, &tv.st, 1)) != MONO_OK) return fail(rc);
  tv.sketch_depth = o.sketch_depth;
  tv.sketch_seed = o.seed;
  if (o.sketch_depth) {
    tv.sketch_mask = o.sketch_width - 1;
    const size_t counters = (size_t)o.sketch_depth * o.sketch_width;
    if ((rc = dev_alloc(t, &tv.sketch, counters)) != MONO_OK) return fail(rc);
    if (cudaMemsetAsync(tv.sketch, 0, counters * sizeof(unsigned int), t->stream) != cudaSuccess) return fail(MONO_ERR_CUDA);
  }
  DevState init;
  std::memset(&init, 0, sizeof(init));
  init.free_top = (long long)capacity;
  if (cudaMemcpyAsync(tv.st, &init, sizeof(init), cudaMemcpyHostToDevice, t->stream) != cudaSuccess ||
      cudaStreamSynchronize(t->stream) != cudaSuccess)
    return fail(MONO_ERR_CUDA);
  init_table_kernel<<<grid_for(t, 8), 256, 0, t->stream>>>(tv, key_cells);
  if (cudaGetLastError() != cudaSuccess) return fail(MONO_ERR_CUDA);
  if (o.max_ids || o.max_bags) {
    if ((rc = reserve(t, (int64_t)o.max_ids, (int64_t)o.max_bags)) != MONO_OK) return fail(rc);
  }
  if (cudaStreamSynchronize(t->stream) != cudaSuccess) return fail(MONO_ERR_CUDA);
  *out = t;
  return MONO_OK;
}

int mono_table_destroy(mono_table* t) {
  if (!t) return MONO_ERR_ARG;
  cudaStreamSynchronize(t->stream);
  if (t->prep_stream) { cudaStreamSynchronize(t->prep_stream); cudaStreamDestroy(t->prep_stream); }
  if (t->sweep_stream) { cudaStreamSynchronize(t->sweep_stream); cudaStreamDestroy(t->sweep_stream); }
  if (t->aux_stream) { cudaStreamSynchronize(t->aux_stream); cudaStreamDestroy(t->aux_stream); }
  for (cudaEvent_t e : {t->ev_fork, t->ev_prepared, t->ev_keys, t->ev_swept, t->ev_group, t->ev_parts, t->ev_reduced,
                        t->ev_aux})
    if (e) cudaEventDestroy(e);
  for (auto& p : t->pending) { cudaEventDestroy(p.second.first); cudaEventDestroy(p.second.second); }
  for (cudaEvent_t e : t->spare_events) cudaEventDestroy(e);
  free_scratch(t);
  dev_free(t->tv.cells); dev_free(t->tv.stash); dev_free(t->tv.rows); dev_free(t->tv.free_rows); dev_free(t->tv.st); dev_free(t->tv.sketch);
  delete t;
  return MONO_OK;
}

int mono_reserve(mono_table* t, int64_t max_ids, int64_t max_bags) {
  if (t) join_sweep(t);
  if (!t || max_ids < 0 || max_bags < 0 || max_ids >= (1ll << 31) || max_bags >= (1ll << 31)) return MONO_ERR_ARG;
  return reserve(t, max_ids, max_bags);
}

int mono_lookup_pool(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                     int64_t n_bags, float* out) {
  if (t) join_sweep(t);
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if (n_bags > 0 && (!out || !aligned(out, 16))) return MONO_ERR_ARG;
  if ((rc = reserve(t, n_ids, n_bags)) != MONO_OK) return rc;
  return launch_lookup(t, reinterpret_cast<const unsigned long long*>(ids), n_ids,
                       reinterpret_cast<const long long*>(slot_offsets), n_bags, out);
}

int mono_apply_grads(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                     int64_t n_bags, const float* grad_pooled, int64_t now) {
  if (t) join_sweep(t);
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if (n_bags > 0 && (!grad_pooled || !aligned(grad_pooled, 16))) return MONO_ERR_ARG;
  if ((rc = check_now(t, now)) != MONO_OK) return rc;
  if ((rc = reserve(t, n_ids, n_bags)) != MONO_OK) return rc;
  t->last_now = now;
  return launch_apply(t, reinterpret_cast<const unsigned long long*>(ids), n_ids,
                      reinterpret_cast<const long long*>(slot_offsets), n_bags, grad_pooled, (uint32_t)now);
}

int mono_prepare_push(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets, int64_t n_bags) {
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if ((rc = reserve(t, n_ids, n_bags)) != MONO_OK) return rc;
  if ((rc = discard_prepared(t)) != MONO_OK) return rc;
  if (n_ids == 0 || n_bags == 0) return MONO_OK;
  // after everything already on the table's stream (the previous push still owns the scratch) ...
  CUDA_TRY(t, cudaEventRecord(t->ev_fork, t->stream));
  CUDA_TRY(t, cudaStreamWaitEvent(t->prep_stream, t->ev_fork, 0));
  // ... and beside everything that comes next on it
  if ((rc = launch_group(t, t->prep_stream, reinterpret_cast<const unsigned long long*>(ids), n_ids,
                         reinterpret_cast<const long long*>(slot_offsets), n_bags)) != MONO_OK) return rc;
  CUDA_TRY(t, cudaEventRecord(t->ev_prepared, t->prep_stream));
  t->prep = {ids, n_ids, slot_offsets, n_bags, true};
  return MONO_OK;
}

int mono_group_lookup_pool(int32_t n_tables, mono_table* const* tables, const uint64_t* const* ids,
                           const int64_t* n_ids, const int64_t* const* slot_offsets, const int64_t* n_bags,
                           float* const* out, void* group_stream) {
  if (n_tables > 0 && (!ids || !n_ids || !slot_offsets || !n_bags || !out)) return MONO_ERR_ARG;
  return group_call(n_tables, tables, group_stream, [&](int32_t i) {
    return mono_lookup_pool(tables[i], ids[i], n_ids[i], slot_offsets[i], n_bags[i], out[i]);
  });
}

int mono_group_apply_grads(int32_t n_tables, mono_table* const* tables, const uint64_t* const* ids,
                           const int64_t* n_ids, const int64_t* const* slot_offsets, const int64_t* n_bags,
                           const float* const* grad_pooled, int64_t now, void* group_stream) {
  if (n_tables > 0 && (!ids || !n_ids || !slot_offsets || !n_bags || !grad_pooled)) return MONO_ERR_ARG;
  return group_call(n_tables, tables, group_stream, [&](int32_t i) {
    return mono_apply_grads(tables[i], ids[i], n_ids[i], slot_offsets[i], n_bags[i], grad_pooled[i], now);
  });
}

static int expire_range(mono_table* t, int64_t now, uint32_t slice, uint32_t n_slices) {
  if (!t || n_slices == 0 || slice >= n_slices) return MONO_ERR_ARG;
  int rc = check_now(t, now);
  if (rc != MONO_OK) return rc;
  t->last_now = now;
  if (t->tv.ttl == 0) return MONO_OK;
  // The sweep runs on its own stream.  It has to follow everything launched so far that
  // touches the key store, the free list or the sketch; the tail of a mono_apply_grads
  // (gradient reduction and row updates) touches none of them, so a sweep that comes
  // straight after one starts as soon as that call's key-store work is done and runs
  // beside the rest.  The next call on the table's stream waits for the sweep.
  cudaStream_t s = t->sweep_stream;
  if (!t->sweep_pending) {
    // (while kernels are being timed one by one, the sweep waits for the whole stream instead)
    if (!t->keys_idle || t->timing) CUDA_TRY(t, cudaEventRecord(t->ev_keys, t->stream));
    CUDA_TRY(t, cudaStreamWaitEvent(s, t->ev_keys, 0));
  }                                               // else: it follows the previous sweep, which waited already
  if (slice == 0 && t->tv.sketch_depth && now - t->sketch_epoch > (int64_t)t->tv.ttl) {
    // the sketch forgets in whole windows: cleared when more than ttl has passed since the last clearing
    CUDA_TRY(t, cudaMemsetAsync(t->tv.sketch, 0, (size_t)t->tv.sketch_depth * (t->tv.sketch_mask + 1) * sizeof(unsigned int), s));
    t->sketch_epoch = now;
  }
  const unsigned long long total = t->key_cells + kStashCells;
  const unsigned long long first = t->key_cells / n_slices * slice;             // key_cells is a power of two >= 64
  const unsigned long long last = slice + 1 == n_slices ? total : t->key_cells / n_slices * (slice + 1);
  if (last > first) {
    unsigned long long blocks = (last - first + 255) / 256;
    if (blocks > (unsigned long long)grid_for(t, 8)) blocks = grid_for(t, 8);
    LAUNCH_ON(t, s, K_EXPIRE, expire_kernel<<<(int)blocks, 256, 0, s>>>(t->tv, t->key_cells, first, last, (long long)now));
  }
  if (slice + 1 == n_slices) LAUNCH_ON(t, s, K_STASH_TRIM, stash_trim_kernel<<<1, 32, 0, s>>>(t->tv));
  CUDA_TRY(t, cudaGetLastError());
  CUDA_TRY(t, cudaEventRecord(t->ev_swept, s));
  t->sweep_pending = true;
  return MONO_OK;
}

int mono_expire(mono_table* t, int64_t now) { return expire_range(t, now, 0, 1); }

int mono_expire_slice(mono_table* t, int64_t now, uint32_t slice, uint32_t n_slices) {
  if (n_slices > 65536) return MONO_ERR_ARG;
  return expire_range(t, now, slice, n_slices);
}

// Device address of g_noalloc_occ_row on the current device, looked up once per
// device (with that device current) and remembered.
static int noalloc_scratch(mono_table* t, uint32_t** out) {
  static std::mutex mu;
  static uint32_t* addr[64] = {};
  int dev = 0;
  CUDA_TRY(t, cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return MONO_ERR_ARG;
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    uint32_t* p = nullptr;
    CUDA_TRY(t, cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_occ_row));
    addr[dev] = p;
  }
  *out = addr[dev];
  return MONO_OK;
}

int mono_lookup_pool_noalloc(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                             int64_t n_bags, float* out) {
  if (t) join_sweep(t);
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if (n_bags > 0 && (!out || !aligned(out, 16))) return MONO_ERR_ARG;
  if (n_ids > (int64_t)MONO_NOALLOC_MAX_IDS) return MONO_ERR_LIMIT;
  if (n_bags == 0) return MONO_OK;
  uint32_t* occ_row = nullptr;
  if ((rc = noalloc_scratch(t, &occ_row)) != MONO_OK) return rc;
  const unsigned long long* d_ids = reinterpret_cast<const unsigned long long*>(ids);
  const long long* d_off = reinterpret_cast<const long long*>(slot_offsets);
  if (n_ids > 0) {
    int64_t blocks = (n_ids + 255) / 256;
    const int64_t cap = (int64_t)grid_for(t, 8) * 4;
    if (blocks > cap) blocks = cap;
    LAUNCH(t, K_PROBE, probe_rows_kernel<<<(int)blocks, 256, 0, t->stream>>>(t->tv, d_ids, n_ids, occ_row));
  }
  return dispatch_dim(t->tv.dim, [&](auto g, auto nv) -> int {
    constexpr int G = decltype(g)::value, NV = decltype(nv)::value;
    const int64_t groups_per_block = 256 / G;
    int64_t blocks = (n_bags + groups_per_block - 1) / groups_per_block;
    const int64_t cap = (int64_t)grid_for(t, 8) * 8;
    if (blocks > cap) blocks = cap;
    LAUNCH(t, K_GATHER, gather_pool_kernel<G, NV><<<(int)blocks, 256, 0, t->stream>>>(t->tv, occ_row, n_ids, d_off,
                                                                                    n_bags, out));
    CUDA_TRY(t, cudaGetLastError());
    return (int)MONO_OK;
  });
}

int mono_lookup_pool_host(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                          int64_t n_bags, float* out) {
  if (t) join_sweep(t);
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if (n_bags > 0 && !out) return MONO_ERR_ARG;
  if ((rc = reserve(t, n_ids, n_bags)) != MONO_OK) return rc;
  cudaStream_t s = t->stream;
  if (n_ids) CUDA_TRY(t, cudaMemcpyAsync(t->stage_ids, ids, (size_t)n_ids * 8, cudaMemcpyHostToDevice, s));
  CUDA_TRY(t, cudaMemcpyAsync(t->stage_off, slot_offsets, (size_t)(n_bags + 1) * 8, cudaMemcpyHostToDevice, s));
  if ((rc = launch_lookup(t, t->stage_ids, n_ids, t->stage_off, n_bags, t->stage_vec)) != MONO_OK) return rc;
  if (n_bags)
    CUDA_TRY(t, cudaMemcpyAsync(out, t->stage_vec, (size_t)n_bags * t->tv.dim * 4, cudaMemcpyDeviceToHost, s));
  CUDA_TRY(t, cudaStreamSynchronize(s));
  return MONO_OK;
}

int mono_apply_grads_host(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                          int64_t n_bags, const float* grad_pooled, int64_t now) {
  if (t) join_sweep(t);
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if (n_bags > 0 && !grad_pooled) return MONO_ERR_ARG;
  if ((rc = check_now(t, now)) != MONO_OK) return rc;
  if ((rc = reserve(t, n_ids, n_bags)) != MONO_OK) return rc;
  cudaStream_t s = t->stream;
  if (n_ids) CUDA_TRY(t, cudaMemcpyAsync(t->stage_ids, ids, (size_t)n_ids * 8, cudaMemcpyHostToDevice, s));
  CUDA_TRY(t, cudaMemcpyAsync(t->stage_off, slot_offsets, (size_t)(n_bags + 1) * 8, cudaMemcpyHostToDevice, s));
  if (n_bags)
    CUDA_TRY(t, cudaMemcpyAsync(t->stage_vec, grad_pooled, (size_t)n_bags * t->tv.dim * 4, cudaMemcpyHostToDevice, s));
  t->last_now = now;
  return launch_apply(t, t->stage_ids, n_ids, t->stage_off, n_bags, t->stage_vec, (uint32_t)now);
}

int mono_status(mono_table* t, mono_status_t* host_out) {
  if (t) join_sweep(t);
  if (!t || !host_out) return MONO_ERR_ARG;
  DevState d;
  CUDA_TRY(t, cudaMemcpyAsync(&d, t->tv.st, sizeof(d), cudaMemcpyDeviceToHost, t->stream));
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  std::memset(host_out, 0, sizeof(*host_out));
  host_out->error_bits = d.error_bits;
  host_out->dim = t->tv.dim;
  host_out->capacity = t->tv.capacity;
  host_out->key_cells = t->key_cells;
  host_out->n_tracked = d.n_tracked;
  host_out->n_resident = d.n_resident;
  host_out->n_admitted_total = d.n_admitted_total;
  host_out->n_expired_total = d.n_expired_total;
  host_out->n_inserted_total = d.n_inserted_total;
  host_out->n_rows_refused = d.n_rows_refused;
  host_out->n_keys_dropped = d.n_keys_dropped;
  host_out->n_evictions_total = d.n_evictions_total;
  host_out->max_chain = d.max_chain;
  host_out->stash_used = d.stash_hw;
  host_out->sum_ids = d.sum_ids;
  host_out->sum_unique = d.sum_unique;
  host_out->sum_unique_resident = d.sum_unique_resident;
  host_out->sum_new = d.sum_new;
  host_out->sum_single_resident = d.sum_single_resident;
  return MONO_OK;
}

int mono_clear_errors(mono_table* t) {
  if (t) join_sweep(t);
  if (!t) return MONO_ERR_ARG;
  CUDA_TRY(t, cudaMemsetAsync(&t->tv.st->error_bits, 0, sizeof(unsigned int), t->stream));
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  return MONO_OK;
}

int mono_probe(mono_table* t, const uint64_t* ids, int64_t n, uint8_t* resident, uint32_t* count,
               int64_t* last_seen) {
  if (t) join_sweep(t);
  if (!t || n < 0 || (n > 0 && (!ids || !aligned(ids, 8)))) return MONO_ERR_ARG;
  if (n > 0) {
    probe_kernel<<<grid_for(t, 4), 256, 0, t->stream>>>(t->tv, reinterpret_cast<const unsigned long long*>(ids), n,
                                                        resident, count, reinterpret_cast<long long*>(last_seen));
    CUDA_TRY(t, cudaGetLastError());
  }
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  return MONO_OK;
}

int mono_read_rows(mono_table* t, const uint64_t* ids, int64_t n, float* w, float* acc) {
  if (t) join_sweep(t);
  if (!t || n < 0 || (n > 0 && (!ids || !aligned(ids, 8)))) return MONO_ERR_ARG;
  if ((w && !aligned(w, 16)) || (acc && !aligned(acc, 16))) return MONO_ERR_ARG;
  if (n > 0) {
    read_rows_kernel<<<grid_for(t, 4), 256, 0, t->stream>>>(t->tv, reinterpret_cast<const unsigned long long*>(ids),
                                                            n, w, acc);
    CUDA_TRY(t, cudaGetLastError());
  }
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  return MONO_OK;
}

int mono_export(mono_table* t, uint64_t* ids, uint32_t* count, int64_t* last_seen, uint8_t* resident,
                float* w, float* acc, int64_t max_n, int64_t* n_out) {
  if (t) join_sweep(t);
  if (!t || !n_out || max_n < 0 || (max_n > 0 && !ids)) return MONO_ERR_ARG;
  CUDA_TRY(t, cudaMemsetAsync(&t->tv.st->export_n, 0, sizeof(unsigned long long), t->stream));
  export_kernel<<<grid_for(t, 8), 256, 0, t->stream>>>(t->tv, t->key_cells,
                                                       reinterpret_cast<unsigned long long*>(ids), count,
                                                       reinterpret_cast<long long*>(last_seen), resident, w, acc, max_n);
  CUDA_TRY(t, cudaGetLastError());
  unsigned long long n = 0;
  CUDA_TRY(t, cudaMemcpyAsync(&n, &t->tv.st->export_n, sizeof(n), cudaMemcpyDeviceToHost, t->stream));
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  *n_out = (int64_t)n;
  return (int64_t)n > max_n ? MONO_ERR_SIZE : MONO_OK;
}

int mono_rehash(mono_table* t, uint64_t new_key_cells, uint64_t new_seed) {
  if (t) join_sweep(t);
  if (!t) return MONO_ERR_ARG;
  if (new_key_cells == 0) new_key_cells = t->key_cells;
  if (!is_pow2(new_key_cells) || new_key_cells < 64 || new_key_cells > (1ull << 34)) return MONO_ERR_ARG;
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  TableView fresh = t->tv;
  fresh.cells = nullptr;
  fresh.stash = nullptr;
  int rc = dev_alloc(t, &fresh.cells, new_key_cells);
  if (rc == MONO_OK) rc = dev_alloc(t, &fresh.stash, kStashCells);
  if (rc != MONO_OK) { dev_free(fresh.cells); dev_free(fresh.stash); return rc; }
  fresh.bucket_mask = new_key_cells / kCellsPerBucket - 1;
  fresh.seed0 = mix_a(new_seed + 0x1234567ull);
  fresh.seed1 = mix_b(new_seed + 0x89ABCDEFull);
  const unsigned long long old_n = t->key_cells;
  // the new store starts empty (capacity 0 keeps the kernel away from the free-row list)
  TableView init_view = fresh;
  init_view.capacity = 0;
  init_table_kernel<<<grid_for(t, 8), 256, 0, t->stream>>>(init_view, new_key_cells);
  cudaError_t e = cudaMemsetAsync(&t->tv.st->stash_hw, 0, sizeof(unsigned int), t->stream);
  if (e == cudaSuccess) {
    rehash_kernel<<<grid_for(t, 8), 256, 0, t->stream>>>(fresh, t->tv.cells, old_n, t->tv.stash);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(t->stream);
  if (e != cudaSuccess) {
    t->last_err = cudaGetErrorString(e);
    dev_free(fresh.cells); dev_free(fresh.stash);
    return MONO_ERR_CUDA;
  }
  dev_free(t->tv.cells);
  dev_free(t->tv.stash);
  t->tv = fresh;
  t->key_cells = new_key_cells;
  return MONO_OK;
}

int mono_export_touched(mono_table* t, uint64_t* ids, float* w, int64_t max_n, int64_t* n_out) {
  if (t) join_sweep(t);
  if (!t || !n_out || max_n < 0 || (max_n > 0 && (!ids || !w || !aligned(w, 16) || !aligned(ids, 8)))) return MONO_ERR_ARG;
  CUDA_TRY(t, cudaMemsetAsync(&t->tv.st->export_n, 0, sizeof(unsigned long long), t->stream));
  export_touched_kernel<<<grid_for(t, 8), 256, 0, t->stream>>>(t->tv, t->key_cells,
                                                               reinterpret_cast<unsigned long long*>(ids), w, max_n);
  CUDA_TRY(t, cudaGetLastError());
  unsigned long long n = 0;
  CUDA_TRY(t, cudaMemcpyAsync(&n, &t->tv.st->export_n, sizeof(n), cudaMemcpyDeviceToHost, t->stream));
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  *n_out = (int64_t)n;
  return (int64_t)n > max_n ? MONO_ERR_SIZE : MONO_OK;
}

int mono_import(mono_table* t, const uint64_t* ids, const uint32_t* count, const int64_t* last_seen,
                const uint8_t* resident, const float* w, const float* acc, int64_t n) {
  if (t) join_sweep(t);
  if (!t || n < 0) return MONO_ERR_ARG;
  if (n == 0) return MONO_OK;
  if (!ids || !count || !last_seen || !resident || !aligned(ids, 8)) return MONO_ERR_ARG;
  if ((w && !aligned(w, 16)) || (acc && !aligned(acc, 16))) return MONO_ERR_ARG;
  uint32_t* row_word = nullptr;
  const int64_t chunk = n < (1ll << 24) ? n : (1ll << 24);
  int rc = dev_alloc(t, &row_word, (size_t)chunk);
  if (rc != MONO_OK) return rc;
  for (int64_t lo = 0; lo < n; lo += chunk) {
    const int64_t m = n - lo < chunk ? n - lo : chunk;
    const size_t ro = (size_t)lo * t->tv.dim;
    import_insert_kernel<<<grid_for(t, 4), 256, 0, t->stream>>>(
        t->tv, reinterpret_cast<const unsigned long long*>(ids) + lo, count + lo,
        reinterpret_cast<const long long*>(last_seen) + lo, resident + lo, m, row_word);
    import_rows_kernel<<<grid_for(t, 8), 256, 0, t->stream>>>(
        t->tv, reinterpret_cast<const unsigned long long*>(ids) + lo, w ? w + ro : nullptr, acc ? acc + ro : nullptr,
        m, row_word);
  }
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaStreamSynchronize(t->stream);
  cudaFree(row_word);
  if (e != cudaSuccess) { t->last_err = cudaGetErrorString(e); return MONO_ERR_CUDA; }
  return MONO_OK;
}

int mono_audit(mono_table* t, mono_audit_t* host_out) {
  if (t) join_sweep(t);
  if (!t || !host_out) return MONO_ERR_ARG;
  std::memset(host_out, 0, sizeof(*host_out));
  unsigned int* marks = nullptr;
  AuditCounters* ctr = nullptr;
  const size_t words = (size_t)((t->tv.capacity + 31) / 32);
  int rc = dev_alloc(t, &marks, words);
  if (rc == MONO_OK) rc = dev_alloc(t, &ctr, 1);
  AuditCounters h;
  std::memset(&h, 0, sizeof(h));
  DevState d;
  cudaError_t e = cudaSuccess;
  if (rc == MONO_OK) {
    cudaStream_t s = t->stream;
    e = cudaMemsetAsync(marks, 0, words * sizeof(unsigned int), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctr, 0, sizeof(AuditCounters), s);
    if (e == cudaSuccess) {
      audit_cells_kernel<<<grid_for(t, 8), 256, 0, s>>>(t->tv, t->key_cells, marks, ctr);
      audit_free_kernel<<<grid_for(t, 8), 256, 0, s>>>(t->tv, marks, ctr);
      audit_rows_kernel<<<grid_for(t, 8), 256, 0, s>>>(t->tv, marks, ctr);
      e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(&h, ctr, sizeof(h), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&d, t->tv.st, sizeof(d), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  }
  if (marks) cudaFree(marks);
  if (ctr) cudaFree(ctr);
  if (rc != MONO_OK) return rc;
  if (e != cudaSuccess) { t->last_err = cudaGetErrorString(e); return MONO_ERR_CUDA; }
  host_out->occupied_cells = h.occupied;
  host_out->misplaced = h.misplaced;
  host_out->duplicate_keys = h.duplicate_keys;
  host_out->resident_cells = h.resident_cells;
  host_out->bad_rows = h.bad_rows;
  host_out->shared_rows = h.shared_rows;
  host_out->free_rows = h.free_rows;
  host_out->unaccounted_rows = h.unaccounted_rows;
  const bool leak_ok = h.unaccounted_rows == 0 || d.n_keys_dropped > 0;   // a dropped key may strand its row
  host_out->ok = (h.misplaced == 0 && h.duplicate_keys == 0 && h.bad_rows == 0 && h.shared_rows == 0 && leak_ok &&
                  h.occupied == d.n_tracked && h.resident_cells == d.n_resident &&
                  h.resident_cells + h.free_rows + h.unaccounted_rows == t->tv.capacity)
                     ? 1u : 0u;
  return MONO_OK;
}

int mono_timing_enable(mono_table* t, int on) {
  if (!t) return MONO_ERR_ARG;
  t->timing = on != 0;
  return MONO_OK;
}

int mono_timing_read(mono_table* t, mono_timing_t* host_out, int reset) {
  if (t) join_sweep(t);
  if (!t || !host_out) return MONO_ERR_ARG;
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  CUDA_TRY(t, cudaStreamSynchronize(t->prep_stream));
  for (auto& p : t->pending) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, p.second.first, p.second.second) == cudaSuccess) t->kernel_ms[p.first] += ms;
    t->spare_events.push_back(p.second.first);
    t->spare_events.push_back(p.second.second);
  }
  t->pending.clear();
  std::memset(host_out, 0, sizeof(*host_out));
  host_out->n_kernels = K_COUNT;
  for (int k = 0; k < K_COUNT; ++k) {
    std::strncpy(host_out->kernel[k].name, kKernelNames[k], sizeof(host_out->kernel[k].name) - 1);
    host_out->kernel[k].launches = t->launches[k];
    host_out->kernel[k].ms = t->kernel_ms[k];
    host_out->launches_total += t->launches[k];
  }
  if (reset) {
    for (int k = 0; k < K_COUNT; ++k) { t->launches[k] = 0; t->kernel_ms[k] = 0.0; }
  }
  return MONO_OK;
}

const char* mono_last_cuda_error(mono_table* t) { return t ? t->last_err.c_str() : ""; }

const char* mono_error_string(int code) {
  switch (code) {
    case MONO_OK: return "MONO_OK";
    case MONO_ERR_ARG: return "MONO_ERR_ARG";
    case MONO_ERR_TIME: return "MONO_ERR_TIME";
    case MONO_ERR_CUDA: return "MONO_ERR_CUDA";
    case MONO_ERR_NOMEM: return "MONO_ERR_NOMEM";
    case MONO_ERR_SIZE: return "MONO_ERR_SIZE";
    case MONO_ERR_LIMIT: return "MONO_ERR_LIMIT";
    default: return "MONO_ERR_UNKNOWN";
  }
}

}  // extern "C"
