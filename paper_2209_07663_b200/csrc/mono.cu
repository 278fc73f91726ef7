// Host side of the C ABI declared in include/mono.h: argument checks, memory
// ownership, and the launch sequence of each call.  Every step of the hot path
// runs in the kernels included below; nothing here computes on the host.
#include <cstdint>
#include <cstdio>
#include <algorithm>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include "../../include/mono.h"
#include "kernels_adagrad.cuh"
#include "kernels_dedup.cuh"
#include "kernels_forward.cuh"
#include "kernels_group.cuh"
#include "kernels_inspect.cuh"
#include "kernels_table.cuh"
#include "table_layout.cuh"

using namespace mono;

// Scratch of mono_lookup_pool_noalloc: part of the library image, so the entry
// point never allocates.  In host code this name is only a handle for
// cudaGetSymbolAddress; kernels get the device address that call returns.
static __device__ __align__(256) uint32_t g_noalloc_occ_row[MONO_NOALLOC_MAX_IDS];

enum KernelId {
  K_PROBE, K_GATHER, K_FILL_BAG, K_DEDUP, K_LOOKUP, K_UPDATE, K_SKETCH, K_INSERT, K_EXPAND, K_ORDER, K_FILE, K_SINGLES, K_REDUCE, K_FOLD, K_COMBINE, K_FINISH, K_EXPIRE,
  K_STASH_TRIM, K_CLEAR, K_REDUCE_PARTS, K_ADOPT, K_COUNT
};
// (table_lookup and table_update are the two halves of table_update_kernel; a push that was not
// announced runs both in one launch, counted as table_update)
static const char* const kKernelNames[K_COUNT] = {
  "probe_rows", "gather_pool", "fill_occ_bag", "dedup_tile", "table_lookup", "table_update", "sketch_add", "table_insert", "expand_parts", "order_parts",
  "file_segments", "update_singletons", "reduce_adagrad", "fold_partials", "combine_adagrad",
  "finish_apply", "expire", "stash_trim", "clear_set", "reduce_parts", "adopt_group"
};
static_assert(K_COUNT <= MONO_MAX_KERNELS, "mono_timing_t has room for MONO_MAX_KERNELS kernels");

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
  // An internal stream, ordered against `stream` with events only, runs the sweep.
  cudaStream_t sweep_stream = nullptr;
  // A third one runs the small kernels that serve only the few hottest IDs of a push beside
  // the large ones (see launch_apply).
  cudaStream_t aux_stream = nullptr;
  cudaEvent_t ev_aux = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_keys = nullptr, ev_swept = nullptr, ev_commit = nullptr;
  cudaEvent_t ev_group = nullptr;  // grouped calls: the group's start (first table's), this table's end
  bool sweep_pending = false;     // the sweep stream has work `stream` has not waited for yet
  bool keys_idle = false;         // nothing launched on `stream` after ev_keys touches the key store
  // The batch mono_prepare_push announced: grouped and looked up, waiting for its push.
  // filed: its lookup has run too, so every occurrence's bag is in bag_of_sorted[] already.
  struct { const void* ids; int64_t n_ids; const void* off; int64_t n_bags; bool valid; bool filed; } prep = {nullptr, 0, nullptr, 0, false, false};
  // The batch mono_group_ahead grouped beside the table's other work: a second copy of the scratch
  // that the grouping fills (the per-call set, the per-occurrence records, the list of distinct
  // IDs) and of the per-call counters, which mono_prepare_push of the same batch swaps in.
  struct {
    BatchSlot* bset = nullptr; uint2* occ = nullptr; uint32_t* occ_bag = nullptr;
    unsigned long long* uid = nullptr; uint32_t* uslot = nullptr; uint32_t* uocc = nullptr;
    DevState* st = nullptr;
    const void* ids = nullptr; int64_t n_ids = 0; const void* off = nullptr; int64_t n_bags = 0;
    bool valid = false;           // holds a grouped batch that no mono_prepare_push has taken yet
  } ahead;
  cudaStream_t ahead_stream = nullptr;
  cudaEvent_t ev_ahead = nullptr;   // the grouping on ahead_stream is done
  cudaEvent_t ev_swap = nullptr;    // what `stream` held when mono_group_ahead was called: the batch's arrays are
                                    // ready, and the copy of the scratch handed back at the last exchange is let go of
  uint32_t* occ_row = nullptr;    // scratch of the two-kernel lookup: row of every occurrence
  int device = 0;                 // the device the table lives on
  uint64_t scratch_reallocs = 0;  // times a hot call had to grow the scratch
  // Grouped calls (one launch over several tables): the first table of a group keeps the
  // descriptors of the group's tables and the block maps of its launches, on the device, and
  // a small ring of pinned host copies they are uploaded from.
  struct GroupScratch {
    static constexpr int kRing = 4;
    char* dev = nullptr; size_t dev_bytes = 0;
    char* host[kRing] = {}; size_t host_bytes[kRing] = {}; cudaEvent_t used[kRing] = {};
    int next = 0;
  } grp;
  // device-resident snapshot (mono_snapshot_save)
  struct {
    Cell* cells = nullptr; Cell* stash = nullptr; float* rows = nullptr; uint32_t* free_rows = nullptr;
    uint32_t* oldest = nullptr; DevState* st = nullptr; unsigned int* sketch = nullptr;
    uint64_t key_cells = 0; int64_t last_now = -1, sketch_epoch = 0; bool valid = false;
  } snap;
  int sm_count = 148;
  uint64_t key_cells = 0;
  int64_t last_now = -1;
  int64_t sketch_epoch = 0;       // time the sketch was last cleared
  int64_t max_ids = 0, max_bags = 0;
  // device staging for the host-buffer calls
  unsigned long long* stage_ids = nullptr;
  long long* stage_off = nullptr;
  float* stage_out = nullptr;     // pooled rows on their way to the host
  float* stage_grad = nullptr;    // gradients on their way in
  // The host-buffer calls copy on two streams of their own, one per direction, so that a step's
  // gradients come in while its pooled rows still go out (the link is full duplex) and both
  // run beside the kernels.  ev_staged: the IDs or gradients have arrived; ev_out: the pooled
  // rows are ready to leave; ev_d2h: they have left; ev_stage_free: the kernels are done with
  // the staged inputs.
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  cudaEvent_t ev_staged = nullptr, ev_grad_in = nullptr, ev_out = nullptr, ev_d2h = nullptr, ev_stage_free = nullptr;
  bool d2h_pending = false;       // a copy to the host is in flight that `stream` has not waited for
  bool stage_used = false;        // ev_stage_free has been recorded
  // the host batch whose IDs and offsets are on the device, staged by mono_lookup_pool_host
  struct { const void* ids; int64_t n_ids; const void* off; int64_t n_bags; bool valid; } staged = {nullptr, 0, nullptr, 0, false};
  std::string last_err;
};

namespace {

// A named range around every call of the ABI, for timelines taken with a profiler that reads
// NVTX (a pointer test when none is attached).
struct ApiRange {
  explicit ApiRange(const char* name) { nvtxRangePushA(name); }
  ~ApiRange() { nvtxRangePop(); }
};
#define MONO_API_RANGE() ApiRange api_range__(__func__)

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
  dev_free(w.bset); dev_free(w.occ); dev_free(w.occ_bag); dev_free(w.bag_of_sorted);
  dev_free(w.uid); dev_free(w.uslot); dev_free(w.uocc); dev_free(w.useg); dev_free(w.ulen); dev_free(w.urow); dev_free(w.ucell); dev_free(w.umeta);
  dev_free(w.multi_list); dev_free(w.ins_list); dev_free(w.long_u); dev_free(w.long_part0); dev_free(w.part_u); dev_free(w.part_order); dev_free(w.win_count); dev_free(w.partials); dev_free(w.fold_li); dev_free(w.fold_idx);
  dev_free(t->stage_ids); dev_free(t->stage_off); dev_free(t->stage_out); dev_free(t->stage_grad); dev_free(t->occ_row);
  auto& ah = t->ahead;
  dev_free(ah.bset); dev_free(ah.occ); dev_free(ah.occ_bag); dev_free(ah.uid); dev_free(ah.uslot); dev_free(ah.uocc); dev_free(ah.st);
  ah.valid = false;
  t->staged.valid = false;
  t->max_ids = t->max_bags = 0;
}

void free_snapshot(mono_table* t) {
  auto& sn = t->snap;
  dev_free(sn.cells); dev_free(sn.stash); dev_free(sn.oldest); dev_free(sn.rows); dev_free(sn.free_rows); dev_free(sn.st); dev_free(sn.sketch);
  sn.valid = false;
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
// Launch with programmatic stream serialisation: the launch may be prepared while the kernel
// before it on the stream still runs; every kernel launched this way starts with
// after_previous_kernel(), which waits for that kernel to complete.  What the stream holds
// before it other than a kernel (a copy, an event wait) is waited for in the ordinary way.
template <typename... P, typename... A>
inline void launch_after(void (*kernel)(P...), unsigned grid, unsigned block, cudaStream_t s, A&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(block, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, std::forward<A>(args)...);
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

// Forget a prepared batch: empty the per-call set and the per-call counters.
int discard_prepared(mono_table* t) {
  if (!t->prep.valid) return MONO_OK;
  t->prep.valid = false;
  const uint64_t slots = (uint64_t)t->wk.primary_mask + 1 + (uint64_t)t->wk.secondary_mask + 1;
  init_bset_kernel<<<grid_for(t, 4), 256, 0, t->stream>>>(t->wk.bset, slots);
  finish_apply_kernel<<<1, 256, 0, t->stream>>>(t->tv.st, t->wk.win_count, 0);
  CUDA_TRY(t, cudaGetLastError());
  return MONO_OK;
}

int reserve(mono_table* t, int64_t max_ids, int64_t max_bags) {
  if (max_ids <= t->max_ids && max_bags <= t->max_bags) return MONO_OK;
  if (max_ids < t->max_ids) max_ids = t->max_ids;
  if (max_bags < t->max_bags) max_bags = t->max_bags;
  if (max_ids < 1024) max_ids = 1024;
  if (max_bags < 1024) max_bags = 1024;
  if (t->max_ids > 0) ++t->scratch_reallocs;               // (the first sizing of a table created without one is not a regrowth)
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  if (t->ahead_stream) CUDA_TRY(t, cudaStreamSynchronize(t->ahead_stream));  // a grouping in flight uses the second copy
  if (t->h2d_stream) CUDA_TRY(t, cudaStreamSynchronize(t->h2d_stream));      // copies in flight use the staging buffers
  if (t->d2h_stream) CUDA_TRY(t, cudaStreamSynchronize(t->d2h_stream));
  t->d2h_pending = false;
  // a prepared batch is lost with the scratch it lives in
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
  ALLOC(w.occ, n); ALLOC(w.occ_bag, n); ALLOC(w.bag_of_sorted, n);
  ALLOC(w.uid, n); ALLOC(w.uslot, n); ALLOC(w.uocc, n); ALLOC(w.useg, n); ALLOC(w.ulen, n); ALLOC(w.urow, n); ALLOC(w.ucell, n); ALLOC(w.umeta, n);
  ALLOC(w.multi_list, n / 2 + 1); ALLOC(w.ins_list, n);
  w.max_long = (uint32_t)(n / kSegChunk + 1);
  w.max_parts = (uint32_t)(2 * (n / kSegChunk) + 2);
  ALLOC(w.long_u, w.max_long); ALLOC(w.long_part0, w.max_long); ALLOC(w.part_u, w.max_parts); ALLOC(w.part_order, w.max_parts); ALLOC(w.win_count, 2 * kWindows);
  ALLOC(w.partials, (size_t)w.max_parts * t->tv.dim);
  w.max_folds = w.max_parts / kFoldWidth + w.max_long + 1;
  ALLOC(w.fold_li, w.max_folds); ALLOC(w.fold_idx, w.max_folds);
  ALLOC(t->stage_ids, n); ALLOC(t->stage_off, (size_t)max_bags + 1);
  // (the two staging buffers of the host-buffer calls, one bag-by-dim matrix each, are allocated by the
  // first such call: callers that keep their batches on the device never pay for them)
  ALLOC(t->occ_row, n);
#undef ALLOC
  w.primary_mask = (uint32_t)(primary - 1);
  w.secondary_mask = (uint32_t)(secondary - 1);
  w.max_ids = (uint32_t)max_ids;
  w.n_slots = (uint32_t)slots;
  w.error_bits = &t->tv.st->error_bits;
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

bool is_prepared_batch(const mono_table* t, const void* ids, int64_t n_ids, const void* off, int64_t n_bags) {
  return t->prep.valid && t->prep.ids == ids && t->prep.n_ids == n_ids && t->prep.off == off && t->prep.n_bags == n_bags;
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

// The pooling kernel over the row indices in `occ_row`.
int launch_gather(mono_table* t, const uint32_t* occ_row, int64_t n_ids, const long long* off, int64_t n_bags, float* out) {
  return dispatch_dim(t->tv.dim, [&](auto g, auto nv) -> int {
    constexpr int G = decltype(g)::value, NV = decltype(nv)::value;
    const int64_t groups_per_block = 256 / G;
    int64_t blocks = (n_bags + groups_per_block - 1) / groups_per_block;
    // (two waves of blocks: measured 0.8 % of a step faster on the largest configuration than eight, and 3.5 %
    // faster than one block per 16 bags, although the kernel alone takes the same time)
    const int64_t cap = (int64_t)grid_for(t, 8) * 2;
    if (blocks > cap) blocks = cap;
    LAUNCH(t, K_GATHER, launch_after(gather_pool_kernel<G, NV>, (int)blocks, 256, t->stream, t->tv, occ_row, n_ids, off, n_bags, out));
    CUDA_TRY(t, cudaGetLastError());
    return (int)MONO_OK;
  });
}

int launch_probe(mono_table* t, const unsigned long long* ids, int64_t n_ids, uint32_t* occ_row) {
  if (n_ids <= 0) return MONO_OK;
  int64_t blocks = (n_ids + 255) / 256;
  const int64_t cap = (int64_t)grid_for(t, 8) * 8;
  if (blocks > cap) blocks = cap;
  LAUNCH(t, K_PROBE, launch_after(probe_rows_kernel, (int)blocks, 256, t->stream, t->tv, ids, n_ids, occ_row));
  CUDA_TRY(t, cudaGetLastError());
  return MONO_OK;
}

int launch_lookup(mono_table* t, const unsigned long long* ids, int64_t n_ids, const long long* off,
                  int64_t n_bags, float* out, bool prepared) {
  if (n_bags == 0) return MONO_OK;
  if (prepared && n_ids > 0) {
    // every distinct ID of this batch was looked up when it was announced: one pass over the
    // occurrences takes the rows from the per-call set and files the bags for the push
    LAUNCH(t, K_FILE, launch_after(file_segments_kernel, grid_for(t, 8), 256, t->stream, t->wk, n_ids, n_bags, t->occ_row,
                                                                                  (uint32_t)t->tv.capacity));
    t->prep.filed = true;
  } else {
    const int rc = launch_probe(t, ids, n_ids, t->occ_row);
    if (rc != MONO_OK) return rc;
  }
  return launch_gather(t, t->occ_row, n_ids, off, n_bags, out);
}

// The part of a push that depends on the IDs alone: bag of every occurrence, and the
// occurrences grouped by ID in the per-call set.
int launch_group(mono_table* t, cudaStream_t s, const unsigned long long* ids, int64_t n_ids, const long long* off,
                 int64_t n_bags, const Work* into = nullptr, DevState* counters = nullptr) {
  const TableView& tv = t->tv;
  const Work& wk = into ? *into : t->wk;
  DevState* st = counters ? counters : tv.st;
  LAUNCH_ON(t, s, K_FILL_BAG, launch_after(fill_occ_bag_kernel, grid_for(t, 8), 256, s, off, n_bags, n_ids, wk.occ_bag, st));
  const int tiles = (int)((n_ids + kTileIds - 1) / kTileIds);
  LAUNCH_ON(t, s, K_DEDUP, launch_after(dedup_tile_kernel, tiles, kTileThreads, s, wk, ids, n_ids, off, n_bags, st,
                                                                          tv.seed0 ^ 0xA5A5A5A55A5A5A5Aull));
  CUDA_TRY(t, cudaGetLastError());
  return MONO_OK;
}

// mono_prepare_push: group the batch and look every distinct ID up once, for the lookup and the
// push of this batch together.  Nothing in the table changes.
int launch_prepare(mono_table* t, const unsigned long long* ids, int64_t n_ids, const long long* off, int64_t n_bags) {
  auto& ah = t->ahead;
  if (ah.valid && ah.ids == ids && ah.n_ids == n_ids && ah.off == off && ah.n_bags == n_bags) {
    // grouped already, beside the table's other work: the two copies of the grouping scratch change
    // places, and the counters the grouping left come over
    ah.valid = false;
    CUDA_TRY(t, cudaStreamWaitEvent(t->stream, t->ev_ahead, 0));        // (recorded when the grouping ran on a stream of its own)
    Work& w = t->wk;
    std::swap(w.bset, ah.bset); std::swap(w.occ, ah.occ); std::swap(w.occ_bag, ah.occ_bag);
    std::swap(w.uid, ah.uid); std::swap(w.uslot, ah.uslot); std::swap(w.uocc, ah.uocc);
    LAUNCH(t, K_ADOPT, launch_after(adopt_group_kernel, 1, 32, t->stream, t->tv.st, ah.st));
    CUDA_TRY(t, cudaGetLastError());
  } else {
    const int rc = launch_group(t, t->stream, ids, n_ids, off, n_bags);
    if (rc != MONO_OK) return rc;
  }
  LAUNCH(t, K_LOOKUP, launch_after(table_update_kernel<kLookUp>, grid_for(t, 8) * 4, 256, t->stream, t->tv, t->wk, 0u));
  CUDA_TRY(t, cudaGetLastError());
  return MONO_OK;
}

// grad_ready: if not null, the gradients are still being copied in; the kernels that read them wait for it
int launch_apply(mono_table* t, const unsigned long long* ids, int64_t n_ids, const long long* off,
                 int64_t n_bags, const float* grad, uint32_t now, cudaEvent_t grad_ready = nullptr) {
  cudaStream_t s = t->stream;
  const TableView& tv = t->tv;
  const Work& wk = t->wk;
  // grids of the grid-stride kernels: several waves of blocks per SM where that measured faster
  // (shorter tails), one wave elsewhere.  The reduction of the short segments runs beside the long
  // segments' chain and the insertions: with four waves of blocks instead of eight the step measured
  // 1.9 % faster on the largest configuration (its own time is the same); the parts launch and
  // update_singletons keep eight.
  const int g4 = grid_for(t, 4), g8 = grid_for(t, 8);
  int rc0 = MONO_OK;
  if (is_prepared_batch(t, ids, n_ids, off, n_bags)) {
    // grouped and looked up already; filed too, if its lookup has run
    t->prep.valid = false;
    if (!t->prep.filed) LAUNCH(t, K_FILE, launch_after(file_segments_kernel, g8, 256, s, wk, n_ids, n_bags, nullptr, 0u));
    LAUNCH(t, K_UPDATE, launch_after(table_update_kernel<kCommit>, g8 * 4, 256, s, tv, wk, now));
  } else {
    if ((rc0 = discard_prepared(t)) != MONO_OK) return rc0;
    if (n_ids == 0 || n_bags == 0) return MONO_OK;
    if ((rc0 = launch_group(t, s, ids, n_ids, off, n_bags)) != MONO_OK) return rc0;
    LAUNCH(t, K_UPDATE, launch_after(table_update_kernel<kLookUp | kCommit>, g8 * 4, 256, s, tv, wk, now));
    LAUNCH(t, K_FILE, launch_after(file_segments_kernel, g8, 256, s, wk, n_ids, n_bags, nullptr, 0u));
  }
  // The long segments (the few hottest IDs) are reduced on a stream of their own -- expand,
  // order, the parts, fold, combine, one after the other with no event in between -- beside
  // the kernels that work through the rest of the batch on the table's stream: the reduction
  // of the short segments and update_singletons.  The two chains touch different rows and meet
  // again before the call's last kernel (measured 0.9 % of a step faster than the parts on the
  // table's stream between two event waits).  With the exact filter the insertion of the new
  // IDs runs on a third stream beside both: their rows were settled by the commit half, so the
  // row updates do not wait for it.  With the probabilistic filter it is the insertion that
  // decides the rows, and it stays on the table's stream.
  // While kernels are being timed one by one, everything stays on the table's stream.
  cudaStream_t a = t->timing ? s : t->aux_stream;
  const bool insert_aside = a != s && tv.sketch_depth == 0;
  if (insert_aside) {
    // (on the stream the sweep uses: a sweep slice that follows this call follows the insertions)
    cudaStream_t k = t->sweep_stream;
    CUDA_TRY(t, cudaEventRecord(t->ev_commit, s));
    CUDA_TRY(t, cudaStreamWaitEvent(k, t->ev_commit, 0));
    CUDA_TRY(t, cudaStreamWaitEvent(a, t->ev_commit, 0));
    LAUNCH_ON(t, k, K_INSERT, launch_after(table_insert_kernel, g8, 256, k, tv, wk, now));
    CUDA_TRY(t, cudaGetLastError());
    // the rest of the call touches rows and scratch only: a sweep may run beside it
    CUDA_TRY(t, cudaEventRecord(t->ev_keys, k));
  } else {
    if (tv.sketch_depth) LAUNCH(t, K_SKETCH, launch_after(sketch_add_kernel, g8, 256, s, tv, wk));
    LAUNCH(t, K_INSERT, launch_after(table_insert_kernel, g8, 256, s, tv, wk, now));
    CUDA_TRY(t, cudaGetLastError());
    CUDA_TRY(t, cudaEventRecord(t->ev_keys, s));
    if (a != s) CUDA_TRY(t, cudaStreamWaitEvent(a, t->ev_keys, 0));
  }
  // (nobody reads the per-call set after the key-store work: its primary tier is wiped beside the rest)
  LAUNCH_ON(t, a, K_CLEAR, launch_after(clear_primary_kernel, g8, 256, a, wk));
  LAUNCH_ON(t, a, K_EXPAND, launch_after(expand_parts_kernel, g8 * 4, 128, a, tv, wk));
  LAUNCH_ON(t, a, K_ORDER, launch_after(order_parts_kernel, 64, kWindows, a, tv, wk));
  CUDA_TRY(t, cudaGetLastError());
  if (grad_ready) CUDA_TRY(t, cudaStreamWaitEvent(s, grad_ready, 0));
  const int rc = dispatch_dim(tv.dim, [&](auto g, auto nv) -> int {
    constexpr int G = decltype(g)::value, NV = decltype(nv)::value;
    LAUNCH(t, K_REDUCE, launch_after(reduce_adagrad_kernel<G, NV>, g8 * 4, 128, s, tv, wk, grad, n_bags, kReduceShort));
    if (grad_ready && a != s) CUDA_TRY(t, cudaStreamWaitEvent(a, grad_ready, 0));
    LAUNCH_ON(t, a, K_REDUCE_PARTS, launch_after(reduce_adagrad_kernel<G, NV>, g8 * 8, 128, a, tv, wk, grad, n_bags, kReduceParts));
    LAUNCH(t, K_SINGLES, launch_after(update_singletons_kernel<G, NV>, g8 * 8, 128, s, tv, wk, grad, n_bags));
    return (int)MONO_OK;
  });
  if (rc != MONO_OK) return rc;
  LAUNCH_ON(t, a, K_FOLD, launch_after(fold_partials_kernel, g4, 256, a, tv, wk));
  LAUNCH_ON(t, a, K_COMBINE, launch_after(combine_adagrad_kernel, g8, kCombineThreads, a, tv, wk));
  if (a != s) {
    CUDA_TRY(t, cudaEventRecord(t->ev_aux, a));
    CUDA_TRY(t, cudaStreamWaitEvent(s, t->ev_aux, 0));
  }
  if (insert_aside) CUDA_TRY(t, cudaStreamWaitEvent(s, t->ev_keys, 0));
  LAUNCH(t, K_FINISH, launch_after(finish_apply_kernel, 1, 256, s, tv.st, wk.win_count, 1));
  CUDA_TRY(t, cudaGetLastError());
  t->keys_idle = true;
  return MONO_OK;
}

int check_now(mono_table* t, int64_t now) {
  if (now < 0 || now > MONO_MAX_NOW || now < t->last_now) return MONO_ERR_TIME;
  return MONO_OK;
}

// ---- grouped calls: one launch over several tables -------------------------------------------

enum GroupKernel {
  GK_FILL, GK_DEDUP, GK_UPDATE, GK_INSERT, GK_FILE, GK_EXPAND, GK_ORDER, GK_GATHER, GK_GATHER_WIDE, GK_REDUCE, GK_REDUCE_WIDE,
  GK_SINGLES, GK_SINGLES_WIDE, GK_FOLD, GK_COMBINE, GK_CLEAR, GK_COUNT
};

uint32_t lane_class_of(uint32_t dim) {
  return dim <= 16 ? 0u : dim <= 32 ? 1u : dim <= 64 ? 2u : dim <= 128 ? 3u : dim <= 256 ? 4u : dim <= 512 ? 5u : 6u;
}
int lanes_of_class(uint32_t c) { return c == 0 ? 4 : c == 1 ? 8 : c == 2 ? 16 : 32; }

void free_group_scratch(mono_table* t) {
  auto& g = t->grp;
  if (g.dev) { cudaFree(g.dev); g.dev = nullptr; g.dev_bytes = 0; }
  for (int i = 0; i < mono_table::GroupScratch::kRing; ++i) {
    if (g.host[i]) { cudaFreeHost(g.host[i]); g.host[i] = nullptr; g.host_bytes[i] = 0; }
    if (g.used[i]) { cudaEventDestroy(g.used[i]); g.used[i] = nullptr; }
  }
}

int64_t clamp_blocks(int64_t work, int64_t per_block, int64_t cap) {
  int64_t b = (work + per_block - 1) / per_block;
  if (b < 1) b = 1;
  return b > cap ? cap : b;
}

// Blocks that table `t` contributes to grouped kernel `k` (the grid it would launch alone, but no
// larger than its batch needs: a group may hold hundreds of small tables).
uint32_t group_blocks(const mono_table* t, int k, int64_t n_ids, int64_t n_bags) {
  const int64_t g8 = grid_for(t, 8), g4 = grid_for(t, 4);
  const uint32_t lc = lane_class_of(t->tv.dim);
  const int G = lanes_of_class(lc);
  const bool wide = lc >= 4;
  switch (k) {
    case GK_FILL: return (uint32_t)clamp_blocks(n_bags, 256, g8);
    case GK_DEDUP: return (uint32_t)((n_ids + kTileIds - 1) / kTileIds);
    case GK_UPDATE: return (uint32_t)clamp_blocks(n_ids, 256, g8 * 4);
    case GK_INSERT: case GK_FILE: return (uint32_t)clamp_blocks(n_ids, 256, g8);
    case GK_EXPAND: return (uint32_t)clamp_blocks(n_ids / kSegChunk + 1, 1, g8 * 4);
    case GK_ORDER: return (uint32_t)clamp_blocks(n_ids / kSegChunk + 1, kWindows, 64);
    case GK_GATHER: return wide ? 0u : (uint32_t)clamp_blocks(n_bags, 256 / G, g8 * 8);
    case GK_GATHER_WIDE: return wide ? (uint32_t)clamp_blocks(n_bags, 256 / G, g8 * 8) : 0u;
    case GK_REDUCE: return wide ? 0u : (uint32_t)clamp_blocks(n_ids / 2 + 1, 128 / G, g8 * 8);
    case GK_REDUCE_WIDE: return wide ? (uint32_t)clamp_blocks(n_ids / 2 + 1, 128 / G, g8 * 8) : 0u;
    case GK_SINGLES: return wide ? 0u : (uint32_t)clamp_blocks(n_ids, 128, g8 * 8);
    case GK_SINGLES_WIDE: return wide ? (uint32_t)clamp_blocks(n_ids, 128, g8 * 8) : 0u;
    case GK_FOLD: return (uint32_t)clamp_blocks(n_ids / (kSegChunk * kFoldWidth) + 1, 1, g4);
    case GK_COMBINE: return (uint32_t)clamp_blocks(n_ids / kSegChunk + 1, 1, g8);
    case GK_CLEAR: return (uint32_t)clamp_blocks((int64_t)t->wk.primary_mask + 1, 2048, g8);
    default: return 0u;
  }
}

// A grouped call in the making: the tables' descriptors, the block map of every kernel, and where
// both live on the device once uploaded.
struct GroupPlan {
  int32_t n = 0;
  mono_table* owner = nullptr;               // tables[0]: holds the scratch and counts the launches
  cudaStream_t gs = nullptr;
  std::vector<GroupItem> items;
  std::vector<uint32_t> starts;              // [GK_COUNT][n + 1]
  const GroupItem* d_items = nullptr;
  const uint32_t* d_starts = nullptr;
  bool any_wide = false, any_narrow = false, any_sketch = false;
  uint32_t grid(int k) const { return starts[(size_t)k * (n + 1) + n]; }
  const uint32_t* map(int k) const { return d_starts + (size_t)k * (n + 1); }
};

int group_check(int32_t n_tables, mono_table* const* tables) {
  if (n_tables < 0 || (n_tables > 0 && !tables)) return MONO_ERR_ARG;
  for (int32_t i = 0; i < n_tables; ++i) {
    if (!tables[i]) return MONO_ERR_ARG;
    if (tables[i]->device != tables[0]->device) return MONO_ERR_ARG;
  }
  // the same table twice would run two batches through one scratch at the same time
  std::vector<mono_table*> sorted(tables, tables + n_tables);
  std::sort(sorted.begin(), sorted.end());
  for (int32_t i = 1; i < n_tables; ++i) if (sorted[i] == sorted[i - 1]) return MONO_ERR_ARG;
  return MONO_OK;
}

// Everything the tables have in flight on their own streams comes before the group's work on `gs`.
int group_begin(GroupPlan& p, int32_t n_tables, mono_table* const* tables, void* group_stream) {
  p.n = n_tables;
  p.owner = tables[0];
  p.gs = static_cast<cudaStream_t>(group_stream);
  for (int32_t i = 0; i < n_tables; ++i) {
    mono_table* t = tables[i];
    join_sweep(t);
    if (t->stream != p.gs) {
      CUDA_TRY(t, cudaEventRecord(t->ev_group, t->stream));
      CUDA_TRY(t, cudaStreamWaitEvent(p.gs, t->ev_group, 0));
    }
  }
  p.items.assign(n_tables, GroupItem{});
  p.starts.assign((size_t)GK_COUNT * (n_tables + 1), 0u);
  return MONO_OK;
}

// ... and whatever the tables are given next on their own streams comes after it.
int group_end(GroupPlan& p, mono_table* const* tables) {
  bool other = false;
  for (int32_t i = 0; i < p.n; ++i) other |= tables[i]->stream != p.gs;
  if (!other) return MONO_OK;
  CUDA_TRY(p.owner, cudaEventRecord(p.owner->ev_fork, p.gs));
  for (int32_t i = 0; i < p.n; ++i)
    if (tables[i]->stream != p.gs) CUDA_TRY(tables[i], cudaStreamWaitEvent(tables[i]->stream, p.owner->ev_fork, 0));
  return MONO_OK;
}

void group_describe(GroupPlan& p, int32_t i, mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* off,
                    int64_t n_bags, float* out, const float* grad, uint32_t now, bool prepared) {
  GroupItem& it = p.items[i];
  it.tv = t->tv; it.wk = t->wk;
  it.ids = reinterpret_cast<const unsigned long long*>(ids);
  it.off = reinterpret_cast<const long long*>(off);
  it.n_ids = n_ids; it.n_bags = n_bags; it.out = out; it.grad = grad; it.now = now;
  it.occ_row = t->occ_row;
  it.dedup_seed = t->tv.seed0 ^ 0xA5A5A5A55A5A5A5Aull;
  it.prepared = prepared ? 1u : 0u;
  it.lane_class = lane_class_of(t->tv.dim);
  it.active = (n_ids > 0 && n_bags > 0) ? 1u : 0u;
  if (it.lane_class >= 4) p.any_wide = true; else p.any_narrow = true;
  if (t->tv.sketch_depth) p.any_sketch = true;
}

// Block maps (a table whose batch is empty gets no blocks), then one upload of descriptors and maps.
int group_upload(GroupPlan& p, mono_table* const* tables) {
  for (int k = 0; k < GK_COUNT; ++k) {
    uint32_t* st = p.starts.data() + (size_t)k * (p.n + 1);
    uint64_t total = 0;
    for (int32_t i = 0; i < p.n; ++i) {
      st[i] = (uint32_t)total;
      if (p.items[i].active) total += group_blocks(tables[i], k, p.items[i].n_ids, p.items[i].n_bags);
      if (total >= (1ull << 31)) return MONO_ERR_ARG;
    }
    st[p.n] = (uint32_t)total;
  }
  auto& g = p.owner->grp;
  const size_t items_bytes = ((p.items.size() * sizeof(GroupItem) + 255) / 256) * 256;
  const size_t bytes = items_bytes + p.starts.size() * sizeof(uint32_t);
  if (bytes > g.dev_bytes) {
    CUDA_TRY(p.owner, cudaStreamSynchronize(p.gs));
    if (g.dev) cudaFree(g.dev);
    g.dev = nullptr; g.dev_bytes = 0;
    CUDA_TRY(p.owner, cudaMalloc(reinterpret_cast<void**>(&g.dev), bytes * 2));
    g.dev_bytes = bytes * 2;
  }
  const int slot = g.next;
  g.next = (g.next + 1) % mono_table::GroupScratch::kRing;
  if (!g.used[slot]) CUDA_TRY(p.owner, cudaEventCreateWithFlags(&g.used[slot], cudaEventDisableTiming));
  else CUDA_TRY(p.owner, cudaEventSynchronize(g.used[slot]));          // the upload that last used this host copy is done
  if (bytes > g.host_bytes[slot]) {
    if (g.host[slot]) cudaFreeHost(g.host[slot]);
    g.host[slot] = nullptr; g.host_bytes[slot] = 0;
    CUDA_TRY(p.owner, cudaMallocHost(reinterpret_cast<void**>(&g.host[slot]), bytes * 2));
    g.host_bytes[slot] = bytes * 2;
  }
  std::memcpy(g.host[slot], p.items.data(), p.items.size() * sizeof(GroupItem));
  std::memcpy(g.host[slot] + items_bytes, p.starts.data(), p.starts.size() * sizeof(uint32_t));
  CUDA_TRY(p.owner, cudaMemcpyAsync(g.dev, g.host[slot], bytes, cudaMemcpyHostToDevice, p.gs));
  CUDA_TRY(p.owner, cudaEventRecord(g.used[slot], p.gs));
  p.d_items = reinterpret_cast<const GroupItem*>(g.dev);
  p.d_starts = reinterpret_cast<const uint32_t*>(g.dev + items_bytes);
  return MONO_OK;
}

// launch grouped kernel `kernel` over block map `gk` with `threads` per block, counted under `kid`
#define GROUP_LAUNCH(p, kid, gk, threads, kernel)                                                         \
  do {                                                                                                    \
    if ((p).grid(gk) > 0) {                                                                               \
      ++(p).owner->launches[kid];                                                                         \
      launch_after(kernel, (p).grid(gk), (threads), (p).gs, (p).d_items, (p).map(gk), (uint32_t)(p).n);    \
    }                                                                                                     \
  } while (0)

int group_launch_ids_only(GroupPlan& p) {
  GROUP_LAUNCH(p, K_FILL_BAG, GK_FILL, 256, group_fill_occ_bag_kernel);
  GROUP_LAUNCH(p, K_DEDUP, GK_DEDUP, kTileThreads, group_dedup_tile_kernel);
  return MONO_OK;
}

}  // namespace

extern "C" {

int mono_table_create(mono_table** out, uint64_t capacity, uint32_t dim, uint32_t filter_threshold,
                      uint32_t ttl, const mono_opt* opt, void* cuda_stream) {
  MONO_API_RANGE();
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
  t->device = dev;
  if (cudaStreamCreateWithFlags(&t->sweep_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaStreamCreateWithFlags(&t->aux_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaStreamCreateWithFlags(&t->ahead_stream, cudaStreamNonBlocking) != cudaSuccess)
    return fail(MONO_ERR_CUDA);
  for (cudaEvent_t* e : {&t->ev_fork, &t->ev_keys, &t->ev_swept, &t->ev_group, &t->ev_aux, &t->ev_commit, &t->ev_ahead, &t->ev_swap})
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
  if ((rc = dev_alloc(t, &tv.oldest, key_cells / kCellsPerBucket)) != MONO_OK) return fail(rc);
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
  MONO_API_RANGE();
  if (!t) return MONO_ERR_ARG;
  cudaStreamSynchronize(t->stream);
  if (t->sweep_stream) { cudaStreamSynchronize(t->sweep_stream); cudaStreamDestroy(t->sweep_stream); }
  if (t->aux_stream) { cudaStreamSynchronize(t->aux_stream); cudaStreamDestroy(t->aux_stream); }
  if (t->ahead_stream) { cudaStreamSynchronize(t->ahead_stream); cudaStreamDestroy(t->ahead_stream); }
  if (t->h2d_stream) { cudaStreamSynchronize(t->h2d_stream); cudaStreamDestroy(t->h2d_stream); }
  if (t->d2h_stream) { cudaStreamSynchronize(t->d2h_stream); cudaStreamDestroy(t->d2h_stream); }
  for (cudaEvent_t e : {t->ev_staged, t->ev_grad_in, t->ev_out, t->ev_d2h, t->ev_stage_free}) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : {t->ev_fork, t->ev_keys, t->ev_swept, t->ev_group, t->ev_aux, t->ev_commit, t->ev_ahead, t->ev_swap})
    if (e) cudaEventDestroy(e);
  for (auto& p : t->pending) { cudaEventDestroy(p.second.first); cudaEventDestroy(p.second.second); }
  for (cudaEvent_t e : t->spare_events) cudaEventDestroy(e);
  free_scratch(t);
  free_snapshot(t);
  free_group_scratch(t);
  dev_free(t->tv.cells); dev_free(t->tv.stash); dev_free(t->tv.oldest); dev_free(t->tv.rows); dev_free(t->tv.free_rows); dev_free(t->tv.st); dev_free(t->tv.sketch);
  delete t;
  return MONO_OK;
}

int mono_reserve(mono_table* t, int64_t max_ids, int64_t max_bags) {
  MONO_API_RANGE();
  if (t) join_sweep(t);
  if (!t || max_ids < 0 || max_bags < 0 || max_ids >= (1ll << 31) || max_bags >= (1ll << 31)) return MONO_ERR_ARG;
  return reserve(t, max_ids, max_bags);
}

int mono_lookup_pool(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                     int64_t n_bags, float* out) {
  MONO_API_RANGE();
  if (t) join_sweep(t);
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if (n_bags > 0 && (!out || !aligned(out, 16))) return MONO_ERR_ARG;
  if ((rc = reserve(t, n_ids, n_bags)) != MONO_OK) return rc;
  return launch_lookup(t, reinterpret_cast<const unsigned long long*>(ids), n_ids,
                       reinterpret_cast<const long long*>(slot_offsets), n_bags, out,
                       is_prepared_batch(t, ids, n_ids, slot_offsets, n_bags));
}

int mono_apply_grads(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                     int64_t n_bags, const float* grad_pooled, int64_t now) {
  MONO_API_RANGE();
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

int mono_group_ahead(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets, int64_t n_bags) {
  MONO_API_RANGE();
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if ((rc = reserve(t, n_ids, n_bags)) != MONO_OK) return rc;
  auto& ah = t->ahead;
  // while kernels are being timed one by one, the grouping runs on the table's stream like everything else
  cudaStream_t g = t->timing ? t->stream : t->ahead_stream;
  const Work& w = t->wk;
  const uint64_t slots = (uint64_t)w.primary_mask + 1 + (uint64_t)w.secondary_mask + 1;
  // The grouping follows what the table's stream holds so far: whatever fills the batch's arrays,
  // and the kernels that still use the copy of the scratch handed back at the last exchange.
  if (g != t->stream) {
    CUDA_TRY(t, cudaEventRecord(t->ev_swap, t->stream));
    CUDA_TRY(t, cudaStreamWaitEvent(g, t->ev_swap, 0));
  }
  if (!ah.bset) {
    // the second copy of what the grouping fills, sized like the first
    const size_t n = (size_t)t->max_ids;
    int arc = dev_alloc(t, &ah.bset, slots);
    if (arc == MONO_OK) arc = dev_alloc(t, &ah.occ, n);
    if (arc == MONO_OK) arc = dev_alloc(t, &ah.occ_bag, n);
    if (arc == MONO_OK) arc = dev_alloc(t, &ah.uid, n);
    if (arc == MONO_OK) arc = dev_alloc(t, &ah.uslot, n);
    if (arc == MONO_OK) arc = dev_alloc(t, &ah.uocc, n);
    if (arc == MONO_OK) arc = dev_alloc(t, &ah.st, 1);
    if (arc != MONO_OK) {
      dev_free(ah.bset); dev_free(ah.occ); dev_free(ah.occ_bag); dev_free(ah.uid); dev_free(ah.uslot); dev_free(ah.uocc); dev_free(ah.st);
      return arc;
    }
    init_bset_kernel<<<grid_for(t, 4), 256, 0, g>>>(ah.bset, slots);
    CUDA_TRY(t, cudaGetLastError());
    CUDA_TRY(t, cudaMemsetAsync(ah.st, 0, sizeof(DevState), g));
    ah.valid = false;
  }
  if (ah.valid) {
    // a batch grouped earlier that was never pushed: forget it
    ah.valid = false;
    init_bset_kernel<<<grid_for(t, 4), 256, 0, g>>>(ah.bset, slots);
    CUDA_TRY(t, cudaGetLastError());
    CUDA_TRY(t, cudaMemsetAsync(ah.st, 0, sizeof(DevState), g));
  }
  if (n_ids == 0 || n_bags == 0) return MONO_OK;
  Work into = w;
  into.bset = ah.bset; into.occ = ah.occ; into.occ_bag = ah.occ_bag; into.uid = ah.uid; into.uslot = ah.uslot; into.uocc = ah.uocc;
  if ((rc = launch_group(t, g, reinterpret_cast<const unsigned long long*>(ids), n_ids,
                         reinterpret_cast<const long long*>(slot_offsets), n_bags, &into, ah.st)) != MONO_OK) return rc;
  if (g != t->stream) CUDA_TRY(t, cudaEventRecord(t->ev_ahead, g));
  ah.ids = ids; ah.n_ids = n_ids; ah.off = slot_offsets; ah.n_bags = n_bags;
  ah.valid = true;
  return MONO_OK;
}

int mono_prepare_push(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets, int64_t n_bags) {
  MONO_API_RANGE();
  if (t) join_sweep(t);                                    // the look-ups read the key store
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if ((rc = reserve(t, n_ids, n_bags)) != MONO_OK) return rc;
  if ((rc = discard_prepared(t)) != MONO_OK) return rc;
  if (n_ids == 0 || n_bags == 0) return MONO_OK;
  if ((rc = launch_prepare(t, reinterpret_cast<const unsigned long long*>(ids), n_ids,
                           reinterpret_cast<const long long*>(slot_offsets), n_bags)) != MONO_OK) return rc;
  t->prep = {ids, n_ids, slot_offsets, n_bags, true, false};
  return MONO_OK;
}

int mono_group_prepare_push(int32_t n_tables, mono_table* const* tables, const uint64_t* const* ids,
                            const int64_t* n_ids, const int64_t* const* slot_offsets, const int64_t* n_bags,
                            void* group_stream) {
  MONO_API_RANGE();
  int rc = group_check(n_tables, tables);
  if (rc != MONO_OK) return rc;
  if (n_tables == 0) return MONO_OK;
  if (!ids || !n_ids || !slot_offsets || !n_bags) return MONO_ERR_ARG;
  for (int32_t i = 0; i < n_tables; ++i) {
    mono_table* t = tables[i];
    join_sweep(t);
    if ((rc = check_batch(t, ids[i], n_ids[i], slot_offsets[i], n_bags[i])) != MONO_OK) return rc;
    if ((rc = reserve(t, n_ids[i], n_bags[i])) != MONO_OK) return rc;
    if ((rc = discard_prepared(t)) != MONO_OK) return rc;
  }
  GroupPlan p;
  if ((rc = group_begin(p, n_tables, tables, group_stream)) != MONO_OK) return rc;
  for (int32_t i = 0; i < n_tables; ++i)
    group_describe(p, i, tables[i], ids[i], n_ids[i], slot_offsets[i], n_bags[i], nullptr, nullptr, 0u, false);
  if ((rc = group_upload(p, tables)) != MONO_OK) return rc;
  group_launch_ids_only(p);
  GROUP_LAUNCH(p, K_LOOKUP, GK_UPDATE, 256, group_table_update_kernel<kLookUp>);
  CUDA_TRY(p.owner, cudaGetLastError());
  for (int32_t i = 0; i < n_tables; ++i)
    if (p.items[i].active) tables[i]->prep = {ids[i], n_ids[i], slot_offsets[i], n_bags[i], true, false};
  return group_end(p, tables);
}

int mono_group_lookup_pool(int32_t n_tables, mono_table* const* tables, const uint64_t* const* ids,
                           const int64_t* n_ids, const int64_t* const* slot_offsets, const int64_t* n_bags,
                           float* const* out, void* group_stream) {
  MONO_API_RANGE();
  int rc = group_check(n_tables, tables);
  if (rc != MONO_OK) return rc;
  if (n_tables == 0) return MONO_OK;
  if (!ids || !n_ids || !slot_offsets || !n_bags || !out) return MONO_ERR_ARG;
  for (int32_t i = 0; i < n_tables; ++i) {
    mono_table* t = tables[i];
    join_sweep(t);
    if ((rc = check_batch(t, ids[i], n_ids[i], slot_offsets[i], n_bags[i])) != MONO_OK) return rc;
    if (n_bags[i] > 0 && (!out[i] || !aligned(out[i], 16))) return MONO_ERR_ARG;
    if ((rc = reserve(t, n_ids[i], n_bags[i])) != MONO_OK) return rc;
  }
  GroupPlan p;
  if ((rc = group_begin(p, n_tables, tables, group_stream)) != MONO_OK) return rc;
  for (int32_t i = 0; i < n_tables; ++i) {
    group_describe(p, i, tables[i], ids[i], n_ids[i], slot_offsets[i], n_bags[i], out[i], nullptr, 0u,
                   is_prepared_batch(tables[i], ids[i], n_ids[i], slot_offsets[i], n_bags[i]));
    p.items[i].active = n_bags[i] > 0 ? 1u : 0u;           // a bag without IDs still pools to zeros
  }
  if ((rc = group_upload(p, tables)) != MONO_OK) return rc;
  bool any_prepared = false;
  for (int32_t i = 0; i < n_tables; ++i) any_prepared |= p.items[i].prepared && p.items[i].n_ids > 0;
  bool any_unprepared = false;
  for (int32_t i = 0; i < n_tables; ++i) any_unprepared |= !p.items[i].prepared && p.items[i].n_ids > 0;
  // (each of the two passes skips the other kind of table)
  if (any_prepared) GROUP_LAUNCH(p, K_FILE, GK_FILE, 256, group_file_rows_kernel);
  if (any_unprepared) GROUP_LAUNCH(p, K_PROBE, GK_FILE, 256, group_probe_rows_kernel);
  GROUP_LAUNCH(p, K_GATHER, GK_GATHER, 256, group_gather_pool_kernel<0>);
  GROUP_LAUNCH(p, K_GATHER, GK_GATHER_WIDE, 256, group_gather_pool_kernel<1>);
  CUDA_TRY(p.owner, cudaGetLastError());
  for (int32_t i = 0; i < n_tables; ++i)
    if (p.items[i].prepared && p.items[i].n_ids > 0) tables[i]->prep.filed = true;
  return group_end(p, tables);
}

int mono_group_apply_grads(int32_t n_tables, mono_table* const* tables, const uint64_t* const* ids,
                           const int64_t* n_ids, const int64_t* const* slot_offsets, const int64_t* n_bags,
                           const float* const* grad_pooled, int64_t now, void* group_stream) {
  MONO_API_RANGE();
  int rc = group_check(n_tables, tables);
  if (rc != MONO_OK) return rc;
  if (n_tables == 0) return MONO_OK;
  if (!ids || !n_ids || !slot_offsets || !n_bags || !grad_pooled) return MONO_ERR_ARG;
  bool all_prepared = true, all_filed = true;
  for (int32_t i = 0; i < n_tables; ++i) {
    mono_table* t = tables[i];
    join_sweep(t);
    if ((rc = check_batch(t, ids[i], n_ids[i], slot_offsets[i], n_bags[i])) != MONO_OK) return rc;
    if (n_bags[i] > 0 && (!grad_pooled[i] || !aligned(grad_pooled[i], 16))) return MONO_ERR_ARG;
    if ((rc = check_now(t, now)) != MONO_OK) return rc;
    if ((rc = reserve(t, n_ids[i], n_bags[i])) != MONO_OK) return rc;
    if (n_ids[i] == 0 || n_bags[i] == 0) continue;
    const bool prepared = is_prepared_batch(t, ids[i], n_ids[i], slot_offsets[i], n_bags[i]);
    all_prepared &= prepared;
    all_filed &= prepared && t->prep.filed;
  }
  // either every table's batch was announced, or the group is pushed as if none had been
  for (int32_t i = 0; i < n_tables; ++i) {
    mono_table* t = tables[i];
    const bool empty = n_ids[i] == 0 || n_bags[i] == 0;
    if ((!all_prepared || empty) && (rc = discard_prepared(t)) != MONO_OK) return rc;
    t->last_now = now;
  }
  GroupPlan p;
  if ((rc = group_begin(p, n_tables, tables, group_stream)) != MONO_OK) return rc;
  for (int32_t i = 0; i < n_tables; ++i)
    group_describe(p, i, tables[i], ids[i], n_ids[i], slot_offsets[i], n_bags[i], nullptr, grad_pooled[i], (uint32_t)now, all_prepared);
  if ((rc = group_upload(p, tables)) != MONO_OK) return rc;
  if (all_prepared) {
    if (!all_filed) GROUP_LAUNCH(p, K_FILE, GK_FILE, 256, group_file_segments_kernel);
    GROUP_LAUNCH(p, K_UPDATE, GK_UPDATE, 256, group_table_update_kernel<kCommit>);
  } else {
    group_launch_ids_only(p);
    GROUP_LAUNCH(p, K_UPDATE, GK_UPDATE, 256, group_table_update_kernel<kLookUp | kCommit>);
    GROUP_LAUNCH(p, K_FILE, GK_FILE, 256, group_file_segments_kernel);
  }
  if (p.any_sketch) GROUP_LAUNCH(p, K_SKETCH, GK_INSERT, 256, group_sketch_add_kernel);
  GROUP_LAUNCH(p, K_INSERT, GK_INSERT, 256, group_table_insert_kernel);
  GROUP_LAUNCH(p, K_CLEAR, GK_CLEAR, 256, group_clear_primary_kernel);
  GROUP_LAUNCH(p, K_EXPAND, GK_EXPAND, 128, group_expand_parts_kernel);
  GROUP_LAUNCH(p, K_ORDER, GK_ORDER, kWindows, group_order_parts_kernel);
  GROUP_LAUNCH(p, K_REDUCE, GK_REDUCE, 128, group_reduce_adagrad_kernel<0>);
  GROUP_LAUNCH(p, K_REDUCE, GK_REDUCE_WIDE, 128, group_reduce_adagrad_kernel<1>);
  GROUP_LAUNCH(p, K_SINGLES, GK_SINGLES, 128, group_update_singletons_kernel<0>);
  GROUP_LAUNCH(p, K_SINGLES, GK_SINGLES_WIDE, 128, group_update_singletons_kernel<1>);
  GROUP_LAUNCH(p, K_FOLD, GK_FOLD, 256, group_fold_partials_kernel);
  GROUP_LAUNCH(p, K_COMBINE, GK_COMBINE, kCombineThreads, group_combine_adagrad_kernel);
  ++p.owner->launches[K_FINISH];
  launch_after(group_finish_apply_kernel, (unsigned)n_tables, 256, p.gs, p.d_items, (uint32_t)n_tables, 1);
  CUDA_TRY(p.owner, cudaGetLastError());
  for (int32_t i = 0; i < n_tables; ++i) tables[i]->prep.valid = false;
  return group_end(p, tables);
}

static int expire_range(mono_table* t, int64_t now, uint32_t slice, uint32_t n_slices) {
  if (!t || n_slices == 0 || slice >= n_slices) return MONO_ERR_ARG;
  if (t->prep.valid) join_sweep(t);                        // (forgetting the announced batch works on the table's stream)
  int rc = check_now(t, now);
  if (rc != MONO_OK) return rc;
  t->last_now = now;
  if (t->tv.ttl == 0) return MONO_OK;
  // a batch that was announced but not pushed yet was looked up in the table as it was: forget it
  if ((rc = discard_prepared(t)) != MONO_OK) return rc;
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
  // slices are multiples of four buckets; the last one takes the remainder and the stash
  const unsigned long long n_buckets = t->key_cells / kCellsPerBucket;           // a power of two >= 16
  const unsigned long long per_slice = n_buckets / n_slices & ~3ull;
  const bool is_last = slice + 1 == n_slices;
  const unsigned long long first = per_slice * slice;
  const unsigned long long last = is_last ? n_buckets : per_slice * (slice + 1);
  if (last > first || is_last) {
    const unsigned long long per_block = 256ull * 4 * kSweepDepth;               // buckets a block reads per round
    unsigned long long blocks = (last - first + per_block - 1) / per_block;
    if (blocks < 1) blocks = 1;
    if (blocks > (unsigned long long)grid_for(t, 8)) blocks = grid_for(t, 8);
    LAUNCH_ON(t, s, K_EXPIRE, launch_after(expire_kernel, (int)blocks, 256, s, t->tv, first, last, is_last ? 1 : 0, (long long)now));
  }
  if (slice + 1 == n_slices) LAUNCH_ON(t, s, K_STASH_TRIM, launch_after(stash_trim_kernel, 1, 32, s, t->tv));
  CUDA_TRY(t, cudaGetLastError());
  CUDA_TRY(t, cudaEventRecord(t->ev_swept, s));
  t->sweep_pending = true;
  return MONO_OK;
}

int mono_expire(mono_table* t, int64_t now) {
  MONO_API_RANGE();
  return expire_range(t, now, 0, 1);
}

int mono_expire_slice(mono_table* t, int64_t now, uint32_t slice, uint32_t n_slices) {
  MONO_API_RANGE();
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
  MONO_API_RANGE();
  if (t) join_sweep(t);
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if (n_bags > 0 && (!out || !aligned(out, 16))) return MONO_ERR_ARG;
  if (n_ids > (int64_t)MONO_NOALLOC_MAX_IDS) return MONO_ERR_LIMIT;
  if (n_bags == 0) return MONO_OK;
  int dev = -1;
  CUDA_TRY(t, cudaGetDevice(&dev));
  if (dev != t->device) return MONO_ERR_ARG;               // the array of another device would be the wrong memory
  uint32_t* occ_row = nullptr;
  if ((rc = noalloc_scratch(t, &occ_row)) != MONO_OK) return rc;
  const unsigned long long* d_ids = reinterpret_cast<const unsigned long long*>(ids);
  const long long* d_off = reinterpret_cast<const long long*>(slot_offsets);
  if ((rc = launch_probe(t, d_ids, n_ids, occ_row)) != MONO_OK) return rc;
  return launch_gather(t, occ_row, n_ids, d_off, n_bags, out);
}

// Streams, events and staging of the host-buffer calls, made by the first of them.
static int host_path_ready(mono_table* t, int64_t n_bags) {
  if (!t->h2d_stream) {
    CUDA_TRY(t, cudaStreamCreateWithFlags(&t->h2d_stream, cudaStreamNonBlocking));
    CUDA_TRY(t, cudaStreamCreateWithFlags(&t->d2h_stream, cudaStreamNonBlocking));
    for (cudaEvent_t* e : {&t->ev_staged, &t->ev_grad_in, &t->ev_out, &t->ev_d2h, &t->ev_stage_free})
      CUDA_TRY(t, cudaEventCreateWithFlags(e, cudaEventDisableTiming));
  }
  if (!t->stage_out) {                                     // sized with the rest of the scratch: max_bags rows
    (void)n_bags;
    int rc = dev_alloc(t, &t->stage_out, (size_t)t->max_bags * t->tv.dim);
    if (rc == MONO_OK) rc = dev_alloc(t, &t->stage_grad, (size_t)t->max_bags * t->tv.dim);
    if (rc != MONO_OK) { dev_free(t->stage_out); dev_free(t->stage_grad); return rc; }
  }
  return MONO_OK;
}

// IDs and offsets of a host batch to the staging buffers, on the inbound copy stream, once the
// kernels of the previous step are done with what is there.
static int stage_batch(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* off, int64_t n_bags) {
  cudaStream_t c = t->h2d_stream;
  if (t->stage_used) CUDA_TRY(t, cudaStreamWaitEvent(c, t->ev_stage_free, 0));
  if (n_ids) CUDA_TRY(t, cudaMemcpyAsync(t->stage_ids, ids, (size_t)n_ids * 8, cudaMemcpyHostToDevice, c));
  CUDA_TRY(t, cudaMemcpyAsync(t->stage_off, off, (size_t)(n_bags + 1) * 8, cudaMemcpyHostToDevice, c));
  CUDA_TRY(t, cudaEventRecord(t->ev_staged, c));
  CUDA_TRY(t, cudaStreamWaitEvent(t->stream, t->ev_staged, 0));
  return MONO_OK;
}

int mono_lookup_pool_host(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                          int64_t n_bags, float* out) {
  MONO_API_RANGE();
  if (t) join_sweep(t);
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if (n_bags > 0 && !out) return MONO_ERR_ARG;
  if ((rc = reserve(t, n_ids, n_bags)) != MONO_OK) return rc;
  if ((rc = host_path_ready(t, n_bags)) != MONO_OK) return rc;
  if ((rc = discard_prepared(t)) != MONO_OK) return rc;
  t->staged.valid = false;
  cudaStream_t s = t->stream;
  // the staging buffers must be free: the kernels that read the last staged batch have been issued on `s`
  CUDA_TRY(t, cudaEventRecord(t->ev_stage_free, s));
  t->stage_used = true;
  if ((rc = stage_batch(t, ids, n_ids, slot_offsets, n_bags)) != MONO_OK) return rc;
  if (n_bags == 0) return MONO_OK;
  // the staged batch is the one the push that follows will be given: group it and look its IDs up once for both
  bool prepared = false;
  if (n_ids > 0) {
    if ((rc = launch_prepare(t, t->stage_ids, n_ids, t->stage_off, n_bags)) != MONO_OK) return rc;
    t->prep = {t->stage_ids, n_ids, t->stage_off, n_bags, true, false};
    t->staged = {ids, n_ids, slot_offsets, n_bags, true};
    prepared = true;
  }
  // the previous result must have left stage_out before this one is written there
  if (t->d2h_pending) { CUDA_TRY(t, cudaStreamWaitEvent(s, t->ev_d2h, 0)); t->d2h_pending = false; }
  if ((rc = launch_lookup(t, t->stage_ids, n_ids, t->stage_off, n_bags, t->stage_out, prepared)) != MONO_OK) return rc;
  CUDA_TRY(t, cudaEventRecord(t->ev_out, s));
  CUDA_TRY(t, cudaStreamWaitEvent(t->d2h_stream, t->ev_out, 0));
  CUDA_TRY(t, cudaMemcpyAsync(out, t->stage_out, (size_t)n_bags * t->tv.dim * 4, cudaMemcpyDeviceToHost, t->d2h_stream));
  CUDA_TRY(t, cudaEventRecord(t->ev_d2h, t->d2h_stream));
  t->d2h_pending = true;
  return MONO_OK;
}

int mono_apply_grads_host(mono_table* t, const uint64_t* ids, int64_t n_ids, const int64_t* slot_offsets,
                          int64_t n_bags, const float* grad_pooled, int64_t now) {
  MONO_API_RANGE();
  if (t) join_sweep(t);
  int rc = check_batch(t, ids, n_ids, slot_offsets, n_bags);
  if (rc != MONO_OK) return rc;
  if (n_bags > 0 && !grad_pooled) return MONO_ERR_ARG;
  if ((rc = check_now(t, now)) != MONO_OK) return rc;
  if ((rc = reserve(t, n_ids, n_bags)) != MONO_OK) return rc;
  if ((rc = host_path_ready(t, n_bags)) != MONO_OK) return rc;
  cudaStream_t s = t->stream;
  const bool reuse = t->staged.valid && t->staged.ids == ids && t->staged.n_ids == n_ids && t->staged.off == slot_offsets &&
                     t->staged.n_bags == n_bags;
  t->staged.valid = false;
  if (!reuse) {
    // not the batch the lookup staged: bring its IDs and offsets in now (what was announced from the
    // staging buffers is about to be overwritten)
    if ((rc = discard_prepared(t)) != MONO_OK) return rc;
    CUDA_TRY(t, cudaEventRecord(t->ev_stage_free, s));
    t->stage_used = true;
    if ((rc = stage_batch(t, ids, n_ids, slot_offsets, n_bags)) != MONO_OK) return rc;
  }
  // the gradients come in on the copy stream while the ID-only kernels of the push run (the previous
  // push, the last reader of stage_grad, was issued before ev_stage_free was last recorded)
  cudaEvent_t grad_ready = nullptr;
  if (n_bags) {
    cudaStream_t c = t->h2d_stream;
    if (t->stage_used) CUDA_TRY(t, cudaStreamWaitEvent(c, t->ev_stage_free, 0));
    CUDA_TRY(t, cudaMemcpyAsync(t->stage_grad, grad_pooled, (size_t)n_bags * t->tv.dim * 4, cudaMemcpyHostToDevice, c));
    CUDA_TRY(t, cudaEventRecord(t->ev_grad_in, c));
    grad_ready = t->ev_grad_in;
  }
  t->last_now = now;
  rc = launch_apply(t, t->stage_ids, n_ids, t->stage_off, n_bags, t->stage_grad, (uint32_t)now, grad_ready);
  if (rc != MONO_OK) return rc;
  // (an empty batch launches nothing, so nothing has waited for the gradient copy yet)
  if (grad_ready && (n_ids == 0 || n_bags == 0)) CUDA_TRY(t, cudaStreamWaitEvent(s, grad_ready, 0));
  return MONO_OK;
}

int mono_fence(mono_table* t) {
  MONO_API_RANGE();
  if (!t) return MONO_ERR_ARG;
  join_sweep(t);
  if (t->d2h_pending) { CUDA_TRY(t, cudaStreamWaitEvent(t->stream, t->ev_d2h, 0)); t->d2h_pending = false; }
  if (t->ahead.valid) CUDA_TRY(t, cudaStreamWaitEvent(t->stream, t->ev_ahead, 0));     // a batch being grouped ahead
  return MONO_OK;
}

int mono_snapshot_save(mono_table* t) {
  MONO_API_RANGE();
  if (!t) return MONO_ERR_ARG;
  join_sweep(t);
  auto& sn = t->snap;
  { const int rc0 = discard_prepared(t); if (rc0 != MONO_OK) return rc0; }   // the per-call counters must be at rest
  const TableView& tv = t->tv;
  const size_t row_floats = ((size_t)tv.capacity + 1) * 2 * tv.dim;
  const size_t counters = tv.sketch_depth ? (size_t)tv.sketch_depth * (tv.sketch_mask + 1) : 0;
  if (sn.cells && sn.key_cells != t->key_cells) free_snapshot(t);            // the key store was resized since
  if (!sn.cells) {
    int rc = dev_alloc(t, &sn.cells, t->key_cells);
    if (rc == MONO_OK) rc = dev_alloc(t, &sn.stash, kStashCells);
    if (rc == MONO_OK) rc = dev_alloc(t, &sn.oldest, t->key_cells / kCellsPerBucket);
    if (rc == MONO_OK) rc = dev_alloc(t, &sn.rows, row_floats);
    if (rc == MONO_OK) rc = dev_alloc(t, &sn.free_rows, tv.capacity);
    if (rc == MONO_OK) rc = dev_alloc(t, &sn.st, 1);
    if (rc == MONO_OK && counters) rc = dev_alloc(t, &sn.sketch, counters);
    if (rc != MONO_OK) { free_snapshot(t); return rc; }
    sn.key_cells = t->key_cells;
  }
  cudaStream_t s = t->stream;
  const cudaMemcpyKind dd = cudaMemcpyDeviceToDevice;
  CUDA_TRY(t, cudaMemcpyAsync(sn.cells, tv.cells, t->key_cells * sizeof(Cell), dd, s));
  CUDA_TRY(t, cudaMemcpyAsync(sn.stash, tv.stash, kStashCells * sizeof(Cell), dd, s));
  CUDA_TRY(t, cudaMemcpyAsync(sn.oldest, tv.oldest, t->key_cells / kCellsPerBucket * sizeof(uint32_t), dd, s));
  CUDA_TRY(t, cudaMemcpyAsync(sn.rows, tv.rows, row_floats * sizeof(float), dd, s));
  CUDA_TRY(t, cudaMemcpyAsync(sn.free_rows, tv.free_rows, tv.capacity * sizeof(uint32_t), dd, s));
  CUDA_TRY(t, cudaMemcpyAsync(sn.st, tv.st, sizeof(DevState), dd, s));
  if (counters) CUDA_TRY(t, cudaMemcpyAsync(sn.sketch, tv.sketch, counters * sizeof(unsigned int), dd, s));
  sn.last_now = t->last_now;
  sn.sketch_epoch = t->sketch_epoch;
  sn.valid = true;
  return MONO_OK;
}

int mono_snapshot_restore(mono_table* t) {
  MONO_API_RANGE();
  if (!t) return MONO_ERR_ARG;
  join_sweep(t);
  auto& sn = t->snap;
  if (!sn.valid || sn.key_cells != t->key_cells) return MONO_ERR_ARG;
  int rc = discard_prepared(t);
  if (rc != MONO_OK) return rc;
  const TableView& tv = t->tv;
  const size_t row_floats = ((size_t)tv.capacity + 1) * 2 * tv.dim;
  const size_t counters = tv.sketch_depth ? (size_t)tv.sketch_depth * (tv.sketch_mask + 1) : 0;
  cudaStream_t s = t->stream;
  const cudaMemcpyKind dd = cudaMemcpyDeviceToDevice;
  CUDA_TRY(t, cudaMemcpyAsync(tv.cells, sn.cells, t->key_cells * sizeof(Cell), dd, s));
  CUDA_TRY(t, cudaMemcpyAsync(tv.stash, sn.stash, kStashCells * sizeof(Cell), dd, s));
  CUDA_TRY(t, cudaMemcpyAsync(tv.oldest, sn.oldest, t->key_cells / kCellsPerBucket * sizeof(uint32_t), dd, s));
  CUDA_TRY(t, cudaMemcpyAsync(tv.rows, sn.rows, row_floats * sizeof(float), dd, s));
  CUDA_TRY(t, cudaMemcpyAsync(tv.free_rows, sn.free_rows, tv.capacity * sizeof(uint32_t), dd, s));
  CUDA_TRY(t, cudaMemcpyAsync(tv.st, sn.st, sizeof(DevState), dd, s));
  if (counters) CUDA_TRY(t, cudaMemcpyAsync(tv.sketch, sn.sketch, counters * sizeof(unsigned int), dd, s));
  t->last_now = sn.last_now;
  t->sketch_epoch = sn.sketch_epoch;
  return MONO_OK;
}

int mono_snapshot_drop(mono_table* t) {
  MONO_API_RANGE();
  if (!t) return MONO_ERR_ARG;
  join_sweep(t);
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  free_snapshot(t);
  return MONO_OK;
}

int mono_status(mono_table* t, mono_status_t* host_out) {
  MONO_API_RANGE();
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
  host_out->scratch_reallocs = t->scratch_reallocs;
  return MONO_OK;
}

int mono_clear_errors(mono_table* t) {
  MONO_API_RANGE();
  if (t) join_sweep(t);
  if (!t) return MONO_ERR_ARG;
  CUDA_TRY(t, cudaMemsetAsync(&t->tv.st->error_bits, 0, sizeof(unsigned int), t->stream));
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  return MONO_OK;
}

int mono_probe(mono_table* t, const uint64_t* ids, int64_t n, uint8_t* resident, uint32_t* count,
               int64_t* last_seen) {
  MONO_API_RANGE();
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
  MONO_API_RANGE();
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
  MONO_API_RANGE();
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
  MONO_API_RANGE();
  if (t) join_sweep(t);
  if (!t) return MONO_ERR_ARG;
  if (new_key_cells == 0) new_key_cells = t->key_cells;
  if (!is_pow2(new_key_cells) || new_key_cells < 64 || new_key_cells > (1ull << 34)) return MONO_ERR_ARG;
  { const int rc0 = discard_prepared(t); if (rc0 != MONO_OK) return rc0; }     // its remembered cells are about to move
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
  TableView fresh = t->tv;
  fresh.cells = nullptr;
  fresh.stash = nullptr;
  fresh.oldest = nullptr;
  int rc = dev_alloc(t, &fresh.cells, new_key_cells);
  if (rc == MONO_OK) rc = dev_alloc(t, &fresh.stash, kStashCells);
  if (rc == MONO_OK) rc = dev_alloc(t, &fresh.oldest, new_key_cells / kCellsPerBucket);
  if (rc != MONO_OK) { dev_free(fresh.cells); dev_free(fresh.stash); dev_free(fresh.oldest); return rc; }
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
    dev_free(fresh.cells); dev_free(fresh.stash); dev_free(fresh.oldest);
    return MONO_ERR_CUDA;
  }
  dev_free(t->tv.cells);
  dev_free(t->tv.stash);
  dev_free(t->tv.oldest);
  t->tv = fresh;
  t->key_cells = new_key_cells;
  return MONO_OK;
}

int mono_export_touched(mono_table* t, uint64_t* ids, float* w, int64_t max_n, int64_t* n_out) {
  MONO_API_RANGE();
  if (t) join_sweep(t);
  if (!t || !n_out || max_n < 0 || (max_n > 0 && (!ids || !w || !aligned(w, 16) || !aligned(ids, 8)))) return MONO_ERR_ARG;
  { const int rc0 = discard_prepared(t); if (rc0 != MONO_OK) return rc0; }
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
  MONO_API_RANGE();
  if (t) join_sweep(t);
  if (!t || n < 0) return MONO_ERR_ARG;
  if (n == 0) return MONO_OK;
  if (!ids || !count || !last_seen || !resident || !aligned(ids, 8)) return MONO_ERR_ARG;
  if ((w && !aligned(w, 16)) || (acc && !aligned(acc, 16))) return MONO_ERR_ARG;
  int rc = discard_prepared(t);
  if (rc != MONO_OK) return rc;
  uint32_t* row_word = nullptr;
  const int64_t chunk = n < (1ll << 24) ? n : (1ll << 24);
  rc = dev_alloc(t, &row_word, (size_t)chunk);
  if (rc != MONO_OK) return rc;
  for (int64_t lo = 0; lo < n; lo += chunk) {
    const int64_t m = n - lo < chunk ? n - lo : chunk;
    const size_t ro = (size_t)lo * t->tv.dim;
    import_check_kernel<<<grid_for(t, 4), 256, 0, t->stream>>>(
        t->tv, reinterpret_cast<const unsigned long long*>(ids) + lo, m, row_word);
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
  MONO_API_RANGE();
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
  host_out->behind_records = h.behind_records > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)h.behind_records;
  const bool leak_ok = h.unaccounted_rows == 0 || d.n_keys_dropped > 0;   // a dropped key may strand its row
  host_out->ok = (h.misplaced == 0 && h.duplicate_keys == 0 && h.behind_records == 0 && h.bad_rows == 0 && h.shared_rows == 0 && leak_ok &&
                  h.occupied == d.n_tracked && h.resident_cells == d.n_resident &&
                  h.resident_cells + h.free_rows + h.unaccounted_rows == t->tv.capacity)
                     ? 1u : 0u;
  return MONO_OK;
}

int mono_timing_enable(mono_table* t, int on) {
  if (!t) return MONO_ERR_ARG;
  if (t->ahead_stream) cudaStreamSynchronize(t->ahead_stream);     // a grouping in flight keeps the stream it started on
  t->timing = on != 0;
  return MONO_OK;
}

int mono_timing_read(mono_table* t, mono_timing_t* host_out, int reset) {
  MONO_API_RANGE();
  if (t) join_sweep(t);
  if (!t || !host_out) return MONO_ERR_ARG;
  CUDA_TRY(t, cudaStreamSynchronize(t->stream));
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
