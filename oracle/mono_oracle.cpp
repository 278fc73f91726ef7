// CPU oracle for the collisionless embedding-table step of Monolith
// (arXiv 2209.07663, Section 2.1 on the hash table and the training step of
// Section 2.2).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
// CUDA library must compute.  It shares no code with the CUDA path, is never
// linked into it, and must only be used by the tests, the smoke check and the
// benchmark's CPU-baseline leg.
//
// Where the method reaches a result that has a plain definition, this file is
// that definition: the cuckoo table of Section 2.1 is a collision-free map from
// a 64-bit ID to its embedding, so the oracle keeps a std::unordered_map and
// never hashes into buckets.  The occurrence filter (Section 2.1, heuristic 1)
// and the expiry of inactive IDs (heuristic 2) are kept as a literal counter
// and a literal last-seen time per ID.  Sum pooling, gradient de-duplication
// and the Adagrad row update are not described in the paper; they follow the
// usual definitions (sum over the bag; one Adagrad step per distinct row with
// the gradients of duplicate IDs summed first).
//
// Pins (see tests/test_oracle_*.py): per-ID replay state machine, brute force
// over tiny streams, torch.nn.functional.embedding_bag and torch.optim.Adagrad
// as library special cases, closed forms for each rule, Philox known answers.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -shared -fPIC mono_oracle.cpp

#include <cmath>
#include <cstdint>
#include <cstring>
#include <unordered_map>
#include <vector>
#include <algorithm>

namespace {

constexpr uint64_t kReservedId = 0xFFFFFFFFFFFFFFFFull;

struct Entry {
  uint32_t count = 0;        // occurrences so far, saturating at the threshold
  int64_t last_seen = 0;     // `now` of the last apply_grads that contained the ID
  bool resident = false;     // owns an embedding row
  bool touched = false;      // row trained since the last export of touched keys
  std::vector<float> w;      // embedding row (empty unless resident)
  std::vector<float> acc;    // Adagrad accumulator (empty unless resident)
};

struct Oracle {
  uint64_t capacity;
  uint32_t dim;
  uint32_t threshold;        // effective threshold, >= 1
  uint32_t ttl;              // 0 disables expiry
  float lr, eps, init_acc, init_scale;
  uint64_t seed;
  int64_t last_now = INT64_MIN;
  uint64_t n_resident = 0;
  std::unordered_map<uint64_t, Entry> map;
  // probabilistic filter (count-min sketch) in place of exact per-ID counters; depth 0 = off
  uint32_t sketch_depth = 0;
  uint64_t sketch_width = 0;        // power of two
  std::vector<uint64_t> sketch;     // [depth][width]
  int64_t sketch_epoch = 0;         // time of the last reset
};

// SplitMix64 output function (Steele, Lea, Flood 2014); the sketch's row hashes are
// built from it so that both sides index the same counters.
inline uint64_t splitmix64_mix(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Counter of row r that ID `id` maps to.
inline uint64_t sketch_index(const Oracle* o, uint32_t r, uint64_t id) {
  return splitmix64_mix(id ^ (o->seed + (uint64_t)(r + 1) * 0x9E3779B97F4A7C15ull)) & (o->sketch_width - 1);
}

inline uint64_t sketch_estimate(const Oracle* o, uint64_t id) {
  uint64_t est = UINT64_MAX;
  for (uint32_t r = 0; r < o->sketch_depth; ++r)
    est = std::min(est, o->sketch[(size_t)r * o->sketch_width + sketch_index(o, r, id)]);
  return est;
}

// One Adagrad step of a row with the summed gradient g (fp64 sums rounded once to fp32).
inline void adagrad_row(const Oracle* o, Entry& e, const std::vector<double>& g) {
  for (uint32_t col = 0; col < o->dim; ++col) {
    const float G = (float)g[col];
    const float a = e.acc[col] + G * G;
    e.acc[col] = a;
    e.w[col] = e.w[col] - o->lr * G / (sqrtf(a) + o->eps);
  }
  e.touched = true;      // Section 2.2.3: the ID joins the set of touched keys
}

inline float init_value(uint64_t seed, uint64_t id, uint32_t col, float scale);   // defined below

inline void give_row(Oracle* o, Entry& e, uint64_t id) {
  e.resident = true;
  ++o->n_resident;
  e.w.resize(o->dim); e.acc.resize(o->dim);
  for (uint32_t col = 0; col < o->dim; ++col) {
    e.w[col] = init_value(o->seed, id, col, o->init_scale);
    e.acc[col] = o->init_acc;
  }
}

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
// as 1, 2, 3", SC'11).  Counter-based, so a row's initial value depends only
// on (seed, id, column) and never on insertion order.
inline void philox_round(uint32_t c[4], const uint32_t k[2]) {
  const uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
  const uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
  const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ k[0];
  const uint32_t n1 = (uint32_t)p1;
  const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ k[1];
  const uint32_t n3 = (uint32_t)p0;
  c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
}

inline void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
  uint32_t k[2] = {key[0], key[1]};
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; }
    philox_round(c, k);
  }
  out[0] = c[0]; out[1] = c[1]; out[2] = c[2]; out[3] = c[3];
}

// Initial embedding value of column `col` of ID `id`: Philox keyed by the
// table seed, counter (id low, id high, col / 4, 0); word col % 4 of the
// output; its top 24 bits u give (u * 2^-23 - 1) * init_scale, uniform on
// [-init_scale, init_scale).  All steps are exact in fp32 except the final
// multiplication, which rounds once.
inline float init_value(uint64_t seed, uint64_t id, uint32_t col, float scale) {
  const uint32_t ctr[4] = {(uint32_t)id, (uint32_t)(id >> 32), col / 4u, 0u};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t r[4];
  philox4x32_10(ctr, key, r);
  const float u = (float)(r[col % 4u] >> 8) * (1.0f / 8388608.0f) - 1.0f;
  return u * scale;
}

}  // namespace

extern "C" {

enum { ORACLE_OK = 0, ORACLE_ERR_ARG = -1, ORACLE_ERR_TIME = -2, ORACLE_ERR_FULL = -3 };

void* oracle_create(uint64_t capacity, uint32_t dim, uint32_t filter_threshold, uint32_t ttl,
                    float lr, float eps, float init_acc, float init_scale, uint64_t seed) {
  if (dim == 0 || capacity == 0) return nullptr;
  Oracle* o = new Oracle();
  o->capacity = capacity;
  o->dim = dim;
  o->threshold = std::max<uint32_t>(filter_threshold, 1u);
  o->ttl = ttl;
  o->lr = lr; o->eps = eps; o->init_acc = init_acc; o->init_scale = init_scale;
  o->seed = seed;
  return o;
}

// Switch the admission filter to a count-min sketch of `depth` rows of `width` counters
// (width a power of two).  Call before the first batch.
int oracle_enable_sketch(void* h, uint32_t depth, uint64_t width) {
  Oracle* o = static_cast<Oracle*>(h);
  if (!o || depth == 0 || width == 0 || (width & (width - 1)) || !o->map.empty()) return ORACLE_ERR_ARG;
  o->sketch_depth = depth;
  o->sketch_width = width;
  o->sketch.assign((size_t)depth * width, 0ull);
  return ORACLE_OK;
}

uint64_t oracle_sketch_index(void* h, uint32_t r, uint64_t id) { return sketch_index(static_cast<Oracle*>(h), r, id); }

void oracle_destroy(void* h) { delete static_cast<Oracle*>(h); }

// Forward: out[b, :] = sum of the rows of the resident IDs of bag b, in the
// order the IDs appear; IDs without a row contribute nothing (Section 2.2:
// the worker pulls parameters; a filtered or unknown ID has none).
// Read-only: neither counts nor times change.
int oracle_lookup_pool(void* h, const uint64_t* ids, int64_t n_ids, const int64_t* offsets,
                       int64_t n_bags, float* out) {
  Oracle* o = static_cast<Oracle*>(h);
  if (!o || n_ids < 0 || n_bags < 0) return ORACLE_ERR_ARG;
  const uint32_t d = o->dim;
  std::vector<double> s(d);
  for (int64_t b = 0; b < n_bags; ++b) {
    std::fill(s.begin(), s.end(), 0.0);
    for (int64_t j = offsets[b]; j < offsets[b + 1]; ++j) {
      if (j < 0 || j >= n_ids) return ORACLE_ERR_ARG;
      if (ids[j] == kReservedId) continue;
      auto it = o->map.find(ids[j]);
      if (it == o->map.end() || !it->second.resident) continue;
      for (uint32_t c = 0; c < d; ++c) s[c] += (double)it->second.w[c];
    }
    for (uint32_t c = 0; c < d; ++c) out[b * (int64_t)d + c] = (float)s[c];
  }
  return ORACLE_OK;
}

// Backward + update (the parameter push of Section 2.2), with the
// occurrence filter and the last-access stamp of Section 2.1:
//   1. group the batch's occurrences by ID: multiplicity and the sum, in
//      double and in occurrence order, of the pooled gradients of their bags;
//   2. per distinct ID: count += multiplicity (saturating at the threshold),
//      last_seen = now;
//   3. an ID whose count has reached the threshold and that has no row gets
//      one, with initial values from init_value and accumulator init_acc;
//   4. every ID that has a row takes one Adagrad step with its summed
//      gradient G rounded once to fp32:  acc += G*G;  w -= lr*G/(sqrt(acc)+eps).
// Gradients of IDs without a row are dropped.
int oracle_apply_grads(void* h, const uint64_t* ids, int64_t n_ids, const int64_t* offsets,
                       int64_t n_bags, const float* grad_pooled, int64_t now) {
  Oracle* o = static_cast<Oracle*>(h);
  if (!o || n_ids < 0 || n_bags < 0) return ORACLE_ERR_ARG;
  if (o->last_now != INT64_MIN && now < o->last_now) return ORACLE_ERR_TIME;
  o->last_now = now;
  const uint32_t d = o->dim;

  struct Group { uint64_t mult = 0; std::vector<double> g; };
  std::unordered_map<uint64_t, size_t> index;
  std::vector<uint64_t> order;        // distinct IDs in order of first appearance
  std::vector<Group> groups;
  for (int64_t b = 0; b < n_bags; ++b) {
    for (int64_t j = offsets[b]; j < offsets[b + 1]; ++j) {
      if (j < 0 || j >= n_ids) return ORACLE_ERR_ARG;
      const uint64_t id = ids[j];
      if (id == kReservedId) continue;
      auto ins = index.emplace(id, groups.size());
      if (ins.second) { order.push_back(id); groups.emplace_back(); groups.back().g.assign(d, 0.0); }
      Group& gr = groups[ins.first->second];
      gr.mult += 1;
      for (uint32_t c = 0; c < d; ++c) gr.g[c] += (double)grad_pooled[b * (int64_t)d + c];
    }
  }

  int rc = ORACLE_OK;
  if (o->sketch_depth) {
    // Probabilistic filter (Section 2.1, heuristic 1, second method): a count-min sketch
    // stands in for the per-ID counters, so an ID without a row costs no entry at all.
    //  a. every distinct ID without a row adds its multiplicity to one counter per sketch row;
    //  b. after all additions of the batch, an ID whose smallest counter has reached the
    //     threshold is given a row (it may get there early through collisions, never late);
    //  c. IDs with a row are stamped and updated as in the exact mode.
    for (size_t u = 0; u < order.size(); ++u) {
      auto it = o->map.find(order[u]);
      if (it != o->map.end() && it->second.resident) continue;
      for (uint32_t r = 0; r < o->sketch_depth; ++r)
        o->sketch[(size_t)r * o->sketch_width + sketch_index(o, r, order[u])] += groups[u].mult;
    }
    for (size_t u = 0; u < order.size(); ++u) {
      const uint64_t id = order[u];
      auto it = o->map.find(id);
      if (it == o->map.end()) {
        if (sketch_estimate(o, id) < o->threshold) continue;
        if (o->n_resident >= o->capacity) { rc = ORACLE_ERR_FULL; continue; }
        it = o->map.emplace(id, Entry()).first;
        it->second.count = o->threshold;
        give_row(o, it->second, id);
      }
      it->second.last_seen = now;
      adagrad_row(o, it->second, groups[u].g);
    }
    return rc;
  }
  for (size_t u = 0; u < order.size(); ++u) {
    const uint64_t id = order[u];
    Entry& e = o->map[id];             // creates {count 0, not resident} if untracked
    const uint64_t c = (uint64_t)e.count + groups[u].mult;
    e.count = (uint32_t)std::min<uint64_t>(c, o->threshold);
    e.last_seen = now;
    if (!e.resident && e.count >= o->threshold) {
      if (o->n_resident >= o->capacity) { rc = ORACLE_ERR_FULL; continue; }
      give_row(o, e, id);
    }
    if (e.resident) adagrad_row(o, e, groups[u].g);
  }
  return rc;
}

// Expiry (Section 2.1, heuristic 2): forget every tracked ID, with or without
// a row, that has been inactive for longer than ttl.  ttl == 0 disables it.
// Returns the number of IDs removed.
int64_t oracle_expire(void* h, int64_t now) {
  Oracle* o = static_cast<Oracle*>(h);
  if (!o) return ORACLE_ERR_ARG;
  if (o->ttl == 0) return 0;
  // the sketch forgets in whole windows: it is cleared when more than ttl has passed since
  // it was last cleared (time 0 at creation)
  if (o->sketch_depth && now - o->sketch_epoch > (int64_t)o->ttl) {
    std::fill(o->sketch.begin(), o->sketch.end(), 0ull);
    o->sketch_epoch = now;
  }
  int64_t removed = 0;
  for (auto it = o->map.begin(); it != o->map.end();) {
    if (now - it->second.last_seen > (int64_t)o->ttl) {
      if (it->second.resident) --o->n_resident;
      it = o->map.erase(it);
      ++removed;
    } else {
      ++it;
    }
  }
  return removed;
}

int64_t oracle_n_tracked(void* h) { return (int64_t)static_cast<Oracle*>(h)->map.size(); }
int64_t oracle_n_resident(void* h) { return (int64_t)static_cast<Oracle*>(h)->n_resident; }

// Parameter synchronisation (Section 2.2.3): the touched keys are the IDs whose
// embeddings were trained since the last synchronisation.  Writes them in
// increasing ID order with their rows and empties the set.  An ID that expired
// in between is simply gone.  Buffers sized by oracle_n_touched.
int64_t oracle_n_touched(void* h) {
  Oracle* o = static_cast<Oracle*>(h);
  int64_t n = 0;
  for (auto& kv : o->map) n += kv.second.touched ? 1 : 0;
  return n;
}

int64_t oracle_export_touched(void* h, uint64_t* ids, float* w) {
  Oracle* o = static_cast<Oracle*>(h);
  std::vector<uint64_t> keys;
  for (auto& kv : o->map) if (kv.second.touched) keys.push_back(kv.first);
  std::sort(keys.begin(), keys.end());
  for (size_t i = 0; i < keys.size(); ++i) {
    Entry& e = o->map[keys[i]];
    ids[i] = keys[i];
    for (uint32_t c = 0; c < o->dim; ++c) w[i * (size_t)o->dim + c] = e.w[c];
    e.touched = false;
  }
  return (int64_t)keys.size();
}

// State of n given IDs.  Untracked: resident 0, count 0, last_seen -1, zeros.
int oracle_probe(void* h, const uint64_t* ids, int64_t n, uint8_t* resident, uint32_t* count,
                 int64_t* last_seen, float* w, float* acc) {
  Oracle* o = static_cast<Oracle*>(h);
  if (!o) return ORACLE_ERR_ARG;
  const uint32_t d = o->dim;
  for (int64_t i = 0; i < n; ++i) {
    auto it = o->map.find(ids[i]);
    const bool tracked = it != o->map.end() && ids[i] != kReservedId;
    const bool res = tracked && it->second.resident;
    if (resident) resident[i] = res ? 1 : 0;
    if (count) {
      count[i] = tracked ? it->second.count : 0;
      if (!tracked && o->sketch_depth && ids[i] != kReservedId)     // sketch mode: the estimate, capped
        count[i] = (uint32_t)std::min<uint64_t>(sketch_estimate(o, ids[i]), o->threshold);
    }
    if (last_seen) last_seen[i] = tracked ? it->second.last_seen : -1;
    for (uint32_t c = 0; c < d; ++c) {
      if (w) w[i * (int64_t)d + c] = res ? it->second.w[c] : 0.0f;
      if (acc) acc[i * (int64_t)d + c] = res ? it->second.acc[c] : 0.0f;
    }
  }
  return ORACLE_OK;
}

// All tracked IDs in increasing ID order (buffers sized by oracle_n_tracked).
int64_t oracle_export(void* h, uint64_t* ids, uint32_t* count, int64_t* last_seen,
                      uint8_t* resident, float* w, float* acc) {
  Oracle* o = static_cast<Oracle*>(h);
  if (!o) return ORACLE_ERR_ARG;
  std::vector<uint64_t> keys;
  keys.reserve(o->map.size());
  for (auto& kv : o->map) keys.push_back(kv.first);
  std::sort(keys.begin(), keys.end());
  for (size_t i = 0; i < keys.size(); ++i) ids[i] = keys[i];
  oracle_probe(h, keys.data(), (int64_t)keys.size(), resident, count, last_seen, w, acc);
  return (int64_t)keys.size();
}

// Pre-load entries (a test fixture: builds a table state without a stream).
// w / acc may be null for entries that are all non-resident.
int oracle_import(void* h, const uint64_t* ids, const uint32_t* count, const int64_t* last_seen,
                  const uint8_t* resident, const float* w, const float* acc, int64_t n) {
  Oracle* o = static_cast<Oracle*>(h);
  if (!o) return ORACLE_ERR_ARG;
  const uint32_t d = o->dim;
  for (int64_t i = 0; i < n; ++i) {
    if (ids[i] == kReservedId) return ORACLE_ERR_ARG;
    if (o->map.count(ids[i])) return ORACLE_ERR_ARG;
    Entry e;
    e.count = std::min<uint32_t>(count[i], o->threshold);
    e.last_seen = last_seen[i];
    e.resident = resident[i] != 0;
    if (e.resident) {
      if (o->n_resident >= o->capacity) return ORACLE_ERR_FULL;
      if (!w || !acc) return ORACLE_ERR_ARG;
      e.count = o->threshold;
      ++o->n_resident;
      e.w.assign(w + i * (int64_t)d, w + (i + 1) * (int64_t)d);
      e.acc.assign(acc + i * (int64_t)d, acc + (i + 1) * (int64_t)d);
    }
    o->map.emplace(ids[i], std::move(e));
  }
  return ORACLE_OK;
}

// Exposed so that the tests can pin the generator against its published
// known-answer vectors and the init rule against a by-hand evaluation.
void oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}
float oracle_init_value(uint64_t seed, uint64_t id, uint32_t col, float scale) {
  return init_value(seed, id, col, scale);
}

}  // extern "C"
