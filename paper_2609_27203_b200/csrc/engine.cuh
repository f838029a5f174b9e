// Host-side engine state and the typed building blocks the fixpoint driver composes:
// sort, reduce-by-key, merge, join evaluation.  Everything here issues work on the context's
// stream and sub-allocates from the caller's arena.
#pragma once
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <functional>
#include <map>
#include <memory>
#include <set>
#include <string>
#include <vector>

#include "../../include/xlog.h"
#include "arena.h"
#include "common.cuh"
#include "dense_reduce.cuh"
#include "join.cuh"
#include "relops.cuh"
#include "scan.cuh"
#include "sort.cuh"

namespace xlog {

struct Fail {
  xlog_status st;
  std::string msg;
};
[[noreturn]] inline void fail(xlog_status st, const std::string& m) { throw Fail{st, m}; }

#define XLOG_CUDA(expr)                                                                            \
  do {                                                                                             \
    cudaError_t e__ = (expr);                                                                      \
    if (e__ != cudaSuccess) fail(XLOG_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__)); \
  } while (0)

constexpr int kCtrlSlots = 96;          // uint64 control words mirrored to pinned host memory
constexpr int kSlotResState = 64;       // the resident loop's state block (resident.cuh) lives in the control words from here on
constexpr int kSlotErr = 0;
constexpr int64_t kProfLargeBytes = (int64_t)4000000 * 12;

struct Ctx;

// Arena allocation with scope lifetime.  Every kernel and copy of a context is issued on its one
// stream, so a block may be released (and handed out again) while work that uses it is still queued:
// whatever reuses the memory is queued later and therefore runs later.
struct DevBuf {
  Ctx* c = nullptr;
  void* p = nullptr;
  size_t bytes = 0;
  DevBuf() {}
  DevBuf(Ctx* ctx, size_t n);
  DevBuf(const DevBuf&) = delete;
  DevBuf& operator=(const DevBuf&) = delete;
  DevBuf(DevBuf&& o) noexcept { *this = std::move(o); }
  DevBuf& operator=(DevBuf&& o) noexcept {
    if (this != &o) { reset(); c = o.c; p = o.p; bytes = o.bytes; o.p = nullptr; o.bytes = 0; }
    return *this;
  }
  ~DevBuf() { reset(); }
  void reset();
  template <typename T> T* as() const { return reinterpret_cast<T*>(p); }
};

struct Index {                          // sorted access path on one column of a relation
  bool valid = false;
  int64_t domain = 0;                   // offsets has domain + 1 entries
  DevBuf off;
  int n_other = 0;
  int other_src[kMaxArity - 1] = {0, 0, 0};     // original column of each non-probed column
  const int32_t* other[kMaxArity - 1] = {nullptr, nullptr, nullptr};
  const float* tags = nullptr;
  DevBuf own_cols[kMaxArity - 1];       // owned storage when the index is a permuted copy
  DevBuf own_tags;
};

struct Relation {
  int arity = 0, sr = 0;
  std::string name;
  // loaded facts: packed keys sorted ascending, unique
  KeyLayout layout{};
  int key_bytes = 4;
  int32_t col_max[kMaxArity] = {0, 0, 0, 0};      // bound of what is stored (the code when the column has a dictionary)
  int32_t fact_max[kMaxArity] = {0, 0, 0, 0};     // column maxima of the loaded facts
  int32_t val_max[kMaxArity] = {0, 0, 0, 0};      // bound of the column's values
  DevBuf dict[kMaxArity];                         // sorted distinct values of a dictionary-encoded column
  uint32_t dict_n[kMaxArity] = {0, 0, 0, 0};
  DevBuf fact_keys, fact_tags;
  uint32_t n_facts = 0;
  // current contents; alias the facts until something is derived
  DevBuf cur_keys, cur_tags;
  bool cur_owned = false;
  uint32_t n = 0;
  // column-major int32 view of the current contents
  DevBuf cols[kMaxArity];
  bool soa_valid = false;
  Index idx[kMaxArity];
  bool is_head = false;

  DictSet dicts() const {
    DictSet d{};
    for (int i = 0; i < kMaxArity; ++i) { d.v[i] = dict[i].as<int32_t>(); d.n[i] = dict_n[i]; }
    return d;
  }
  const void* keys() const { return cur_owned ? cur_keys.p : fact_keys.p; }
  float* tags() const { return reinterpret_cast<float*>(cur_owned ? cur_tags.p : fact_tags.p); }
};

struct JoinShape {                      // how a two-atom rule is evaluated with `outer` as the scanned side
  bool ok = false;
  int outer = 0, inner = 1;
  int probe_col = 0;                    // column of the inner atom that is looked up
  int probe_var = 0, probe_mul = 1, probe_add = 0;
};

struct RuleC {
  xlog_plan plan;
  int kind = 0;                         // 1: one atom, 2: two-atom join, 3/4: directed triangle (aggregate / rows), 5: atom + negated atom, 6: four-cycle (rows)
  int neg_prefix = 0;                   // kind 5: how many leading columns of the negated atom are fixed
  JoinShape shape[2];                   // indexed by the outer atom
};

// Everything the resident rounds of one head relation need, kept across fixpoint calls so that the instantiated
// graph (which holds the buffers' addresses) can be launched again: the tag mirror, the delta and the join scratch
// at their fixed capacities.
struct Resident {
  uint64_t slots = 0;
  uint32_t max_tiles = 0;
  DevBuf table, bitmap, present, ch_sums, ch_counts, dkeys, dtags, rowinfo, start, tile_rows, scan_status, tickets;
  uint32_t scan_tiles_cap = 0;
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  std::vector<char> sig;                  // every kernel argument of the captured body, byte for byte
  int64_t body_launches = 0;
  ~Resident() {
    if (exec) cudaGraphExecDestroy(exec);
    if (graph) cudaGraphDestroy(graph);
  }
};

struct Ctx {
  int device = 0;
  cudaStream_t stream = nullptr;
  cudaStream_t capture_stream = nullptr;  // only ever records graph bodies
  Arena arena;
  int64_t max_iter = 1 << 20;
  size_t chunk_bytes = 0;
  uint32_t flags = 0;
  std::string err;
  std::vector<Relation*> rels;
  std::vector<RuleC> rules;
  bool idb_dirty = false, poisoned = false, evaluated = false;
  uint64_t* d_ctrl = nullptr;
  uint64_t* h_ctrl = nullptr;
  int64_t launches = 0, d2h_bytes = 0, h2d_bytes = 0;
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  // receipt counters of the running fixpoint
  int64_t r_candidates = 0, r_unique = 0, r_new = 0, r_improved = 0, r_iterations = 0, r_strata = 0, r_index_builds = 0;
  // optional per-kernel timing (XLOG_FLAG_PROFILE): CUDA events around every launch
  struct ProfEntry { std::string name; int64_t launches = 0; double ms = 0; int64_t bytes = 0; };
  struct ProfPending { int entry; cudaEvent_t a, b; int big_entry; };      // big_entry >= 0: also counted under "<name> (large)"
  std::vector<ProfEntry> prof;
  std::map<std::string, int> prof_index;
  std::vector<ProfPending> prof_pending;
  std::vector<cudaEvent_t> ev_pool;
  int64_t note_bytes = 0;                 // algorithmic bytes of the next launch (consumed by the launch macro)
  std::map<int, std::unique_ptr<Resident>> resident;   // by head relation
  int last_triangle_plan = 0;             // XLOG_PLAN_* of the last materialised triangle join
  uint32_t spin_limit = kSpinLimit;      // polls of one status word before a look-back wait gives up (sort passes, resident scan)
  bool unique_untracked = false;          // a stratum went through the tag mirror, which does not count distinct candidate keys
  std::vector<char> stratum_done;         // per relation: its stratum has been evaluated in the running fixpoint
};

inline DevBuf::DevBuf(Ctx* ctx, size_t n) : c(ctx), bytes(n) {
  p = ctx->arena.alloc(n);
  if (!p) {
    char m[160];
    snprintf(m, sizeof m, "arena exhausted: need %zu bytes, %zu of %zu in use, largest free block %zu", n,
             ctx->arena.in_use(), ctx->arena.capacity(), ctx->arena.largest_free());
    fail(XLOG_ERR_RESOURCE_EXHAUSTED, m);
  }
}
inline void DevBuf::reset() {
  if (p && c) c->arena.release(p);
  p = nullptr; bytes = 0;
}

inline cudaEvent_t prof_event(Ctx* c) {
  if (!c->ev_pool.empty()) { cudaEvent_t e = c->ev_pool.back(); c->ev_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) fail(XLOG_ERR_CUDA, "cudaEventCreate");
  return e;
}
inline void prof_begin(Ctx* c, const char* what) {
  std::string name(what);
  if (!name.empty() && name[0] == '(') name = name.substr(1);
  name = name.substr(0, name.find_first_of("<)"));
  auto it = c->prof_index.find(name);
  if (it == c->prof_index.end()) {
    it = c->prof_index.emplace(name, (int)c->prof.size()).first;
    c->prof.push_back(Ctx::ProfEntry{name, 0, 0.0, 0});
  }
  // launches that declare at least kProfLargeBytes (4 M candidates of 12 bytes) are also totalled on their own, so that the
  // large rounds of a fixpoint can be told from the launch-bound small ones
  int big = -1;
  if (c->note_bytes >= kProfLargeBytes) {
    const std::string bn = name + " (large)";
    auto bt = c->prof_index.find(bn);
    if (bt == c->prof_index.end()) {
      bt = c->prof_index.emplace(bn, (int)c->prof.size()).first;
      c->prof.push_back(Ctx::ProfEntry{bn, 0, 0.0, 0});
    }
    big = bt->second;
    it = c->prof_index.find(name);                       // the emplace may have moved nothing, but look the entry up again to be safe
  }
  Ctx::ProfPending p{it->second, prof_event(c), prof_event(c), big};
  cudaEventRecord(p.a, c->stream);
  c->prof_pending.push_back(p);
}
// Fold finished launches into the table; call only when the stream is known to be idle.
inline void prof_collect(Ctx* c) {
  for (Ctx::ProfPending& p : c->prof_pending) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, p.a, p.b) == cudaSuccess) {
      c->prof[p.entry].ms += ms;
      if (p.big_entry >= 0) c->prof[p.big_entry].ms += ms;
    }
    c->ev_pool.push_back(p.a); c->ev_pool.push_back(p.b);
  }
  c->prof_pending.clear();
}
inline void check_launch(Ctx* c, const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) fail(XLOG_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
  ++c->launches;
  if (c->flags & XLOG_FLAG_PROFILE) {
    Ctx::ProfPending& p = c->prof_pending.back();
    cudaEventRecord(p.b, c->stream);
    c->prof[p.entry].launches += 1;
    c->prof[p.entry].bytes += c->note_bytes;
    if (p.big_entry >= 0) { c->prof[p.big_entry].launches += 1; c->prof[p.big_entry].bytes += c->note_bytes; }
  }
  c->note_bytes = 0;
}
#define XLOG_LAUNCH(ctx, kern, grid, block, smem, ...)                   \
  do {                                                                   \
    if ((ctx)->flags & XLOG_FLAG_PROFILE) prof_begin((ctx), #kern);      \
    kern<<<(grid), (block), (smem), (ctx)->stream>>>(__VA_ARGS__);       \
    check_launch((ctx), #kern);                                          \
  } while (0)

inline unsigned grid_for(uint64_t n, int block, int cap = kSMs * 16) {
  const uint64_t g = (n + block - 1) / block;
  return (unsigned)std::max<uint64_t>(1, std::min<uint64_t>(g, (uint64_t)cap));
}

// Copy the control block to pinned host memory and wait: the bounded control read of an iteration.
inline void sync_ctrl(Ctx* c) {
  XLOG_CUDA(cudaMemcpyAsync(c->h_ctrl, c->d_ctrl, kCtrlSlots * sizeof(uint64_t), cudaMemcpyDeviceToHost, c->stream));
  XLOG_CUDA(cudaStreamSynchronize(c->stream));
  if (!c->prof_pending.empty()) prof_collect(c);
  c->d2h_bytes += kCtrlSlots * sizeof(uint64_t);
  const uint32_t e = (uint32_t)c->h_ctrl[kSlotErr];
  if (e) {
    XLOG_CUDA(cudaMemsetAsync(c->d_ctrl, 0, sizeof(uint64_t), c->stream));
    if (e & kErrNegativeKey) fail(XLOG_ERR_INVALID_VALUE, "negative key");
    if (e & kErrBadTag) fail(XLOG_ERR_INVALID_VALUE, "tag is NaN or the semiring zero");
    if (e & kErrHeadRange) fail(XLOG_ERR_CAPACITY_EXCEEDED, "head column value outside the relation's key range [0, 2^31)");
    if (e & kErrCountOverflow) fail(XLOG_ERR_CAPACITY_EXCEEDED, "count exceeds INT32_MAX");
    if (e & kErrNotSorted) fail(XLOG_ERR_INTERNAL, "invariant violated: keys not strictly increasing");
    fail(XLOG_ERR_INTERNAL, "device error flag set");
  }
}
inline uint32_t* ctrl_u32(Ctx* c, int slot) { return reinterpret_cast<uint32_t*>(c->d_ctrl + slot); }
inline void zero_ctrl(Ctx* c, int slot, int n = 1) {
  XLOG_CUDA(cudaMemsetAsync(c->d_ctrl + slot, 0, n * sizeof(uint64_t), c->stream));
}

inline int bit_length(int64_t v) { int b = 0; while (v > 0) { ++b; v >>= 1; } return std::max(b, 1); }

inline KeyLayout make_layout(int arity, const int32_t* col_max) {
  KeyLayout L{};
  L.arity = arity;
  int bits[kMaxArity], total = 0;
  for (int c = 0; c < arity; ++c) { bits[c] = bit_length(col_max[c]); total += bits[c]; }
  int sh = total;
  for (int c = 0; c < arity; ++c) { sh -= bits[c]; L.shift[c] = sh; L.mask[c] = (uint32_t)((1ull << bits[c]) - 1); }
  L.total_bits = total;
  return L;
}
inline bool same_layout(const KeyLayout& a, const KeyLayout& b) {
  if (a.arity != b.arity || a.total_bits != b.total_bits) return false;
  for (int c = 0; c < a.arity; ++c) if (a.shift[c] != b.shift[c] || a.mask[c] != b.mask[c]) return false;
  return true;
}

// ---------------------------------------------------------------------------------
// typed building blocks
// ---------------------------------------------------------------------------------

// Sort n (key, tag) pairs on key bits [0, nbits).  On return keys/tags point at the sorted data
// (either the original buffers or the alternates).
template <typename K>
inline void sort_pairs(Ctx* c, K*& keys, float*& tags, K*& keys_alt, float*& tags_alt, uint64_t n, int nbits, int low_bit = 0) {
  if (n <= 1) return;
  if (n > kSortMaxN) fail(XLOG_ERR_CAPACITY_EXCEEDED, "a single sort is limited to 2^30 - 1 rows");
  const SortPasses P = make_sort_passes(low_bit, nbits);
  if (P.passes == 0) return;
  const uint32_t ntiles = (uint32_t)((n + sort_tile<K>() - 1) / sort_tile<K>());
  // scratch: digit histograms of every pass, one ticket per pass, a block counter, then the look-back status words of
  // every pass; zeroed by one memset
  const size_t head_words = (size_t)kSortMaxPasses * kSortMaxBins + kSortMaxPasses + 8;
  const size_t pass_words = (size_t)ntiles * kSortMaxBins;
  DevBuf scratch(c, (head_words + pass_words * P.passes) * 4);
  uint32_t* hist = scratch.as<uint32_t>();
  uint32_t* tickets = hist + kSortMaxPasses * kSortMaxBins;
  uint32_t* done = tickets + kSortMaxPasses;
  XLOG_CUDA(cudaMemsetAsync(hist, 0, (head_words + pass_words * P.passes) * 4, c->stream));
  c->note_bytes = (int64_t)n * sizeof(K);
  XLOG_LAUNCH(c, (k_sort_digit_hist<K>), grid_for(n, 256 * 8, kSMs * 8), 256, 0, keys, (uint32_t)n, P, hist, done);
  for (int pass = 0; pass < P.passes; ++pass) {
    uint32_t* status = hist + head_words + pass_words * pass;
    c->note_bytes = (int64_t)n * 2 * (sizeof(K) + 4);
#define XLOG_SORT_PASS(B)                                                                                                          \
  XLOG_LAUNCH(c, (k_sort_pass<K, B>), ntiles, kSortBlock, sort_pass_smem<K>(), keys, reinterpret_cast<const uint32_t*>(tags), keys_alt, \
              reinterpret_cast<uint32_t*>(tags_alt), (uint32_t)n, P.shift[pass], hist + pass * kSortMaxBins, status, tickets + pass,  \
              ctrl_u32(c, kSlotErr), c->spin_limit)
    switch (P.bits[pass]) {
      case 1: XLOG_SORT_PASS(1); break;
      case 2: XLOG_SORT_PASS(2); break;
      case 3: XLOG_SORT_PASS(3); break;
      case 4: XLOG_SORT_PASS(4); break;
      case 5: XLOG_SORT_PASS(5); break;
      case 6: XLOG_SORT_PASS(6); break;
      case 7: XLOG_SORT_PASS(7); break;
      default: XLOG_SORT_PASS(8); break;
    }
#undef XLOG_SORT_PASS
    std::swap(keys, keys_alt);
    std::swap(tags, tags_alt);
  }
}

// Sorted unique (key, tag) list in arena buffers of exact size.
struct KeyTags {
  DevBuf keys, tags;
  uint32_t n = 0;                       // row count; an upper bound (the buffers' capacity) while n_slot >= 0
  int n_slot = -1;                      // >= 0: the exact count is still on the device, in this control slot
  DevBuf head_pos;                      // optional: row index of each group head in the reduced input (+ sentinel n)
};
constexpr size_t kDeferBytes = 32u << 20;   // results up to this size are allocated at their upper bound to skip a control read

constexpr int kSlotA = 8, kSlotB = 9, kSlotC = 10, kSlotD = 11;

// Reduce-by-key of a sorted list.  One control read returns the number of groups; the idle buffers
// `free_a` / `free_b` (the other half of the sort's double buffer) are released at that point, so the
// result can be allocated at its exact size without raising the peak.  head_pos (optional) gets the row
// index of each group's first row plus a sentinel n, so that a group's size is head_pos[u+1] - head_pos[u].
template <typename K, typename Op>
inline KeyTags reduce_by_key_t(Ctx* c, const K* keys, const float* tags, uint32_t n, DevBuf* free_a, DevBuf* free_b, bool want_head_pos,
                               int defer_slot) {
  KeyTags out;
  if (n == 0) { if (free_a) free_a->reset(); if (free_b) free_b->reset(); return out; }
  typedef typename Op::A A;
  const unsigned tiles = (n + kRbkTile - 1) / kRbkTile;
  DevBuf heads(c, (size_t)tiles * 4), tails(c, (size_t)tiles * sizeof(A)), carry(c, (size_t)tiles * sizeof(A));
  c->note_bytes = (int64_t)n * (sizeof(K) + 4);
  XLOG_LAUNCH(c, (k_rbk_tiles<K, Op>), tiles, kRbkBlock, 0, keys, tags, n, heads.as<uint32_t>(), tails.as<A>());
  if (defer_slot >= 0 && !want_head_pos && (size_t)n * (sizeof(K) + 4) <= kDeferBytes) {
    // small result: write it into buffers of the upper-bound size n and leave the exact count on the device
    XLOG_LAUNCH(c, (k_rbk_spine<Op>), 1, 1024, 0, heads.as<uint32_t>(), tails.as<A>(), carry.as<A>(), tiles, ctrl_u32(c, defer_slot));
    if (free_a) free_a->reset();
    if (free_b) free_b->reset();
    out.n = n; out.n_slot = defer_slot;
    out.keys = DevBuf(c, (size_t)n * sizeof(K));
    out.tags = DevBuf(c, (size_t)n * 4);
    c->note_bytes = (int64_t)n * 2 * (sizeof(K) + 4);
    XLOG_LAUNCH(c, (k_rbk_emit<K, Op>), tiles, kRbkBlock, 0, keys, tags, n, heads.as<uint32_t>(), carry.as<A>(), out.keys.as<K>(),
                out.tags.as<float>(), (uint32_t*)nullptr);
    return out;
  }
  XLOG_LAUNCH(c, (k_rbk_spine<Op>), 1, 1024, 0, heads.as<uint32_t>(), tails.as<A>(), carry.as<A>(), tiles, ctrl_u32(c, kSlotA));
  sync_ctrl(c);
  const uint32_t u = (uint32_t)c->h_ctrl[kSlotA];
  if (free_a) free_a->reset();
  if (free_b) free_b->reset();
  out.n = u;
  out.keys = DevBuf(c, (size_t)std::max(u, 1u) * sizeof(K));
  out.tags = DevBuf(c, (size_t)std::max(u, 1u) * 4);
  uint32_t* hp = nullptr;
  if (want_head_pos) { out.head_pos = DevBuf(c, ((size_t)u + 1) * 4); hp = out.head_pos.as<uint32_t>(); }
  c->note_bytes = ((int64_t)n + u) * (sizeof(K) + 4);
  XLOG_LAUNCH(c, (k_rbk_emit<K, Op>), tiles, kRbkBlock, 0, keys, tags, n, heads.as<uint32_t>(), carry.as<A>(), out.keys.as<K>(),
              out.tags.as<float>(), hp);
  if (hp) XLOG_CUDA(cudaMemcpyAsync(hp + u, &n, 4, cudaMemcpyHostToDevice, c->stream));
  return out;
}
template <typename K>
inline KeyTags reduce_by_key(Ctx* c, int sr, const K* keys, const float* tags, uint32_t n, DevBuf* free_a, DevBuf* free_b,
                             bool want_head_pos = false, int defer_slot = -1) {
  switch (sr) {
    case XLOG_SR_MAXPLUS: return reduce_by_key_t<K, OpMax>(c, keys, tags, n, free_a, free_b, want_head_pos, defer_slot);
    case XLOG_SR_MINPLUS: return reduce_by_key_t<K, OpMin>(c, keys, tags, n, free_a, free_b, want_head_pos, defer_slot);
    case XLOG_SR_LOGSUMEXP: return reduce_by_key_t<K, OpLse>(c, keys, tags, n, free_a, free_b, want_head_pos, defer_slot);
    default: return reduce_by_key_t<K, OpSum>(c, keys, tags, n, free_a, free_b, want_head_pos, defer_slot);
  }
}

// max/min reduce-by-key that sorts only the high key bits and reduces each group of equal high
// bits in a shared-memory table (dense_reduce.cuh).  Worth it when groups are well filled.
inline bool dense_reduce_applies(int sr, uint64_t n, int nbits, bool want_head_pos) {
  if (want_head_pos || (sr != XLOG_SR_MAXPLUS && sr != XLOG_SR_MINPLUS)) return false;
  const int H = nbits > kDenseBits ? nbits - kDenseBits : 0;
  if (H > kDenseMaxGroupBits) return false;
  return n >= (1u << 18) && n >= ((uint64_t)32 << H);
}

// presorted_top: the input is already ordered by its top `presorted_top` key bits (see GroupShape), so those
// bits need no sorting; what is left of the group bits is sorted, and the reduced rows are put back into key
// order by a sort on the top bits (the reduced rows are few).
template <typename K, typename Op>
inline KeyTags sort_dense_reduce(Ctx* c, DevBuf& k0, DevBuf& t0, DevBuf& k1, DevBuf& t1, uint64_t n, int nbits, int defer_slot,
                                 int presorted_top) {
  KeyTags out;
  K* ka = k0.as<K>(); K* kb = k1.as<K>();
  float* ta = t0.as<float>(); float* tb = t1.as<float>();
  const int L = std::min(nbits, kDenseBits), H = nbits - L;
  const uint32_t G = 1u << H;
  GroupShape GS{L, H, 0};
  if (presorted_top >= H) {
    // every group bit is already in order: no radix pass at all (M = H, T = 0 describes plain key order)
  } else if (presorted_top > 0) {
    GS.T = presorted_top; GS.M = H - presorted_top;
    sort_pairs<K>(c, ka, ta, kb, tb, n, nbits - presorted_top, L);     // middle bits only; rows end up ordered by (mid, top)
    defer_slot = -1;                                                   // the reorder below needs the exact row count
  } else {
    sort_pairs<K>(c, ka, ta, kb, tb, n, nbits, L);                     // all group bits
  }
  uint32_t part = (uint32_t)std::min<uint64_t>(std::max<uint64_t>(n / (kSMs * 8), 8192), 131072);
  part = (part + 1023) / 1024 * 1024;
  const uint32_t spill_cap = std::min<uint32_t>((uint32_t)(n / part) + 1, G), max_items = (uint32_t)(n / part) + G + 1;
  DevBuf gstart(c, ((size_t)G + 1) * 4), part_base(c, ((size_t)G + 1) * 4), spill(c, (size_t)G * 4), done(c, (size_t)G * 4),
      ucount(c, ((size_t)G + 1) * 4), spill_tab(c, (size_t)spill_cap * kDenseSlots * 4);
  XLOG_CUDA(cudaMemsetAsync(ucount.p, 0, ((size_t)G + 1) * 4, c->stream));
  XLOG_LAUNCH(c, (k_group_bounds<K>), grid_for((uint64_t)G + 1, 256), 256, 0, (const K*)ka, (uint32_t)n, GS, G, gstart.as<uint32_t>());
  XLOG_LAUNCH(c, k_group_plan, 1, 1024, 0, (const uint32_t*)gstart.as<uint32_t>(), G, part, part_base.as<uint32_t>(), spill.as<uint32_t>(),
              done.as<uint32_t>(), ctrl_u32(c, kSlotB));
  XLOG_LAUNCH(c, k_fill_i32, grid_for((uint64_t)spill_cap * kDenseSlots, 256 * 8), 256, 0, spill_tab.as<int32_t>(),
              (uint64_t)spill_cap * kDenseSlots, DenseOp<Op>::empty);
  c->note_bytes = (int64_t)n * (sizeof(K) + 4);
  XLOG_LAUNCH(c, (k_dense_reduce<K, Op>), max_items, kDenseBlock, 0, (const K*)ka, (const float*)ta, GS, G, part,
              (const uint32_t*)gstart.as<uint32_t>(), (const uint32_t*)part_base.as<uint32_t>(), (const uint32_t*)spill.as<uint32_t>(), spill_cap,
              spill_tab.as<int32_t>(), done.as<uint32_t>(), kb, tb, ucount.as<uint32_t>());
  const bool sorted_in_0 = (void*)ka == k0.p;
  const uint64_t ucap = std::min<uint64_t>(n, nbits >= 32 ? n : ((uint64_t)1 << nbits));
  if (defer_slot >= 0 && ucap * (sizeof(K) + 4) <= kDeferBytes) {
    // small result: compact into buffers of the upper-bound size and leave the exact count on the device
    XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, ucount.as<uint32_t>(), (int64_t)G + 1, ctrl_u32(c, defer_slot));
    (sorted_in_0 ? k0 : k1).reset();
    (sorted_in_0 ? t0 : t1).reset();
    spill_tab.reset();
    out.n = (uint32_t)ucap; out.n_slot = defer_slot;
    out.keys = DevBuf(c, (size_t)ucap * sizeof(K));
    out.tags = DevBuf(c, (size_t)ucap * 4);
    XLOG_LAUNCH(c, (k_dense_compact<K>), grid_for(ucap, 256), 256, 0, (const K*)kb, (const float*)tb, (const uint32_t*)gstart.as<uint32_t>(),
                (const uint32_t*)ucount.as<uint32_t>(), G, (const uint32_t*)ctrl_u32(c, defer_slot), out.keys.as<K>(), out.tags.as<float>());
    k0.reset(); t0.reset(); k1.reset(); t1.reset();
    return out;
  }
  XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, ucount.as<uint32_t>(), (int64_t)G + 1, ctrl_u32(c, kSlotA));
  sync_ctrl(c);
  out.n = (uint32_t)c->h_ctrl[kSlotA];
  (sorted_in_0 ? k0 : k1).reset();
  (sorted_in_0 ? t0 : t1).reset();
  spill_tab.reset();
  out.keys = DevBuf(c, (size_t)std::max(out.n, 1u) * sizeof(K));
  out.tags = DevBuf(c, (size_t)std::max(out.n, 1u) * 4);
  if (out.n) {
    c->note_bytes = (int64_t)out.n * 2 * (sizeof(K) + 4);
    XLOG_LAUNCH(c, (k_dense_compact<K>), grid_for(out.n, 256), 256, 0, (const K*)kb, (const float*)tb, (const uint32_t*)gstart.as<uint32_t>(),
                (const uint32_t*)ucount.as<uint32_t>(), G, (const uint32_t*)ctrl_u32(c, kSlotA), out.keys.as<K>(), out.tags.as<float>());
  }
  k0.reset(); t0.reset(); k1.reset(); t1.reset();
  if (GS.T && out.n > 1) {
    // rows are ordered by (mid, top, low): a stable sort on the top bits restores key order (top, mid, low)
    DevBuf ak(c, (size_t)out.n * sizeof(K)), at(c, (size_t)out.n * 4);
    K* pk = out.keys.as<K>(); K* qk = ak.as<K>();
    float* pt = out.tags.as<float>(); float* qt = at.as<float>();
    sort_pairs<K>(c, pk, pt, qk, qt, out.n, nbits, nbits - GS.T);
    if ((void*)pk != out.keys.p) { std::swap(out.keys, ak); std::swap(out.tags, at); }
  }
  return out;
}

// Sort + reduce the first n pairs of (k0,t0) using (k1,t1) as the second half of the double
// buffer; releases both and returns the groups in exact-size buffers.
template <typename K>
inline KeyTags sort_reduce(Ctx* c, int sr, DevBuf& k0, DevBuf& t0, DevBuf& k1, DevBuf& t1, uint64_t n, int nbits, bool want_head_pos,
                           int defer_slot = -1, int presorted_top = 0) {
  if (dense_reduce_applies(sr, n, nbits, want_head_pos))
    return sr == XLOG_SR_MAXPLUS ? sort_dense_reduce<K, OpMax>(c, k0, t0, k1, t1, n, nbits, defer_slot, presorted_top)
                                 : sort_dense_reduce<K, OpMin>(c, k0, t0, k1, t1, n, nbits, defer_slot, presorted_top);
  K* ka = k0.as<K>(); K* kb = k1.as<K>();
  float* ta = t0.as<float>(); float* tb = t1.as<float>();
  // Candidates that arrive ordered by their top key bits need only their low bits sorted for equal keys to become
  // neighbours (a stable sort: rows end up ordered by (low, top), each key's candidates in their arrival order, so a
  // floating-point oplus sees them as the full sort would show them); the groups, far fewer than the candidates,
  // are then put in key order by a stable sort on the top bits.
  const bool top_presorted = presorted_top > 0 && presorted_top < nbits && !want_head_pos && defer_slot < 0;
  sort_pairs<K>(c, ka, ta, kb, tb, n, top_presorted ? nbits - presorted_top : nbits);
  const bool sorted_in_0 = (void*)ka == k0.p;
  KeyTags out = reduce_by_key<K>(c, sr, ka, ta, (uint32_t)n, sorted_in_0 ? &k1 : &k0, sorted_in_0 ? &t1 : &t0, want_head_pos, defer_slot);
  k0.reset(); t0.reset(); k1.reset(); t1.reset();
  if (top_presorted && out.n > 1) {
    DevBuf ak(c, (size_t)out.n * sizeof(K)), at(c, (size_t)out.n * 4);
    K* pk = out.keys.as<K>(); K* qk = ak.as<K>();
    float* pt = out.tags.as<float>(); float* qt = at.as<float>();
    sort_pairs<K>(c, pk, pt, qk, qt, out.n, nbits, nbits - presorted_top);
    if ((void*)pk != out.keys.p) { std::swap(out.keys, ak); std::swap(out.tags, at); }
  }
  return out;
}

// Merge A (reduced candidates) into B (full): returns full' and, if want_delta, delta'.
// If no key of A is new, B's tags are updated in place and full' stays empty (n_new == 0).
struct MergeResult {
  KeyTags full, delta;
  uint32_t n_new = 0, n_improved = 0;
  bool in_place = false;
  int slot = -1;                        // >= 0: totals are still on the device (slot: merged rows, slot + 1: delta rows)
  uint32_t nb = 0;
  bool allow_in_place = false;
};

// Read the totals of a deferred merge from the (already synchronised) control block and settle sizes.
inline void finish_merge(Ctx* c, MergeResult& r) {
  if (r.slot < 0) return;
  const uint32_t tot_f = (uint32_t)c->h_ctrl[r.slot], tot_d = (uint32_t)c->h_ctrl[r.slot + 1];
  r.n_new = tot_f - r.nb;
  r.n_improved = tot_d - r.n_new;
  r.in_place = r.allow_in_place && r.n_new == 0;
  if (r.in_place) { r.full.keys.reset(); r.full.tags.reset(); r.full.n = 0; } else r.full.n = tot_f;
  r.delta.n = tot_d;
  r.full.n_slot = r.delta.n_slot = -1;
  r.slot = -1;
}

// na_slot >= 0: A's exact row count is still on the device (na is then its upper bound).
// defer_slot >= 0: if the upper-bound outputs are small, allocate them at once and skip the control read between the
// count pass and the emit pass; finish_merge() settles the sizes after the caller's next control read.
template <typename K, typename Op>
inline MergeResult merge_t(Ctx* c, const K* A, const float* TA, uint32_t na, int na_slot, const K* B, float* TB, uint32_t nb,
                           bool want_delta, bool allow_in_place, int defer_slot) {
  MergeResult r;
  const uint64_t total = (uint64_t)na + nb;
  const unsigned tiles = (unsigned)((total + kMrgTile - 1) / kMrgTile);
  if (tiles == 0) return r;
  const uint32_t* na_ptr = na_slot >= 0 ? ctrl_u32(c, na_slot) : nullptr;
  DevBuf a_start(c, ((size_t)tiles + 1) * 4), nf(c, (size_t)tiles * 4), nd(c, (size_t)tiles * 4);
  XLOG_LAUNCH(c, (k_merge_partition<K>), (tiles + 1 + 255) / 256, 256, 0, A, na, na_ptr, B, nb, tiles, a_start.as<uint32_t>());
  c->note_bytes = (int64_t)total * (sizeof(K) + 4);
  XLOG_LAUNCH(c, (k_merge<K, Op, false>), tiles, kMrgBlock, 0, A, TA, na, na_ptr, B, TB, nb, a_start.as<uint32_t>(), nf.as<uint32_t>(),
              nd.as<uint32_t>(), (K*)nullptr, (float*)nullptr, (K*)nullptr, (float*)nullptr, 0, (const uint32_t*)nullptr);
  const bool defer = defer_slot >= 0 && want_delta && total * (sizeof(K) + 4) <= 2 * kDeferBytes;
  if (defer) {
    XLOG_LAUNCH(c, (k_scan_spine2<uint32_t>), 1, 1024, 0, nf.as<uint32_t>(), nd.as<uint32_t>(), (int64_t)tiles, ctrl_u32(c, defer_slot),
                ctrl_u32(c, defer_slot + 1));
    r.slot = defer_slot; r.nb = nb; r.allow_in_place = allow_in_place;
    r.full.n = (uint32_t)total; r.delta.n = std::max(na, 1u);
    r.full.keys = DevBuf(c, (size_t)total * sizeof(K));
    r.full.tags = DevBuf(c, (size_t)total * 4);
    r.delta.keys = DevBuf(c, (size_t)std::max(na, 1u) * sizeof(K));
    r.delta.tags = DevBuf(c, (size_t)std::max(na, 1u) * 4);
    c->note_bytes = (int64_t)total * 2 * (sizeof(K) + 4);
    XLOG_LAUNCH(c, (k_merge<K, Op, true>), tiles, kMrgBlock, 0, A, TA, na, na_ptr, B, TB, nb, a_start.as<uint32_t>(), nf.as<uint32_t>(),
                nd.as<uint32_t>(), r.full.keys.as<K>(), r.full.tags.as<float>(), r.delta.keys.as<K>(), r.delta.tags.as<float>(),
                allow_in_place ? -1 : 0, (const uint32_t*)ctrl_u32(c, defer_slot));
    return r;
  }
  XLOG_LAUNCH(c, (k_scan_spine2<uint32_t>), 1, 1024, 0, nf.as<uint32_t>(), nd.as<uint32_t>(), (int64_t)tiles, ctrl_u32(c, kSlotB), ctrl_u32(c, kSlotC));
  sync_ctrl(c);
  const uint32_t tot_f = (uint32_t)c->h_ctrl[kSlotB], tot_d = (uint32_t)c->h_ctrl[kSlotC];
  r.n_new = tot_f - nb;
  r.n_improved = tot_d - r.n_new;
  r.in_place = allow_in_place && r.n_new == 0;
  if (r.in_place && tot_d == 0) return r;             // nothing new, nothing improved
  if (!r.in_place) {
    r.full.n = tot_f;
    r.full.keys = DevBuf(c, (size_t)tot_f * sizeof(K));
    r.full.tags = DevBuf(c, (size_t)tot_f * 4);
  }
  // delta buffers are always written by the emit kernel (they are small); size >= 1 keeps pointers valid
  r.delta.n = tot_d;
  r.delta.keys = DevBuf(c, (size_t)std::max(tot_d, 1u) * sizeof(K));
  r.delta.tags = DevBuf(c, (size_t)std::max(tot_d, 1u) * 4);
  c->note_bytes = ((int64_t)total + (r.in_place ? 0 : tot_f) + tot_d) * (sizeof(K) + 4);
  XLOG_LAUNCH(c, (k_merge<K, Op, true>), tiles, kMrgBlock, 0, A, TA, na, na_ptr, B, TB, nb, a_start.as<uint32_t>(), nf.as<uint32_t>(),
              nd.as<uint32_t>(), r.full.keys.as<K>(), r.full.tags.as<float>(), r.delta.keys.as<K>(), r.delta.tags.as<float>(),
              r.in_place ? 1 : 0, (const uint32_t*)nullptr);
  if (!want_delta) { r.delta.keys.reset(); r.delta.tags.reset(); r.delta.n = 0; }
  return r;
}
template <typename K>
inline MergeResult merge(Ctx* c, int sr, const K* A, const float* TA, uint32_t na, int na_slot, const K* B, float* TB, uint32_t nb,
                         bool want_delta, bool allow_in_place, int defer_slot = -1) {
  switch (sr) {
    case XLOG_SR_MAXPLUS: return merge_t<K, OpMax>(c, A, TA, na, na_slot, B, TB, nb, want_delta, allow_in_place, defer_slot);
    case XLOG_SR_MINPLUS: return merge_t<K, OpMin>(c, A, TA, na, na_slot, B, TB, nb, want_delta, allow_in_place, defer_slot);
    case XLOG_SR_LOGSUMEXP: return merge_t<K, OpLse>(c, A, TA, na, na_slot, B, TB, nb, want_delta, false, defer_slot);
    default: return merge_t<K, OpSum>(c, A, TA, na, na_slot, B, TB, nb, want_delta, false, defer_slot);
  }
}

}  // namespace xlog
