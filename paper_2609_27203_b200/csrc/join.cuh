// Join of an outer relation (the delta, or a full relation in the seed round) with an indexed
// inner relation, fused with head projection and the otimes of the tags (paper kernel table:
// `join`, count -> scan -> materialise; Algorithm 1 lines 5-6; RIR `Project`).
//
// The paper's join is a chained hash join over FNV-1a hashes.  Here the inner side is a sorted
// column store with an offsets array over its probed column (keys are dense ids), so a probe is
// two offset reads, and materialisation is tiled by OUTPUT position: every block produces the
// same number of candidates no matter how skewed the degrees are.
#pragma once
#include "common.cuh"

namespace xlog {

struct ArgSpec { int kind; int var; int mul; int add; };      // kind 0: constant `add`; 1: column == mul*var + add

struct JoinSpec {
  // outer side: packed keys + tags
  KeyLayout outer;
  ArgSpec outer_args[kMaxArity];
  DictSet outer_dict;                                         // dictionaries of the outer relation's columns
  int outer_decode[kMaxArity];                                // 1: turn the stored code into the value when binding

  // inner side (absent for one-atom rules): offsets over the probed column, the other columns, tags
  int has_inner;
  int probe_var, probe_mul, probe_add;                        // probed value = probe_mul * var + probe_add
  int64_t inner_domain;                                       // offsets has inner_domain + 1 entries
  const uint32_t* inner_off;
  int inner_free;                                             // number of non-probed inner columns
  const int32_t* inner_col[kMaxArity - 1];
  int inner_var[kMaxArity - 1];                               // variable bound by each non-probed column (pattern var + add)
  int inner_add[kMaxArity - 1];
  const float* inner_tag;
  // head
  KeyLayout head;
  DictSet head_dict;                                          // dictionaries of the head relation's columns
  int head_encode[kMaxArity];                                 // 1: the head expression yields a value that must be ranked;
                                                              // 0 with a dictionary: the variable already carries the code
  int64_t head_c0[kMaxArity];
  int32_t head_coef[kMaxArity][kMaxVars];
  int times;                                                  // otimes: 0 = add, 1 = multiply
  // negated second atom (negation as failure): a row of the scanned atom survives iff the other relation has no row
  // whose first neg_prefix (1 or 2) columns equal the given constants / variables
  int neg_prefix;                                             // 0: no negated atom
  ArgSpec neg_args[2];
  int64_t neg_domain;
  const uint32_t* neg_off;                                    // offsets over the negated relation's first column
  const int32_t* neg_col1;                                    // its second column (sorted inside each first-column run)
  // simple shape (a fast shape whose scanned atom binds each column to a constant or to a distinct bare variable, without
  // dictionaries, and whose head columns each take a constant plus at most one of those variables): the per-row work
  // is a handful of shifts and masks on the packed key instead of the general binding / affine evaluation
  int simple;
  uint64_t s_const_mask, s_const_val;                         // (key & mask) == val: every constant column matches
  int s_probe_shift; uint32_t s_probe_mask;                   // column that binds the probe variable
  int s_src_shift[kMaxArity]; uint32_t s_src_mask[kMaxArity]; // per head column: the outer column it copies (mask 0: none)
  uint32_t s_c0[kMaxArity];
  // fast shape: head key = row part + sum_j inner_col[j] * inner_mult[j]
  int fast;
  int32_t head_coef_outer[kMaxArity][kMaxVars];               // head_coef restricted to variables the outer atom binds
  uint64_t inner_mult[kMaxArity - 1];
};

// Decode an outer row into variable values; false if a constant / repeated variable /
// divisibility test fails.
template <typename KO>
__device__ __forceinline__ bool bind_outer(const JoinSpec& S, KO key, int64_t* var) {
  bool ok = true;
  bool bound[kMaxVars];
#pragma unroll
  for (int v = 0; v < kMaxVars; ++v) { bound[v] = false; var[v] = 0; }
#pragma unroll
  for (int c = 0; c < kMaxArity; ++c) {
    if (c < S.outer.arity) {
      int64_t val = key_col<KO>(S.outer, key, c);
      if (S.outer_decode[c]) val = S.outer_dict.v[c][min((uint32_t)val, S.outer_dict.n[c] - 1)];
      const ArgSpec a = S.outer_args[c];
      if (a.kind == 0) ok = ok && val == a.add;
      else {
        const int64_t d = val - a.add;
        int64_t q = d;
        bool divides = true;
        if (a.mul != 1) { q = d / a.mul; divides = q * a.mul == d; }       // the 64-bit division is rare: keep it off the common path
#pragma unroll
        for (int v = 0; v < kMaxVars; ++v)
          if (v == a.var) {
            if (bound[v]) ok = ok && divides && var[v] == q;
            else { ok = ok && divides; var[v] = q; bound[v] = true; }
          }
      }
    }
  }
  return ok;
}

// One thread per outer row: degree (number of inner matches) and a 16-byte row record
// {first matching inner row, outer tag, row part of the head key}.  In the fast shape the head key
// is linear in the inner columns, key = rowkey + sum_j inner_col_j * inner_mult[j], so everything that
// depends on the outer row alone (constants, outer variables, dictionary ranks, range checks) is done
// here once per row instead of once per candidate.
// The row is given by value (its packed key and tag); rowinfo == nullptr: the degree only, nothing is written.
template <typename KO>
__device__ __forceinline__ uint32_t join_count_kv(const JoinSpec& S, const KO okey, const float otag, uint32_t i, uint4* __restrict__ rowinfo,
                                                  uint32_t* __restrict__ err) {
  int64_t var[kMaxVars];
  uint32_t d = 0, lo = 0;
  uint64_t rowkey = 0;
  if (S.simple) {
    const uint64_t k = (uint64_t)okey;
    if ((k & S.s_const_mask) == S.s_const_val) {
      d = 1;
      if (S.has_inner) {
        const int64_t pv = (int64_t)((uint32_t)(k >> S.s_probe_shift) & S.s_probe_mask) * S.probe_mul + S.probe_add;
        d = 0;
        if (pv >= 0 && pv < S.inner_domain) {
          lo = S.inner_off[pv];
          d = S.inner_off[pv + 1] - lo;
        }
      }
      if (d) {
        uint32_t e = 0;
#pragma unroll
        for (int c = 0; c < kMaxArity; ++c)
          if (c < S.head.arity) {
            uint64_t h = (uint64_t)S.s_c0[c] + ((uint32_t)(k >> S.s_src_shift[c]) & S.s_src_mask[c]);
            if (h > (uint64_t)S.head.mask[c]) { e |= kErrHeadRange; h = 0; }
            rowkey |= h << S.head.shift[c];
          }
        if (e) atomicOr(err, e);
      }
    }
  } else if (bind_outer<KO>(S, okey, var)) {
    if (S.neg_prefix) {
      int64_t val[2] = {0, 0};
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const ArgSpec a = S.neg_args[k];
        int64_t x = 0;
#pragma unroll
        for (int v = 0; v < kMaxVars; ++v) if (v == a.var) x = var[v];
        val[k] = a.kind == 0 ? (int64_t)a.add : x * a.mul + a.add;
      }
      bool exists = false;
      if (val[0] >= 0 && val[0] < S.neg_domain) {
        uint32_t a0 = S.neg_off[val[0]], a1 = S.neg_off[val[0] + 1];
        if (S.neg_prefix == 1) exists = a1 > a0;
        else {
          while (a0 < a1) { const uint32_t mid = a0 + ((a1 - a0) >> 1); if ((int64_t)S.neg_col1[mid] < val[1]) a0 = mid + 1; else a1 = mid; }
          exists = a0 < S.neg_off[val[0] + 1] && (int64_t)S.neg_col1[a0] == val[1];
        }
      }
      d = exists ? 0 : 1;
    } else if (!S.has_inner) d = 1;
    else {
      int64_t pv = 0;
#pragma unroll
      for (int v = 0; v < kMaxVars; ++v) if (v == S.probe_var) pv = var[v];
      pv = pv * S.probe_mul + S.probe_add;
      if (pv >= 0 && pv < S.inner_domain) {
        lo = S.inner_off[pv];
        d = S.inner_off[pv + 1] - lo;
      }
    }
    if (S.fast && d) {
      uint32_t e = 0;
#pragma unroll
      for (int c = 0; c < kMaxArity; ++c)
        if (c < S.head.arity) {
          int64_t h = S.head_c0[c];
#pragma unroll
          for (int v = 0; v < kMaxVars; ++v) h += (int64_t)S.head_coef_outer[c][v] * var[v];
          if (S.head_encode[c]) {
            const uint32_t r = dict_rank(S.head_dict.v[c], S.head_dict.n[c], h);
            if (r >= S.head_dict.n[c] || (int64_t)S.head_dict.v[c][r] != h) { e |= kErrInternal; h = 0; } else h = r;
          }
          if (h < 0 || h > (int64_t)S.head.mask[c]) { e |= kErrHeadRange; h = 0; }
          rowkey |= (uint64_t)h << S.head.shift[c];
        }
      if (e) atomicOr(err, e);
    }
  }
  if (rowinfo) rowinfo[i] = make_uint4(lo, __float_as_uint(otag), (uint32_t)rowkey, (uint32_t)(rowkey >> 32));
  return d;
}

template <typename KO>
__device__ __forceinline__ uint32_t join_count_row(const JoinSpec& S, const KO* __restrict__ okeys, const float* __restrict__ otags, uint32_t i,
                                                   uint4* __restrict__ rowinfo, uint32_t* __restrict__ err) {
  return join_count_kv<KO>(S, okeys[i], otags[i], i, rowinfo, err);
}

template <typename KO>
__global__ void __launch_bounds__(256) k_join_count(JoinSpec S, const KO* __restrict__ okeys, const float* __restrict__ otags,
                                                    uint32_t n_outer, uint32_t* __restrict__ deg, uint4* __restrict__ rowinfo,
                                                    uint32_t* __restrict__ err) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_outer) deg[i] = join_count_row<KO>(S, okeys, otags, i, rowinfo, err);
}

// Tile shape of the materialising kernel.  The tag-mirror sinks are bound by the latency of one random L2 sector per
// candidate, so what counts is how many slot reads an SM keeps in flight: resident warps first, items per thread second.
// Measured on the two large workloads (single-source R-MAT 20 / 64-source R-MAT 22, ms per fixpoint; items, staged
// rows, blocks per SM): 8, 1024, 5: 0.62 / 34.6; 8, 1024, 6: 0.63 / 32.7; 6, 768, 6: 0.60 / 31.5; 6, 768, 7: 0.61 / 29.3;
// 4, 512, 8 (64 warps, no spills): 0.58 / 29.0.
// The kernel that writes candidates (streaming) keeps 8 items per thread; it, too, gains from residency: on the 64-source
// workload 2048 staged rows at 5 blocks per SM ran at 2.9 TB/s of algorithmic traffic, 1024 rows at 8 blocks (32 registers) at 3.9 TB/s.
constexpr int kExpBlock = 256;
constexpr int kExpMirrorBlocksPerSM = 8;
constexpr int kExpWriteBlocksPerSM = 8;               // and of the candidate-writing ones
template <bool MIRROR> struct ExpShapeT {
  static constexpr int items = MIRROR ? 4 : 8;        // candidates per thread
  static constexpr int tile = kExpBlock * items;      // candidates per block
  static constexpr int rows = MIRROR ? 512 : 1024;    // outer rows staged in shared memory per tile
};
constexpr int kExpTileWrite = ExpShapeT<false>::tile, kExpTileMirror = ExpShapeT<true>::tile;

// Backward pass of a logsumexp / sum rule: instead of writing the candidate, look its head row up
// and scatter the gradient to the two body rows (Section "End-to-end training": exact gradients
// of a query value with respect to the weighted facts).
struct BwdArgs {
  const void* head_keys;        // stored head relation: packed keys (KH), ascending
  const float* head_tags;       // its tags (the forward result)
  uint32_t n_head;
  int count_bits;               // a counted head stores (declared columns, count): compare keys >> count_bits
  const float* grad_head;       // upstream gradient per head row
  float* grad_outer;            // per row of the scanned atom's relation
  float* grad_inner;            // per row of the looked-up atom's relation (NULL for one-atom rules)
  int lse;                      // 1: logsumexp weights, 0: sum-product
};

enum { kExpFast = 0, kExpGeneric = 1, kExpBackward = 2 };

// Where a candidate goes.  kSinkWrite: into the candidate arrays (to be sorted and reduced).  kSinkMin / kSinkMax:
// straight into the head relation's tag mirror, a table with one order-mapped tag per possible head key
// (max / min are idempotent and order-independent, so "oplus into the slot" is one atomic and needs no sort).
// A candidate that is better than what its slot holds issues the atomic and sets the key's bit in `changed`, both as
// fire-and-forget reductions: no thread ever waits for an atomic's result.  (If another candidate lowers the slot
// between the read and the atomic, the key has changed in this round all the same, so the bit is right either way.)
// The slot is read first because most candidates of a fixpoint round do not improve anything.  Which of the changed
// keys are new is settled when the bitmap is compacted, against a bitmap of the keys the relation already holds.
enum { kSinkWrite = 0, kSinkMin = 1, kSinkMax = 2 };
struct MirrorArgs {
  int32_t* table;               // 2^key_bits order-mapped tags; kMirrorEmptyMin / kMirrorEmptyMax where no tuple is
  uint32_t* changed;            // one bit per key
  unsigned long long* n_new;    // running count of keys that entered the relation (kept by the compaction kernels)
  uint32_t key_max;             // last valid key; anything above raises the head-range error instead of being stored
  uint32_t* err;
};
constexpr int32_t kMirrorEmptyMin = 0x7fffffff;
constexpr int32_t kMirrorEmptyMax = (int32_t)0x80000000;

// The pre-check may read a stale slot: slots only ever move towards the better value, so a stale value can only make a
// candidate look better than it is, and the atomic that follows decides.  The grouped joins read whole lines of a table
// far larger than L2 and bypass L1 (measured on the 64-source workload: 6.77 ms against 7.06 ms through L1); the
// row-wise join reads one slot per candidate of a table that fits L2, and on skewed graphs the slots of the hub nodes
// then hit in L1 (single-source R-MAT 20: 0.514 -> 0.465 ms per fixpoint), so it takes the default cached load.
#ifndef XLOG_TABLE_LOAD
#define XLOG_TABLE_LOAD(p) __ldcg(p)
#endif
#ifndef XLOG_TABLE_LOAD_ROWWISE
#define XLOG_TABLE_LOAD_ROWWISE(p) (*(p))
#endif

template <int SINK>
__device__ __forceinline__ void mirror_commit(const MirrorArgs& m, uint32_t key, int32_t v) {
  if (SINK == kSinkMin) atomicMin(m.table + key, v); else atomicMax(m.table + key, v);
  atomicOr(m.changed + (key >> 5), 1u << (key & 31));
}
template <int SINK>
__device__ __forceinline__ void mirror_apply(const MirrorArgs& m, uint32_t key, float tag) {
  const int32_t v = f2ord(tag);
  if (key > m.key_max) { atomicOr(m.err, kErrHeadRange); return; }
  const int32_t cur = __ldcg(m.table + key);
  if (SINK == kSinkMin ? v < cur : v > cur) mirror_commit<SINK>(m, key, v);
}

// One thread per tile: the first and last outer row that contribute candidates to the tile
// (r_lo = last row with start <= tile begin, r_hi = last row with start < tile end).  Done for all
// tiles at once so that the dependent binary-search loads of one tile overlap with those of the others.
static __global__ void __launch_bounds__(256) k_expand_partition(const uint64_t* __restrict__ start, uint32_t n_outer, uint64_t out_lo,
                                                                 uint64_t out_hi, uint32_t ntiles, uint32_t tile, uint2* __restrict__ tile_rows) {
  const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= ntiles) return;
  const uint64_t t_lo = out_lo + (uint64_t)t * tile;
  const uint64_t t_hi = min(t_lo + tile, out_hi);
  uint32_t r[2];
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const uint64_t target = k == 0 ? t_lo : t_hi - 1;
    uint32_t lo = 0, hi = n_outer;                    // upper_bound(start, target) - 1
    while (lo < hi) {
      const uint32_t mid = lo + ((hi - lo) >> 1);
      if (start[mid] <= target) lo = mid + 1; else hi = mid;
    }
    r[k] = lo - 1;
  }
  tile_rows[t] = make_uint2(r[0], r[1]);
}

template <typename SH> struct ExpSmem {
  uint32_t sstart[SH::rows];
  uint4 sinfo[SH::rows];
  uint16_t srowidx[SH::tile];             // staged row of every candidate position of the tile
  uint32_t swarp[kExpBlock / 32];
};

// Candidates [t_lo, t_hi) (one tile, at most SH::tile of them), covered by outer rows tr.x .. tr.y.  Called by all
// threads of a block; error bits go to `e` (the caller flushes them).
template <typename KO, typename KH, int MODE, int SINK>
__device__ __forceinline__ void expand_tile(ExpSmem<ExpShapeT<SINK != kSinkWrite>>& sm, const JoinSpec& S, const KO* __restrict__ okeys, uint32_t n_outer,
                                            const uint64_t* __restrict__ start, const uint4* __restrict__ rowinfo, const uint2 tr,
                                            const uint64_t t_lo, const uint64_t t_hi, const uint64_t out_lo, KH* __restrict__ ckeys,
                                            float* __restrict__ ctags, const BwdArgs& bw, const MirrorArgs& mr, uint32_t& e) {
  typedef ExpShapeT<SINK != kSinkWrite> SH;
  constexpr int kExpItems = SH::items, kExpRows = SH::rows;
  uint32_t* sstart = sm.sstart;
  uint4* sinfo = sm.sinfo;
  uint16_t* srowidx = sm.srowidx;
  uint32_t* swarp = sm.swarp;
#pragma unroll
  for (int i = 0; i < kExpItems; ++i) srowidx[i * kExpBlock + threadIdx.x] = 0;
  const uint32_t r_lo = tr.x, r_hi = tr.y;
  const uint32_t nrows = r_hi - r_lo + 1;
  const bool staged = nrows <= kExpRows;
  const uint64_t first_start = start[r_lo];
  if (staged) {
    for (uint32_t i = threadIdx.x; i < nrows; i += kExpBlock) {
      const uint64_t st = start[r_lo + i];
      const uint32_t rel = st <= t_lo ? 0u : (uint32_t)(st - t_lo);    // only the first row can start before the tile
      sstart[i] = rel;
      sinfo[i] = rowinfo[r_lo + i];
    }
    __syncthreads();
    // mark the position where each row with at least one match starts (rows without matches share a start with
    // their successor and are skipped), then a running maximum turns the marks into "row of position q"
    for (uint32_t i = threadIdx.x; i < nrows; i += kExpBlock) {
      const uint32_t rel = sstart[i];
      const uint32_t nxt = i + 1 < nrows ? sstart[i + 1] : (uint32_t)(t_hi - t_lo);
      if (i > 0 && nxt > rel) srowidx[rel] = (uint16_t)i;
    }
    __syncthreads();
    uint32_t loc[kExpItems];
    uint32_t run = 0;
#pragma unroll
    for (int i = 0; i < kExpItems; ++i) { run = max(run, (uint32_t)srowidx[threadIdx.x * kExpItems + i]); loc[i] = run; }
    uint32_t incl = run;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d); if ((int)lane_id() >= d) incl = max(incl, o); }
    if (lane_id() == 31) swarp[warp_id()] = incl;
    __syncthreads();
    uint32_t carry = 0;
    for (int w = 0; w < (int)warp_id(); ++w) carry = max(carry, swarp[w]);
    const uint32_t prev = __shfl_up_sync(0xffffffffu, incl, 1);
    if (lane_id() > 0) carry = max(carry, prev);
#pragma unroll
    for (int i = 0; i < kExpItems; ++i) srowidx[threadIdx.x * kExpItems + i] = (uint16_t)max(loc[i], carry);
  }
  __syncthreads();

  if (MODE == kExpFast && staged) {
    // lean loop of the common case: everything per row is in shared memory; all indices are 32-bit
    const uint32_t ntile = (uint32_t)(t_hi - t_lo);
    const uint32_t j0 = (uint32_t)(t_lo - first_start);              // candidates of the first row that precede the tile
    KH* __restrict__ kout = ckeys + (t_lo - out_lo);
    float* __restrict__ tout = ctags + (t_lo - out_lo);
    const float* __restrict__ itg = S.inner_tag;
    const int32_t* __restrict__ ic0 = S.inner_col[0];
    const KH m0 = (KH)S.inner_mult[0];
    const int nin = S.has_inner ? S.inner_free : -1;                 // -1: one-atom rule
    const bool times = S.times != 0;
    if (SINK == kSinkWrite) {
      // everything per candidate is one (or a few) coalesced inner reads, one multiply-add and two coalesced writes
#pragma unroll
      for (int k = 0; k < kExpItems; ++k) {
        const uint32_t q = threadIdx.x + k * kExpBlock;
        if (q < ntile) {
          const uint32_t li = srowidx[q];
          const uint4 info = sinfo[li];
          const uint32_t ir = info.x + (li ? q - sstart[li] : q + j0);
          KH key = (KH)(((uint64_t)info.w << 32) | info.z);
          float tag = __uint_as_float(info.y);
          if (nin >= 0) {
            const float it = itg[ir];
            tag = times ? tag * it : tag + it;
            if (nin >= 1) key += (KH)(uint32_t)ic0[ir] * m0;
            for (int c = 1; c < nin; ++c) key += (KH)(uint32_t)S.inner_col[c][ir] * (KH)S.inner_mult[c];
          }
          kout[q] = key;
          tout[q] = tag;
        }
      }
    } else {
    // tag mirror: three sweeps over the thread's items, so that the loads of one kind are all in flight together:
    // (1) row record from shared memory, inner tag and columns from global memory; (2) the current slot values;
    // (3) the atomics of the few candidates that improve their slot
    KH key[kExpItems];
    float tag[kExpItems];
#pragma unroll
    for (int k = 0; k < kExpItems; ++k) {
      const uint32_t q = threadIdx.x + k * kExpBlock;
      key[k] = 0; tag[k] = 0.f;
      if (q < ntile) {
        const uint32_t li = srowidx[q];
        const uint4 info = sinfo[li];
        const uint32_t ir = info.x + (li ? q - sstart[li] : q + j0);
        key[k] = (KH)(((uint64_t)info.w << 32) | info.z);
        tag[k] = __uint_as_float(info.y);
        if (nin >= 0) {
          const float it = __ldcs(itg + ir);                 // streamed once: evict first, the slots should stay in L2
          tag[k] = times ? tag[k] * it : tag[k] + it;
          if (nin >= 1) key[k] += (KH)(uint32_t)__ldcs(ic0 + ir) * m0;
          for (int c = 1; c < nin; ++c) key[k] += (KH)(uint32_t)S.inner_col[c][ir] * (KH)S.inner_mult[c];
        }
      }
    }
    int32_t cur[kExpItems];
#pragma unroll
    for (int k = 0; k < kExpItems; ++k) {
      const uint32_t q = threadIdx.x + k * kExpBlock;
      cur[k] = SINK == kSinkMin ? (int32_t)0x80000000 : 0x7fffffff;        // nothing improves on this
      if (q < ntile) {
        if ((uint32_t)key[k] > mr.key_max) atomicOr(mr.err, kErrHeadRange);
        else cur[k] = XLOG_TABLE_LOAD_ROWWISE(mr.table + (uint32_t)key[k]);
      }
    }
#pragma unroll
    for (int k = 0; k < kExpItems; ++k) {
      const int32_t v = f2ord(tag[k]);
      if (SINK == kSinkMin ? v < cur[k] : v > cur[k]) mirror_commit<SINK>(mr, (uint32_t)key[k], v);
    }
    }
    return;
  }

  for (uint32_t q = threadIdx.x; q < (uint32_t)(t_hi - t_lo); q += kExpBlock) {
    const uint64_t p = t_lo + q;
    uint32_t row, j;
    uint4 info;
    if (staged) {
      const uint32_t li = srowidx[q];
      row = r_lo + li;
      j = li == 0 ? (uint32_t)(p - first_start) : q - sstart[li];
      info = sinfo[li];
    } else {
      // row = last row in [r_lo, r_hi] with start <= p   (rows of degree 0 share a start and are skipped)
      uint32_t lo = 0, hi = nrows;
      while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (start[r_lo + mid] <= p) lo = mid + 1; else hi = mid; }
      row = r_lo + lo - 1;
      j = (uint32_t)(p - start[row]);
      info = rowinfo[row];
    }
    const uint32_t ir = info.x + j;
    const float otag = __uint_as_float(info.y);
    float itag = S.times ? 1.f : 0.f;
    float tag = otag;
    if (S.has_inner) {
      itag = S.inner_tag[ir];
      tag = S.times ? otag * itag : otag + itag;
    }
    if (MODE == kExpFast) {
      KH key = (KH)(((uint64_t)info.w << 32) | info.z);
#pragma unroll
      for (int c = 0; c < kMaxArity - 1; ++c)
        if (c < S.inner_free) key += (KH)(uint32_t)S.inner_col[c][ir] * (KH)S.inner_mult[c];
      if (SINK == kSinkWrite) { ckeys[q + (t_lo - out_lo)] = key; ctags[q + (t_lo - out_lo)] = tag; }
      else mirror_apply<SINK>(mr, (uint32_t)key, tag);
      continue;
    }
    int64_t var[kMaxVars];
    bind_outer<KO>(S, okeys[row], var);
    if (S.has_inner) {
#pragma unroll
      for (int c = 0; c < kMaxArity - 1; ++c)
        if (c < S.inner_free) {
          const int64_t val = (int64_t)S.inner_col[c][ir] - S.inner_add[c];
#pragma unroll
          for (int v = 0; v < kMaxVars; ++v) if (v == S.inner_var[c]) var[v] = val;
        }
    }
    KH key = 0;
#pragma unroll
    for (int c = 0; c < kMaxArity; ++c)
      if (c < S.head.arity) {
        int64_t h = S.head_c0[c];
#pragma unroll
        for (int v = 0; v < kMaxVars; ++v) h += (int64_t)S.head_coef[c][v] * var[v];
        if (S.head_encode[c]) {
          const uint32_t r = dict_rank(S.head_dict.v[c], S.head_dict.n[c], h);
          if (r >= S.head_dict.n[c] || (int64_t)S.head_dict.v[c][r] != h) { e |= kErrInternal; h = 0; } else h = r;
        }
        if (h < 0 || h > (int64_t)S.head.mask[c]) { e |= kErrHeadRange; h = 0; }
        key |= (KH)(uint32_t)h << S.head.shift[c];
      }
    if (MODE != kExpBackward) {
      if (SINK == kSinkWrite) { ckeys[p - out_lo] = key; ctags[p - out_lo] = tag; }
      else if (!e) mirror_apply<SINK>(mr, (uint32_t)key, tag);
    } else {
      // head row of this binding: lower bound of the key among the stored head keys
      const KH* hk = reinterpret_cast<const KH*>(bw.head_keys);
      const KH want = key;
      uint32_t a = 0, b = bw.n_head;
      while (a < b) { const uint32_t mid = a + ((b - a) >> 1); if ((hk[mid] >> bw.count_bits) < want) a = mid + 1; else b = mid; }
      if (a < bw.n_head && (hk[a] >> bw.count_bits) == want) {
        const float g = bw.grad_head[a];
        if (bw.lse) {
          const float w = g * expf(tag - bw.head_tags[a]);
          atomicAdd(&bw.grad_outer[row], w);
          if (bw.grad_inner) atomicAdd(&bw.grad_inner[ir], w);
        } else {
          atomicAdd(&bw.grad_outer[row], g * itag);
          if (bw.grad_inner) atomicAdd(&bw.grad_inner[ir], g * otag);
        }
      } else e |= kErrInternal;
    }
  }
}

// Block b produces candidates [out_lo + b*tile, ...).  `start` is the exclusive scan of `deg`
// (global candidate index of each outer row's first match).  The outer rows covering the tile are
// staged in shared memory (their starts relative to the tile and their row records), so the per-
// candidate work is a short binary search in shared memory plus the coalesced inner reads.
template <typename KO, typename KH, int MODE, int SINK = kSinkWrite>
__global__ void __launch_bounds__(kExpBlock, SINK == kSinkWrite ? kExpWriteBlocksPerSM : kExpMirrorBlocksPerSM) k_join_expand(JoinSpec S, const KO* __restrict__ okeys, uint32_t n_outer,
                                                           const uint64_t* __restrict__ start, const uint4* __restrict__ rowinfo,
                                                           const uint2* __restrict__ tile_rows, uint64_t out_lo, uint64_t out_hi,
                                                           KH* __restrict__ ckeys,
                                                           float* __restrict__ ctags, uint32_t* __restrict__ err, BwdArgs bw, MirrorArgs mr) {
  typedef ExpShapeT<SINK != kSinkWrite> SH;
  __shared__ ExpSmem<SH> sm;
  const uint64_t t_lo = out_lo + (uint64_t)blockIdx.x * SH::tile;
  const uint64_t t_hi = min(t_lo + SH::tile, out_hi);
  if (t_lo >= t_hi) return;
  uint32_t e = 0;
  expand_tile<KO, KH, MODE, SINK>(sm, S, okeys, n_outer, start, rowinfo, tile_rows[blockIdx.x], t_lo, t_hi, out_lo, ckeys, ctags, bw, mr, e);
  if (e) atomicOr(err, e);
}

}  // namespace xlog
