// One round of rule evaluation on the sorting route: join specs, count -> scan -> materialise, sort, reduce-by-key.
// Host-side driver code of the engine; included by xlog_api.cu only (one translation unit).
#pragma once
#include "host_plan.cuh"

namespace xlog {
namespace {

// ---- one round of rule evaluation --------------------------------------------------
struct Source {                          // a packed (keys, tags) list standing for one atom's relation
  const void* keys; const float* tags; uint32_t n; KeyLayout layout; int key_bytes;
};
Source full_source(const Relation& R) { return Source{R.keys(), R.tags(), R.n, R.layout, R.key_bytes}; }

struct Variant {
  const RuleC* rule;
  int outer_atom;                        // the scanned atom (delta position for delta variants)
  Source outer;
};

struct Counted {                         // a variant after count + scan
  JoinSpec spec;
  Source outer;
  DevBuf deg, rowinfo, start, sums;
  int presorted_top = 0;                 // the candidates come out ordered by this many leading key bits
  uint64_t total = 0;
  int slot = 0;
};

JoinSpec make_spec(Ctx* c, const Variant& v, const Relation& H, const KeyLayout* head_layout = nullptr) {
  const xlog_plan& p = v.rule->plan;
  JoinSpec S;
  memset(&S, 0, sizeof S);                 // padding included: specs are compared byte for byte (graph reuse)
  S.outer = v.outer.layout;
  const xlog_atom& A = p.atoms[v.outer_atom];
  for (int i = 0; i < c->rels[A.rel]->arity; ++i) S.outer_args[i] = ArgSpec{A.args[i].kind, A.args[i].var, A.args[i].mul, A.args[i].add};
  S.has_inner = 0;
  S.neg_prefix = 0;
  if (v.rule->kind == 5) {
    const xlog_atom& B = p.atoms[1];
    Relation& RB = *c->rels[B.rel];
    if (RB.is_head && !c->stratum_done[B.rel]) fail(XLOG_ERR_UNSUPPORTED, "negation must be stratified: '" + RB.name + "' is not complete yet");
    Index& ix = ensure_index(c, RB, 0);
    S.neg_prefix = v.rule->neg_prefix;
    for (int k = 0; k < S.neg_prefix; ++k) S.neg_args[k] = ArgSpec{B.args[k].kind, B.args[k].var, B.args[k].mul, B.args[k].add};
    S.neg_domain = ix.domain;
    S.neg_off = ix.off.as<uint32_t>();
    S.neg_col1 = RB.arity > 1 ? ix.other[0] : nullptr;
  }
  if (v.rule->kind == 2) {
    const JoinShape& sh = v.rule->shape[v.outer_atom];
    if (!sh.ok) fail(XLOG_ERR_UNSUPPORTED, "this rule cannot be evaluated with the required atom as the scanned side");
    const xlog_atom& B = p.atoms[sh.inner];
    Relation& RB = *c->rels[B.rel];
    Index& ix = ensure_index(c, RB, sh.probe_col);
    S.has_inner = 1;
    S.probe_var = sh.probe_var; S.probe_mul = sh.probe_mul; S.probe_add = sh.probe_add;
    S.inner_domain = ix.domain;
    S.inner_off = ix.off.as<uint32_t>();
    S.inner_free = ix.n_other;
    for (int i = 0; i < ix.n_other; ++i) {
      S.inner_col[i] = ix.other[i];
      S.inner_var[i] = B.args[ix.other_src[i]].var;
      S.inner_add[i] = B.args[ix.other_src[i]].add;
    }
    S.inner_tag = ix.tags;
  }
  // dictionaries: the outer relation's codes are turned into values when a variable is bound, and head
  // values are ranked into codes, unless a variable only carries a column of the head relation
  // itself through unchanged (then the code is passed along untouched)
  const Relation& RA = *c->rels[A.rel];
  S.outer_dict = RA.dicts();
  S.head_dict = H.dicts();
  for (int i = 0; i < kMaxArity; ++i) { S.outer_decode[i] = i < RA.arity && RA.dict_n[i] ? 1 : 0; S.head_encode[i] = i < p.n_head_cols && H.dict_n[i] ? 1 : 0; }
  for (int i = 0; i < RA.arity; ++i) {
    if (!RA.dict_n[i] || !is_plain_var(A.args[i])) continue;
    const int v = A.args[i].var;
    int uses = 0;
    for (int j = 0; j < p.n_atoms; ++j)
      for (int k = 0; k < c->rels[p.atoms[j].rel]->arity; ++k)
        if (p.atoms[j].args[k].kind == XLOG_ARG_VAR && p.atoms[j].args[k].var == v) ++uses;
    bool pass = uses == 1 && A.rel == p.head_rel;
    for (int h = 0; h < p.n_head_cols && pass; ++h) {
      if (p.head[h].coef[v] == 0) continue;
      bool identity = h == i && p.head[h].c0 == 0 && p.head[h].coef[v] == 1;
      for (int k = 0; k < kMaxVars; ++k) if (k != v && p.head[h].coef[k] != 0) identity = false;
      pass = identity;
    }
    if (pass) { S.outer_decode[i] = 0; S.head_encode[i] = 0; }
  }
  S.head = head_layout ? *head_layout : H.layout;      // a tag mirror may order the head's columns its own way
  if (p.emit_count_column) {             // candidates are keyed by the declared head columns only
    int32_t mx[kMaxArity] = {0, 0, 0, 0};
    for (int i = 0; i < p.n_head_cols; ++i) mx[i] = H.col_max[i];
    S.head = make_layout(p.n_head_cols, mx);
  }
  for (int i = 0; i < p.n_head_cols; ++i) {
    S.head_c0[i] = p.head[i].c0;
    for (int k = 0; k < kMaxVars; ++k) S.head_coef[i][k] = p.head[i].coef[k];
  }
  S.times = H.sr == XLOG_SR_SUMPROD ? 1 : 0;
  // Fast shape: the head key is the row part plus non-negative multiples of the looked-up atom's other
  // columns.  Needs: those columns bind bare variables; their head coefficients are >= 0; any head column
  // they feed has a non-negative row part (c0 >= 0, outer coefficients >= 0, outer variables >= 0) and no dictionary.
  bool outer_bound[kMaxVars] = {false};
  for (int i = 0; i < c->rels[A.rel]->arity; ++i) if (A.args[i].kind == XLOG_ARG_VAR) outer_bound[A.args[i].var] = true;
  bool outer_nonneg = true;
  for (int i = 0; i < c->rels[A.rel]->arity; ++i) if (A.args[i].kind == XLOG_ARG_VAR && A.args[i].add > 0) outer_nonneg = false;
  bool fast = true;
  for (int h = 0; h < p.n_head_cols; ++h)
    for (int k = 0; k < kMaxVars; ++k) S.head_coef_outer[h][k] = outer_bound[k] ? p.head[h].coef[k] : 0;
  for (int j = 0; j < kMaxArity - 1; ++j) S.inner_mult[j] = 0;
  if (S.has_inner) {
    for (int j = 0; j < S.inner_free && fast; ++j) {
      if (S.inner_add[j] != 0) fast = false;
      uint64_t mult = 0;
      for (int h = 0; h < p.n_head_cols && fast; ++h) {
        const int cf = p.head[h].coef[S.inner_var[j]];
        if (cf == 0) continue;
        if (cf < 0 || S.head_encode[h] || H.dict_n[h] || p.head[h].c0 < 0 || !outer_nonneg) { fast = false; break; }
        for (int k = 0; k < kMaxVars; ++k) if (outer_bound[k] && p.head[h].coef[k] < 0) fast = false;
        mult += (uint64_t)cf << S.head.shift[h];
      }
      S.inner_mult[j] = mult;
    }
  }
  S.fast = fast ? 1 : 0;
  // simple shape: see JoinSpec
  bool simple = fast && S.neg_prefix == 0;
  int col_of_var[kMaxVars];
  for (int k = 0; k < kMaxVars; ++k) col_of_var[k] = -1;
  for (int i = 0; i < RA.arity && simple; ++i) {
    if (S.outer_decode[i]) simple = false;
    else if (A.args[i].kind == XLOG_ARG_VAR) {
      if (!is_plain_var(A.args[i]) || col_of_var[A.args[i].var] >= 0) simple = false; else col_of_var[A.args[i].var] = i;
    } else {
      const int64_t cv = A.args[i].add;
      if (cv < 0 || cv > (int64_t)S.outer.mask[i]) simple = false;          // can never match: leave it to the general path
      else { S.s_const_mask |= (uint64_t)S.outer.mask[i] << S.outer.shift[i]; S.s_const_val |= (uint64_t)cv << S.outer.shift[i]; }
    }
  }
  if (simple && S.has_inner) {
    const int pc = col_of_var[S.probe_var];
    if (pc < 0) simple = false; else { S.s_probe_shift = S.outer.shift[pc]; S.s_probe_mask = S.outer.mask[pc]; }
  }
  for (int hc = 0; hc < p.n_head_cols && simple; ++hc) {
    int src = -1;
    if (S.head_encode[hc] || p.head[hc].c0 < 0 || p.head[hc].c0 > 0x7fffffff) simple = false;
    for (int k = 0; k < kMaxVars && simple; ++k) {
      const int cf = S.head_coef_outer[hc][k];
      if (cf == 0) continue;
      if (cf != 1 || src >= 0 || col_of_var[k] < 0) simple = false; else src = col_of_var[k];
    }
    S.s_c0[hc] = (uint32_t)p.head[hc].c0;
    S.s_src_shift[hc] = src >= 0 ? S.outer.shift[src] : 0;
    S.s_src_mask[hc] = src >= 0 ? S.outer.mask[src] : 0u;
  }
  if (p.emit_count_column) simple = false;
  S.simple = simple ? 1 : 0;
  return S;
}

// count -> scan for one variant; the grand total lands in control slot `slot` (read after sync_ctrl)
void count_variant(Ctx* c, const Variant& v, const Relation& H, Counted& q, int slot, const KeyLayout* head_layout = nullptr) {
  q.spec = make_spec(c, v, H, head_layout);
  q.outer = v.outer;
  q.slot = slot;
  {
    // Leading head columns that follow the leading columns of the scanned atom, in the same order, through strictly
    // increasing maps (column = mul * v + add with mul >= 1 in the atom, c0 + coef * v with coef >= 1 in the head, v in no
    // earlier column): the scanned relation is sorted by those columns (dictionary codes keep the order of the values),
    // equal column values give equal head values and the other way round, so the candidate stream is already ordered by
    // those key bits.  sum(p, a + b) :- digit(2p, a), digit(2p + 1, b) has its first head column of this kind.
    const xlog_plan& p = v.rule->plan;
    const xlog_atom& A = p.atoms[v.outer_atom];
    const int ka = c->rels[A.rel]->arity;
    int k = 0;
    for (; k < p.n_head_cols && k < ka; ++k) {
      if (A.args[k].kind != XLOG_ARG_VAR || A.args[k].mul < 1) break;
      const int var = A.args[k].var;
      bool fresh = true;
      for (int j = 0; j < k; ++j) fresh = fresh && A.args[j].var != var;
      bool mono = fresh && p.head[k].coef[var] >= 1;
      for (int w = 0; w < kMaxVars; ++w) mono = mono && (w == var || p.head[k].coef[w] == 0);
      if (!mono) break;
    }
    q.presorted_top = k ? q.spec.head.total_bits - q.spec.head.shift[k - 1] : 0;
  }
  const uint32_t n = v.outer.n;
  const unsigned tiles = (n + kScanTile - 1) / kScanTile;
  q.deg = DevBuf(c, (size_t)n * 4); q.rowinfo = DevBuf(c, (size_t)n * 16);
  q.start = DevBuf(c, (size_t)n * 8); q.sums = DevBuf(c, (size_t)tiles * 8);
  DISPATCH_K(v.outer.key_bytes, XLOG_LAUNCH(c, (k_join_count<K>), (n + 255) / 256, 256, 0, q.spec, (const K*)v.outer.keys, v.outer.tags, n,
                                             q.deg.as<uint32_t>(), q.rowinfo.as<uint4>(), ctrl_u32(c, kSlotErr)));
  if (n <= (1u << 13)) {
    XLOG_LAUNCH(c, (k_scan_block<uint32_t, uint64_t>), 1, 1024, 0, (const uint32_t*)q.deg.as<uint32_t>(), (int64_t)n, q.start.as<uint64_t>(),
                (uint64_t*)(c->d_ctrl + q.slot));
    return;
  }
  XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint64_t>), tiles, kScanBlock, 0, (const uint32_t*)q.deg.as<uint32_t>(), (int64_t)n, q.sums.as<uint64_t>());
  XLOG_LAUNCH(c, (k_scan_spine<uint64_t>), 1, 1024, 0, q.sums.as<uint64_t>(), (int64_t)tiles, (uint64_t*)(c->d_ctrl + q.slot));
  XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint64_t>), tiles, kScanBlock, 0, (const uint32_t*)q.deg.as<uint32_t>(), (int64_t)n,
              (const uint64_t*)q.sums.as<uint64_t>(), q.start.as<uint64_t>());
}

// materialise candidates [lo, hi) of a counted variant into (ckeys, ctags), or (MODE == kExpBackward) run the backward
// scatter, or (SINK != kSinkWrite) apply them to the head relation's tag mirror
template <int MODE, int SINK>
void launch_expand_mode(Ctx* c, Counted& q, uint64_t lo, uint64_t hi, int ckb, void* ckeys, float* ctags, const BwdArgs& bw, const MirrorArgs& mr) {
  constexpr uint32_t tile = SINK == kSinkWrite ? kExpTileWrite : kExpTileMirror;
  const unsigned blocks = (unsigned)((hi - lo + tile - 1) / tile);
  if (blocks == 0) return;                               // no candidates in the range
  const uint64_t* st = q.start.as<uint64_t>();
  const uint4* ri = q.rowinfo.as<uint4>();
  uint32_t* err = ctrl_u32(c, kSlotErr);
  // all work is issued on one stream, so a scratch block may be released as soon as its last kernel is queued:
  // whatever reuses the memory runs later in stream order
  DevBuf tile_rows(c, (size_t)blocks * 8);
  const int64_t bytes = c->note_bytes;
  c->note_bytes = 0;
  XLOG_LAUNCH(c, k_expand_partition, (blocks + 255) / 256, 256, 0, st, q.outer.n, lo, hi, blocks, tile, tile_rows.as<uint2>());
  const uint2* tr = tile_rows.as<uint2>();
  c->note_bytes = bytes;
  if (q.outer.key_bytes == 4 && ckb == 4)
    XLOG_LAUNCH(c, (k_join_expand<uint32_t, uint32_t, MODE, SINK>), blocks, kExpBlock, 0, q.spec, (const uint32_t*)q.outer.keys, q.outer.n, st, ri, tr, lo, hi, (uint32_t*)ckeys, ctags, err, bw, mr);
  else if (ckb == 4)
    XLOG_LAUNCH(c, (k_join_expand<uint64_t, uint32_t, MODE, SINK>), blocks, kExpBlock, 0, q.spec, (const uint64_t*)q.outer.keys, q.outer.n, st, ri, tr, lo, hi, (uint32_t*)ckeys, ctags, err, bw, mr);
  else if (SINK != kSinkWrite)
    fail(XLOG_ERR_INTERNAL, "tag mirror with wide keys");
  else if (q.outer.key_bytes == 4)
    XLOG_LAUNCH(c, (k_join_expand<uint32_t, uint64_t, MODE, kSinkWrite>), blocks, kExpBlock, 0, q.spec, (const uint32_t*)q.outer.keys, q.outer.n, st, ri, tr, lo, hi, (uint64_t*)ckeys, ctags, err, bw, mr);
  else
    XLOG_LAUNCH(c, (k_join_expand<uint64_t, uint64_t, MODE, kSinkWrite>), blocks, kExpBlock, 0, q.spec, (const uint64_t*)q.outer.keys, q.outer.n, st, ri, tr, lo, hi, (uint64_t*)ckeys, ctags, err, bw, mr);
}
template <bool BWD>
void launch_expand(Ctx* c, Counted& q, uint64_t lo, uint64_t hi, int ckb, void* ckeys, float* ctags, const BwdArgs& bw) {
  const MirrorArgs none{};
  if (BWD) launch_expand_mode<kExpBackward, kSinkWrite>(c, q, lo, hi, ckb, ckeys, ctags, bw, none);
  else if (q.spec.fast) launch_expand_mode<kExpFast, kSinkWrite>(c, q, lo, hi, ckb, ckeys, ctags, bw, none);
  else launch_expand_mode<kExpGeneric, kSinkWrite>(c, q, lo, hi, ckb, ckeys, ctags, bw, none);
}
// every candidate of a counted variant goes straight into the tag mirror
void launch_expand_mirror(Ctx* c, Counted& q, bool is_max, const MirrorArgs& mr) {
  const BwdArgs bw{};
  if (q.spec.fast) {
    if (is_max) launch_expand_mode<kExpFast, kSinkMax>(c, q, 0, q.total, 4, nullptr, nullptr, bw, mr);
    else launch_expand_mode<kExpFast, kSinkMin>(c, q, 0, q.total, 4, nullptr, nullptr, bw, mr);
  } else {
    if (is_max) launch_expand_mode<kExpGeneric, kSinkMax>(c, q, 0, q.total, 4, nullptr, nullptr, bw, mr);
    else launch_expand_mode<kExpGeneric, kSinkMin>(c, q, 0, q.total, 4, nullptr, nullptr, bw, mr);
  }
}

constexpr int kSlotTotals = 16;          // uint64 candidate totals of the variants of a round

// Evaluate the variants, all deriving head relation H: join, project, sort, reduce by key.
// `extra` (optional) is appended to the candidates before the sort (loaded facts of H in a
// non-recursive stratum).  Returns the sorted unique candidates.
// defer_slot >= 0: a small single-batch result may come back with its exact row count still on the device
// (KeyTags::n_slot), saving a control read; the caller settles it after its next sync_ctrl.
KeyTags evaluate(Ctx* c, Relation& H, std::vector<Variant>& variants, const Source* extra, const KeyLayout& cand_layout,
                 bool want_head_pos, int defer_slot = -1) {
  const int ckb = cand_layout.total_bits <= 32 ? 4 : 8;
  std::vector<Counted> counted;
  counted.reserve(variants.size());
  if (variants.size() > 16) fail(XLOG_ERR_UNSUPPORTED, "too many rule variants for one head");
  // count + scan for every variant, then one control read for all totals
  for (Variant& v : variants) {
    if (v.outer.n == 0) continue;
    counted.emplace_back();
    Counted& q = counted.back();
    count_variant(c, v, H, q, kSlotTotals + (int)counted.size() - 1);
  }
  uint64_t total = extra ? extra->n : 0;
  if (!counted.empty()) {
    sync_ctrl(c);
    for (Counted& q : counted) { q.total = c->h_ctrl[q.slot]; total += q.total; q.deg.reset(); q.sums.reset(); }
    // a variant without candidates takes no part in the batches below (left in, it would open one more, empty batch
    // after the last full one)
    counted.erase(std::remove_if(counted.begin(), counted.end(), [](const Counted& q) { return q.total == 0; }), counted.end());
  }
  c->r_candidates += (int64_t)total;
  KeyTags result;
  if (total == 0) return result;

  // batch capacity: bounded by the configured chunk size and by what the arena can hold
  const size_t per = (size_t)(ckb + 4) * 2;                                  // two buffers per candidate (sort ping-pong)
  uint64_t cap = total;
  if (c->chunk_bytes) cap = std::min<uint64_t>(cap, std::max<uint64_t>(1, c->chunk_bytes / per));
  cap = std::min<uint64_t>(cap, (uint64_t)kSortMaxN);
  {
    // besides the two candidate buffers a batch needs sort status words (1/4 B per row), the reduce's
    // spill tables (up to 2 B per row) and a few MB of per-group arrays
    const size_t free_bytes = c->arena.largest_free();
    const uint64_t fit = free_bytes > (6u << 20) ? (free_bytes - (6u << 20)) / (per + 3) : 1;
    if (fit < cap) cap = std::max<uint64_t>(fit, 1);
  }
  if (want_head_pos && cap < total) fail(XLOG_ERR_RESOURCE_EXHAUSTED, "a counted aggregate must fit one candidate batch");
  // one variant and nothing appended: every batch is a contiguous slice of one ordered stream
  const int presorted_top = counted.size() == 1 && (extra == nullptr || extra->n == 0) ? counted[0].presorted_top : 0;

  size_t vi = 0; uint64_t vpos = 0; bool extra_done = extra == nullptr || extra->n == 0;
  while (vi < counted.size() || !extra_done) {
    DevBuf k0(c, cap * ckb), t0(c, cap * 4), k1(c, cap * ckb), t1(c, cap * 4);
    uint64_t fill = 0;
    while (fill < cap && vi < counted.size()) {
      Counted& q = counted[vi];
      const uint64_t take = std::min<uint64_t>(cap - fill, q.total - vpos);
      if (take) {
        // per candidate: key + tag written, one inner column + inner tag read (outer rows amortise over the degree)
        c->note_bytes = (int64_t)take * (ckb + 4 + (q.spec.has_inner ? 4 * (q.spec.inner_free + 1) : 0));
        launch_expand<false>(c, q, vpos, vpos + take, ckb, (char*)k0.p + fill * ckb, t0.as<float>() + fill, BwdArgs{});
        fill += take; vpos += take;
      }
      if (vpos == q.total) { q.start.reset(); q.rowinfo.reset(); ++vi; vpos = 0; }
    }
    if (!extra_done && vi == counted.size() && cap - fill >= extra->n) {
      XLOG_CUDA(cudaMemcpyAsync((char*)k0.p + fill * ckb, extra->keys, (size_t)extra->n * ckb, cudaMemcpyDeviceToDevice, c->stream));
      XLOG_CUDA(cudaMemcpyAsync(t0.as<float>() + fill, extra->tags, (size_t)extra->n * 4, cudaMemcpyDeviceToDevice, c->stream));
      fill += extra->n;
      extra_done = true;
    } else if (!extra_done && vi == counted.size() && fill == 0) {
      fail(XLOG_ERR_RESOURCE_EXHAUSTED, "candidate batch too small for the relation's loaded facts");
    }
    KeyTags part;
    DISPATCH_K(ckb, part = sort_reduce<K>(c, H.sr, k0, t0, k1, t1, fill, cand_layout.total_bits, want_head_pos, cap >= total ? defer_slot : -1,
                                          presorted_top));
    if (result.n == 0) result = std::move(part);
    else {
      // a later batch: union with oplus into the running result
      if (result.n_slot >= 0) fail(XLOG_ERR_INTERNAL, "evaluate: a deferred row count met a second candidate batch");
      MergeResult m;
      DISPATCH_K(ckb, m = merge<K>(c, H.sr, part.keys.as<K>(), part.tags.as<float>(), part.n, -1, result.keys.as<K>(), result.tags.as<float>(),
                                    result.n, false, false));
      result = std::move(m.full);
    }
  }
  if (result.n_slot < 0) c->r_unique += result.n;     // a deferred count is added by the caller once it is known
  return result;
}

// Which atom a rule scans in the seed round (every atom reads its full relation): the recursive side if exactly one atom
// is recursive, else whichever side has an index path.
int seed_outer(const std::vector<int>& comp, const RuleC* r) {
  int outer = 0;
  if (r->kind == 2) {
    const bool in0 = in_set(comp, r->plan.atoms[0].rel), in1 = in_set(comp, r->plan.atoms[1].rel);
    // scan the recursive side and look up the stable side; with two recursive atoms (non-linear rule)
    // the looked-up side is the full relation, indexed afresh in every round it changed
    outer = in1 && !in0 ? 1 : 0;
    if (!r->shape[outer].ok) { if (in0 == in1 && r->shape[1 - outer].ok) outer = 1 - outer; else fail(XLOG_ERR_UNSUPPORTED, "no index path for this rule"); }
  }
  return outer;
}

}  // namespace
}  // namespace xlog
