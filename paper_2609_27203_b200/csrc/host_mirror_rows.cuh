// Row-local fixpoint of closure-shaped rules (row_fixpoint.cuh): when it applies, and the stratum driver around the one launch.
// Host-side driver code of the engine; included by xlog_api.cu only (one translation unit).
#pragma once
#include "host_mirror.cuh"
#include "row_fixpoint.cuh"

namespace xlog {
namespace {

// control words of the routes that keep one tag mirror per head of a component
constexpr int kMultiMaxHeads = 8;
constexpr int kSlotMultiChanged = 32, kSlotMultiNew = 40;     // per head: changed keys of the round, running count of new keys
static_assert(kSlotMultiNew + kMultiMaxHeads <= kSlotResState, "control words overlap");

// ---- row-local fixpoint (row_fixpoint.cuh) -------------------------------------------------------------------------
constexpr int kSlotRow = kSlotBm;          // the kRowTotals counters of k_row_fixpoint (a stratum takes this route or the bitmap-driven one)
static_assert(kSlotRow + kRowTotals <= kSlotDense, "control words overlap");
constexpr size_t kRowMaxSmem = 200u << 10;

// The rules over the component's heads when all of them read  h_i(a, c) :- h_j(a, b), r(b, c)  (r outside the component), the
// heads share one key layout and a value of a owns few enough keys for shared memory: fills `rules` (source head, target
// head, r's index) in the relations' own key order.
bool row_fixpoint_applies(Ctx* c, const std::vector<int>& comp, const std::vector<const RuleC*>& rs, std::vector<RowRule>& rules) {
  if (c->flags & (XLOG_FLAG_NO_ROW_FIXPOINT | XLOG_FLAG_NO_RESIDENT_LOOP | XLOG_FLAG_NO_GRAPH | XLOG_FLAG_NO_GROUPED_JOIN)) return false;
  if (comp.size() > (size_t)kRowMaxHeads) return false;
  const Relation& H0 = *c->rels[comp[0]];
  const int c_bits = H0.layout.shift[0];
  if (c_bits < 5 || c_bits > kRowMaxBits || row_fix_smem(c_bits, (int)comp.size()) > kRowMaxSmem) return false;
  for (int h : comp) {
    const Relation& H = *c->rels[h];
    if (H.arity != 2 || H.key_bytes != 4 || H.dict_n[1] || H.layout.shift[1] != 0) return false;   // a dictionary on column 0 is fine: its codes pass through the rules unchanged
    if (H.sr != XLOG_SR_MAXPLUS && H.sr != XLOG_SR_MINPLUS) return false;
    if (H.layout.shift[0] != c_bits || H.layout.total_bits != H0.layout.total_bits || H.dict_n[0] != H0.dict_n[0]) return false;
  }
  rules.clear();
  for (const RuleC* r : rs) {
    int pos = -1, in = 0;
    for (int j = 0; j < r->plan.n_atoms; ++j) if (in_set(comp, r->plan.atoms[j].rel)) { ++in; pos = j; }
    if (in == 0) continue;                                 // a seed rule: evaluated once, by the host
    if (in != 1 || r->kind != 2 || !r->shape[pos].ok || r->plan.emit_count_column) return false;
    const xlog_plan& p = r->plan;
    const xlog_atom& A = p.atoms[pos];
    const xlog_atom& B = p.atoms[1 - pos];
    if (A.negated || B.negated || !is_plain_var(A.args[0]) || !is_plain_var(A.args[1]) || A.args[0].var == A.args[1].var) return false;
    if (c->rels[B.rel]->arity != 2 || r->shape[pos].probe_col != 0 || r->shape[pos].probe_var != A.args[1].var || r->shape[pos].probe_mul != 1 ||
        r->shape[pos].probe_add != 0 || !is_plain_var(B.args[1]))
      return false;
    const int hv[2] = {A.args[0].var, B.args[1].var};
    for (int col = 0; col < 2; ++col) {
      if (p.head[col].c0 != 0) return false;
      for (int v = 0; v < XLOG_MAX_VARS; ++v) if (p.head[col].coef[v] != (v == hv[col] ? 1 : 0)) return false;
    }
    const Relation& HS = *c->rels[A.rel];
    Relation& HD = *c->rels[p.head_rel];
    const Variant v{r, pos, Source{nullptr, nullptr, 0, HS.layout, HS.key_bytes}};
    const JoinSpec S = make_spec(c, v, HD);                // builds the looked-up relation's index if it is missing
    if (!S.fast || !S.has_inner || S.inner_free != 1 || S.outer_decode[0] || S.outer_decode[1] || S.head_encode[0] || S.head_encode[1] ||
        S.inner_mult[0] != 1 || S.times)
      return false;
    RowRule R{};
    for (size_t i = 0; i < comp.size(); ++i) { if (comp[i] == A.rel) R.src = (int)i; if (comp[i] == p.head_rel) R.dst = (int)i; }
    R.off = S.inner_off; R.domain = (uint32_t)std::min<int64_t>(S.inner_domain, 0xffffffffll);
    R.z = S.inner_col[0]; R.w = S.inner_tag;
    rules.push_back(R);
  }
  if (rules.empty() || rules.size() > (size_t)kRowMaxRules) return false;
  uint64_t need = 1u << 20;
  for (int h : comp) need += ((uint64_t)4 << c->rels[h]->layout.total_bits) + ((uint64_t)1 << c->rels[h]->layout.total_bits) / 4 + (1u << 16);
  return need <= c->arena.largest_free() / 2;
}

// The stratum by the row-local route: the seed round from the host (every rule over the full relations, into the tables),
// then every row's rounds in one launch, then every table in key order is its relation.
void stratum_row_fixpoint(Ctx* c, const std::vector<int>& comp, const std::vector<const RuleC*>& rs, const std::vector<RowRule>& rules) {
  struct Head { Relation* H; bool is_max; int32_t empty; DevBuf table, bitmap, present; uint32_t n_start; MirrorArgs mr; };
  const Relation& H0 = *c->rels[comp[0]];
  const int bits = H0.layout.total_bits, c_bits = H0.layout.shift[0];
  const uint64_t dom = (uint64_t)1 << bits, slots = dom;
  const uint32_t nwords = (uint32_t)(dom / 32);
  std::vector<Head> heads(comp.size());
  zero_ctrl(c, kSlotMultiNew, kMultiMaxHeads);
  zero_ctrl(c, kSlotRow, kRowTotals);
  for (size_t i = 0; i < comp.size(); ++i) {
    Head& X = heads[i];
    X.H = c->rels[comp[i]];
    Relation& H = *X.H;
    X.is_max = H.sr == XLOG_SR_MAXPLUS;
    X.empty = X.is_max ? kMirrorEmptyMax : kMirrorEmptyMin;
    X.table = DevBuf(c, slots * 4); X.bitmap = DevBuf(c, (size_t)nwords * 4); X.present = DevBuf(c, (size_t)nwords * 4);
    XLOG_LAUNCH(c, k_fill_i32, grid_for(slots, 256 * 8), 256, 0, X.table.as<int32_t>(), slots, X.empty);
    XLOG_CUDA(cudaMemsetAsync(X.bitmap.p, 0, (size_t)nwords * 4, c->stream));
    XLOG_CUDA(cudaMemsetAsync(X.present.p, 0, (size_t)nwords * 4, c->stream));
    X.n_start = H.n;
    if (X.n_start)
      XLOG_LAUNCH(c, (k_mirror_scatter<uint32_t>), grid_for(X.n_start, 256, 1 << 30), 256, 0, (const uint32_t*)H.keys(), (const float*)H.tags(), X.n_start, H.layout,
                  H.layout, X.table.as<int32_t>(), X.present.as<uint32_t>());
    X.mr = MirrorArgs{X.table.as<int32_t>(), X.bitmap.as<uint32_t>(), (unsigned long long*)(c->d_ctrl + kSlotMultiNew + i), (uint32_t)(dom - 1), ctrl_u32(c, kSlotErr)};
  }
  c->unique_untracked = true;
  // seed round (Algorithm 1 lines 1-3)
  if (c->max_iter < 1) fail(XLOG_ERR_CONVERGENCE_FAILURE, "iteration cap reached before the fixpoint");
  ++c->r_iterations;
  uint64_t seed_total = 0;
  {
    std::vector<Variant> vs;
    for (const RuleC* r : rs) { const int outer = seed_outer(comp, r); vs.push_back(Variant{r, outer, full_source(*c->rels[r->plan.atoms[outer].rel])}); }
    for (size_t v0 = 0; v0 < vs.size(); v0 += 16) {
      std::vector<Counted> counted;
      std::vector<Head*> target;
      counted.reserve(16);
      for (size_t v = v0; v < std::min(vs.size(), v0 + 16); ++v) {
        if (vs[v].outer.n == 0) continue;
        Head* T = nullptr;
        for (size_t i = 0; i < comp.size(); ++i) if (comp[i] == vs[v].rule->plan.head_rel) T = &heads[i];
        counted.emplace_back();
        count_variant(c, vs[v], *T->H, counted.back(), kSlotTotals + (int)counted.size() - 1);
        target.push_back(T);
      }
      if (counted.empty()) continue;
      sync_ctrl(c);
      for (size_t i = 0; i < counted.size(); ++i) {
        Counted& q = counted[i];
        q.total = c->h_ctrl[q.slot];
        q.deg.reset(); q.sums.reset();
        seed_total += q.total;
        c->r_candidates += (int64_t)q.total;
        if (q.total) {
          c->note_bytes = (int64_t)q.total * (4 + (q.spec.has_inner ? 4 * (q.spec.inner_free + 1) : 0));
          launch_expand_mirror(c, q, target[i]->is_max, target[i]->mr);
        }
      }
    }
  }
  uint64_t total_new = 0;
  if (seed_total) {
    RowFix P{};
    P.n_heads = (int)heads.size(); P.n_rules = (int)rules.size();
    for (size_t i = 0; i < heads.size(); ++i) P.heads[i] = RowHead{heads[i].table.as<int32_t>(), heads[i].bitmap.as<uint32_t>(), heads[i].present.as<uint32_t>(), heads[i].is_max ? 1 : 0};
    for (size_t i = 0; i < rules.size(); ++i) P.rules[i] = rules[i];
    P.n_rows = (uint32_t)(slots >> c_bits); P.c_bits = c_bits; P.z_max = H0.layout.mask[1];
    P.max_rounds = (uint32_t)std::min<int64_t>(c->max_iter - 1, 0x7fffffff);
    P.totals = (unsigned long long*)(c->d_ctrl + kSlotRow); P.err = ctrl_u32(c, kSlotErr);
    const size_t smem = row_fix_smem(c_bits, P.n_heads);
    // per row and head: its slots read and written, its bitmap words; the candidates' reads of r are not known before the launch
    c->note_bytes = ((int64_t)slots * 8 + (int64_t)nwords * 12) * P.n_heads;
    const unsigned grid = std::min<unsigned>(P.n_rows, kSMs * 16);
#define XLOG_ROW_FIX(NH)                                                                                                          \
  do {                                                                                                                            \
    XLOG_CUDA(cudaFuncSetAttribute(k_row_fixpoint<NH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRowMaxSmem));             \
    XLOG_LAUNCH(c, (k_row_fixpoint<NH>), grid, kRowBlock, smem, P);                                                               \
  } while (0)
    switch (P.n_heads) {
      case 1: XLOG_ROW_FIX(1); break;
      case 2: XLOG_ROW_FIX(2); break;
      case 3: XLOG_ROW_FIX(3); break;
      default: XLOG_ROW_FIX(4); break;
    }
#undef XLOG_ROW_FIX
    sync_ctrl(c);
    const uint64_t cand = c->h_ctrl[kSlotRow + kRowCandidates], changed = c->h_ctrl[kSlotRow + kRowChanged], n_new = c->h_ctrl[kSlotRow + kRowNew];
    c->r_candidates += (int64_t)cand;
    c->r_new += (int64_t)n_new; c->r_improved += (int64_t)changed - (int64_t)n_new;
    c->r_iterations += (int64_t)c->h_ctrl[kSlotRow + kRowRounds];
    total_new = n_new;
    if (c->h_ctrl[kSlotRow + kRowCapped]) fail(XLOG_ERR_CONVERGENCE_FAILURE, "iteration cap reached before the fixpoint");
  }
  // every head in sorted form: the occupied slots in slot order (the tables are in key order); with several heads the sizes
  // come with the count (one control read per head), with one head it is what was there plus what was new
  for (Head& X : heads) {
    Relation& H = *X.H;
    const uint64_t nquads = slots / 4;
    const unsigned tiles = (unsigned)((slots + kMirSlotsPerTile - 1) / kMirSlotsPerTile);
    DevBuf sums(c, (size_t)tiles * 4);
    c->note_bytes = (int64_t)slots * 4;
    XLOG_LAUNCH(c, k_mirror_full_count, tiles, kMirBlock, 0, (const int4*)X.table.as<int4>(), nquads, X.empty, sums.as<uint32_t>());
    XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, sums.as<uint32_t>(), (int64_t)tiles, ctrl_u32(c, kSlotA));
    uint64_t n_out = (uint64_t)X.n_start + total_new;
    if (heads.size() > 1) { sync_ctrl(c); n_out = (uint32_t)c->h_ctrl[kSlotA]; }
    KeyTags full;
    full.n = (uint32_t)n_out;
    full.keys = DevBuf(c, (size_t)std::max<uint64_t>(n_out, 1) * 4);
    full.tags = DevBuf(c, (size_t)std::max<uint64_t>(n_out, 1) * 4);
    if (n_out) {
      c->note_bytes = (int64_t)slots * 4 + (int64_t)n_out * 8;
      XLOG_LAUNCH(c, (k_mirror_full_emit<uint32_t>), tiles, kMirBlock, 0, (const int4*)X.table.as<int4>(), nquads, X.empty, (const uint32_t*)sums.as<uint32_t>(), H.layout,
                  H.layout, full.keys.as<uint32_t>(), full.tags.as<float>());
    }
    set_current(H, std::move(full));
    X.table.reset(); X.bitmap.reset(); X.present.reset();
    if (c->flags & XLOG_FLAG_CHECK_INVARIANTS) {
      XLOG_LAUNCH(c, (k_check_sorted<uint32_t>), grid_for(H.n, 256), 256, 0, (const uint32_t*)H.keys(), (int64_t)H.n, ctrl_u32(c, kSlotErr));
      sync_ctrl(c);
    }
  }
}

}  // namespace
}  // namespace xlog
