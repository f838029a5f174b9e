// Strata: non-recursive evaluation, Algorithm 1 for max/min components (sorting route), the delta form for sum / logsumexp components, the fixpoint driver.
// Host-side driver code of the engine; included by xlog_api.cu only (one translation unit).
#pragma once
#include "host_backward.cuh"
#include "host_cyclic.cuh"
#include "host_mirror_strata.cuh"

namespace xlog {
namespace {

// Non-recursive stratum:  I(P) = facts(P) oplus (oplus over rules of T_r), each rule evaluated once.
void stratum_once(Ctx* c, int head, const std::vector<const RuleC*>& rs) {
  Relation& H = *c->rels[head];
  const bool counted = rs[0]->plan.emit_count_column != 0;
  for (const RuleC* r : rs) if ((r->plan.emit_count_column != 0) != counted) fail(XLOG_ERR_UNSUPPORTED, "rules of one head disagree on emit_count_column");
  if (counted && H.n_facts) fail(XLOG_ERR_UNSUPPORTED, "a counted head relation cannot also hold loaded facts");
  if (counted && rs.size() > 1) fail(XLOG_ERR_UNSUPPORTED, "a counted head relation takes exactly one rule");
  ++c->r_iterations;
  if (rs.size() == 1 && rs[0]->kind == 3) { triangle_aggregate(c, H, *rs[0]); return; }
  if (rs.size() == 1 && rs[0]->kind == 4) { triangle_materialise(c, H, *rs[0]); c->r_new += H.n; return; }
  if (rs.size() == 1 && rs[0]->kind == 6) { cycle4_materialise(c, H, *rs[0]); c->r_new += H.n; return; }
  std::vector<Variant> vs;
  for (const RuleC* r : rs) {
    if (r->kind == 3 || r->kind == 4 || r->kind == 6) fail(XLOG_ERR_UNSUPPORTED, "a triangle or four-cycle rule must be the only rule of its head");
    int outer = 0;
    if (r->kind == 2 && !r->shape[0].ok) outer = 1;
    vs.push_back(Variant{r, outer, full_source(*c->rels[r->plan.atoms[outer].rel])});
  }
  KeyLayout cl = H.layout;
  if (counted) { int32_t mx[kMaxArity] = {0, 0, 0, 0}; for (int i = 0; i < rs[0]->plan.n_head_cols; ++i) mx[i] = H.col_max[i]; cl = make_layout(rs[0]->plan.n_head_cols, mx); }
  Source facts{H.fact_keys.p, H.fact_tags.as<float>(), H.n_facts, H.layout, H.key_bytes};
  KeyTags u = evaluate(c, H, vs, H.n_facts ? &facts : nullptr, cl, counted);
  if (counted) append_count_column(c, H, u, cl);
  else set_current(H, std::move(u));
  c->r_new += (int64_t)H.n - H.n_facts;
}

// Recursive component under a non-idempotent oplus (logsumexp / sum): the tag of a tuple is the oplus over all of its
// derivations, which is finite when the tuples' dependencies form a DAG (path counting, path-probability sums on an
// acyclic graph).  Algorithm 1 with the delta carrying tag DIFFERENCES: the rules are linear in the component's relations
// (one recursive atom each), so  I_{k+1} - I_k = T_rec(I_k - I_{k-1}):
//   Delta_1 = T(facts) with every atom reading the full relation;  Delta_{k+1} = T_rec(Delta_k);  I_{k+1} = I_k oplus Delta_{k+1}
// (sort -> reduce-by-key gives Delta, the merge kernel's union-with-oplus gives I), until a round derives nothing.  A cyclic
// dependency never gets there and ends at the iteration cap.  The component is recomputed from its loaded facts on
// every call: adding to an earlier result would count every derivation twice.
void stratum_recursive_additive(Ctx* c, const std::vector<int>& comp, const std::vector<const RuleC*>& rs) {
  for (const RuleC* r : rs) {
    int in = 0;
    for (int j = 0; j < r->plan.n_atoms; ++j) if (in_set(comp, r->plan.atoms[j].rel)) ++in;
    if (in > 1) fail(XLOG_ERR_UNSUPPORTED, "a rule with two recursive atoms under a non-idempotent oplus (logsumexp / sum)");
  }
  for (int p : comp) drop_current(*c->rels[p]);
  std::vector<KeyTags> delta(c->rels.size());
  for (int64_t round = 0;; ++round) {
    if (round >= c->max_iter) fail(XLOG_ERR_CONVERGENCE_FAILURE, "iteration cap reached before the fixpoint (cyclic derivations under a non-idempotent oplus never end)");
    ++c->r_iterations;
    std::vector<std::pair<int, KeyTags>> produced;
    for (int h : comp) {
      Relation& H = *c->rels[h];
      std::vector<Variant> vs;
      for (const RuleC* r : rs) {
        if (r->plan.head_rel != h) continue;
        if (round == 0) {
          const int outer = seed_outer(comp, r);
          vs.push_back(Variant{r, outer, full_source(*c->rels[r->plan.atoms[outer].rel])});
        } else {
          for (int j = 0; j < r->plan.n_atoms; ++j) {
            const int ar = r->plan.atoms[j].rel;
            if (!in_set(comp, ar) || r->plan.atoms[j].negated || delta[ar].n == 0) continue;
            const Relation& RA = *c->rels[ar];
            vs.push_back(Variant{r, j, Source{delta[ar].keys.p, delta[ar].tags.as<float>(), delta[ar].n, RA.layout, RA.key_bytes}});
          }
        }
      }
      if (!vs.empty()) produced.emplace_back(h, evaluate(c, H, vs, nullptr, H.layout, false));
    }
    for (int p : comp) delta[p] = KeyTags();
    uint64_t derived = 0;
    for (auto& pr : produced) {
      Relation& H = *c->rels[pr.first];
      KeyTags& u = pr.second;
      if (u.n == 0) continue;
      derived += u.n;
      MergeResult m;
      DISPATCH_K(H.key_bytes, m = merge<K>(c, H.sr, u.keys.as<K>(), u.tags.as<float>(), u.n, -1, (const K*)H.keys(), H.tags(), H.n, false, false));
      c->r_new += m.n_new; c->r_improved += (int64_t)u.n - m.n_new;
      set_current(H, std::move(m.full));
      delta[pr.first] = std::move(u);
      if (c->flags & XLOG_FLAG_CHECK_INVARIANTS) {
        DISPATCH_K(H.key_bytes, XLOG_LAUNCH(c, (k_check_sorted<K>), grid_for(H.n, 256), 256, 0, (const K*)H.keys(), (int64_t)H.n, ctrl_u32(c, kSlotErr)));
        sync_ctrl(c);
      }
    }
    if (derived == 0) break;
  }
}

// Recursive component: Algorithm 1 with tag improvement.
void stratum_recursive(Ctx* c, const std::vector<int>& comp, const std::vector<const RuleC*>& rs) {
  int idem = 0, additive = 0;
  for (int p : comp) { if (c->rels[p]->sr == XLOG_SR_MAXPLUS || c->rels[p]->sr == XLOG_SR_MINPLUS) ++idem; else ++additive; }
  if (idem && additive) fail(XLOG_ERR_UNSUPPORTED, "a recursive component mixes max/min relations with logsumexp/sum relations");
  for (const RuleC* r : rs) {
    if (r->plan.emit_count_column) fail(XLOG_ERR_UNSUPPORTED, "count inside a recursive component");
    if (r->kind == 3 || r->kind == 4 || r->kind == 6) fail(XLOG_ERR_UNSUPPORTED, "triangle or four-cycle rule inside a recursive component");
  }
  if (additive) { stratum_recursive_additive(c, comp, rs); return; }
  if (mirror_applies(c, comp, rs)) { stratum_recursive_mirror(c, comp[0], rs); return; }
  if (mirror_multi_applies(c, comp, rs)) { stratum_recursive_mirror_multi(c, comp, rs); return; }
  std::vector<KeyTags> delta(c->rels.size());
  for (int64_t round = 0;; ++round) {
    if (round >= c->max_iter) fail(XLOG_ERR_CONVERGENCE_FAILURE, "iteration cap reached before the fixpoint");
    ++c->r_iterations;
    // evaluate every head against the same state, then absorb
    std::vector<std::pair<int, KeyTags>> produced;
    for (int h : comp) {
      Relation& H = *c->rels[h];
      std::vector<Variant> vs;
      for (const RuleC* r : rs) {
        if (r->plan.head_rel != h) continue;
        if (round == 0) {                                   // seed: every atom reads the full relation
          const int outer = seed_outer(comp, r);
          vs.push_back(Variant{r, outer, full_source(*c->rels[r->plan.atoms[outer].rel])});
        } else {
          for (int j = 0; j < r->plan.n_atoms; ++j) {
            const int ar = r->plan.atoms[j].rel;
            if (!in_set(comp, ar) || r->plan.atoms[j].negated) continue;
            const KeyTags& d = delta[ar];
            if (d.n == 0) continue;
            const Relation& RA = *c->rels[ar];
            vs.push_back(Variant{r, j, Source{d.keys.p, d.tags.as<float>(), d.n, RA.layout, RA.key_bytes}});
          }
        }
      }
      if (vs.empty()) continue;
      const int slot = produced.size() < 8 ? 32 + 4 * (int)produced.size() : -1;
      produced.emplace_back(h, evaluate(c, H, vs, nullptr, H.layout, false, slot));
    }
    for (int p : comp) delta[p] = KeyTags();
    // merge every head's candidates into its full relation; small merges leave their totals on the device and all of
    // them are settled by one control read
    std::vector<MergeResult> merged(produced.size());
    bool need_read = false;
    for (size_t i = 0; i < produced.size(); ++i) {
      Relation& H = *c->rels[produced[i].first];
      KeyTags& u = produced[i].second;
      if (u.n == 0) continue;
      if (!H.cur_owned && H.n_facts) {
        // first derivation into a relation that holds facts: work on a private copy
        KeyTags copy; copy.n = H.n_facts;
        copy.keys = DevBuf(c, (size_t)H.n_facts * H.key_bytes); copy.tags = DevBuf(c, (size_t)H.n_facts * 4);
        XLOG_CUDA(cudaMemcpyAsync(copy.keys.p, H.fact_keys.p, (size_t)H.n_facts * H.key_bytes, cudaMemcpyDeviceToDevice, c->stream));
        XLOG_CUDA(cudaMemcpyAsync(copy.tags.p, H.fact_tags.p, (size_t)H.n_facts * 4, cudaMemcpyDeviceToDevice, c->stream));
        set_current(H, std::move(copy));
      }
      const int slot = i < 8 ? 32 + 4 * (int)i + 1 : -1;
      DISPATCH_K(H.key_bytes, merged[i] = merge<K>(c, H.sr, u.keys.as<K>(), u.tags.as<float>(), u.n, u.n_slot, (const K*)H.keys(), H.tags(), H.n,
                                                    true, H.cur_owned, slot));
      if (merged[i].slot >= 0) need_read = true;
    }
    if (need_read) sync_ctrl(c);
    uint64_t changed = 0;
    for (size_t i = 0; i < produced.size(); ++i) {
      Relation& H = *c->rels[produced[i].first];
      KeyTags& u = produced[i].second;
      if (u.n == 0) continue;
      if (u.n_slot >= 0) c->r_unique += (int64_t)(uint32_t)c->h_ctrl[u.n_slot];
      MergeResult& m = merged[i];
      finish_merge(c, m);
      if (!m.in_place) set_current(H, std::move(m.full));
      else if (m.n_improved) drop_indices(H);           // tags changed in place: permuted index copies are stale
      c->r_new += m.n_new; c->r_improved += m.n_improved;
      changed += (uint64_t)m.n_new + m.n_improved;
      delta[produced[i].first] = std::move(m.delta);
      if (c->flags & XLOG_FLAG_CHECK_INVARIANTS) {
        DISPATCH_K(H.key_bytes, XLOG_LAUNCH(c, (k_check_sorted<K>), grid_for(H.n, 256), 256, 0, (const K*)H.keys(), (int64_t)H.n, ctrl_u32(c, kSlotErr)));
        sync_ctrl(c);
      }
    }
    if (changed == 0) break;
  }
}

void run_fixpoint(Ctx* c) {
  if (c->idb_dirty) { reset_idb(c); c->idb_dirty = false; }
  c->stratum_done.assign(c->rels.size(), 0);
  if (c->poisoned) fail(XLOG_ERR_INVALID_STATE, "derived relations are poisoned by an earlier failure; call xlog_ctx_reset_idb");
  c->poisoned = true;                      // cleared on success
  zero_ctrl(c, kSlotErr);
  propagate_bounds(c);
  for (const std::vector<int>& comp : components(c)) {
    std::vector<const RuleC*> rs;
    for (const RuleC& r : c->rules) if (in_set(comp, r.plan.head_rel)) rs.push_back(&r);
    if (rs.empty()) continue;
    ++c->r_strata;
    bool recursive = comp.size() > 1;
    for (const RuleC* r : rs) for (int j = 0; j < r->plan.n_atoms; ++j) if (in_set(comp, r->plan.atoms[j].rel)) recursive = true;
    for (const RuleC* r : rs)
      if (r->kind == 5 && in_set(comp, r->plan.atoms[1].rel)) fail(XLOG_ERR_UNSUPPORTED, "negation must be stratified: the negated relation depends on the rule's head");
    if (!recursive) stratum_once(c, comp[0], rs); else stratum_recursive(c, comp, rs);
    for (int p : comp) c->stratum_done[p] = 1;
  }
  for (Relation* R : c->rels) if (R->is_head) ensure_soa(c, *R);
  sync_ctrl(c);
  c->poisoned = false;
  c->evaluated = true;
}

}  // namespace
}  // namespace xlog
