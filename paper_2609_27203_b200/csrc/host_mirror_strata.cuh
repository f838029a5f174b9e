// Strata over tag mirrors: one head (row-local, resident, bitmap-driven, grouped, dense path doubling or plain host-driven
// rounds) and several mutually recursive heads (one mirror per head).
// Host-side driver code of the engine; included by xlog_api.cu only (one translation unit).
#pragma once
#include "host_mirror.cuh"
#include "host_mirror_rows.cuh"

namespace xlog {
namespace {

// Algorithm 1 over a tag mirror (mirror.cuh): per round  count -> scan -> join straight into the table -> compact the
// changed bitmap into the next delta.  No candidate is ever written to memory.  The seed round is driven by the host
// (its rules scan whole relations of known size); the delta rounds run resident where the fixed-capacity buffers fit.
void stratum_recursive_mirror(Ctx* c, int h, const std::vector<const RuleC*>& rs) {
  {
    std::vector<RowRule> row_rules;
    const std::vector<int> one{h};
    if (row_fixpoint_applies(c, one, rs, row_rules)) { c->resident.erase(h); stratum_row_fixpoint(c, one, rs, row_rules); return; }
  }
  Relation& H = *c->rels[h];
  const std::vector<int> comp{h};
  const int bits = H.layout.total_bits;
  const uint64_t dom = (uint64_t)1 << bits;
  const bool is_max = H.sr == XLOG_SR_MAXPLUS;
  const int32_t empty = is_max ? kMirrorEmptyMax : kMirrorEmptyMin;
  const uint64_t slots = std::max<uint64_t>(dom, 4);
  const uint32_t bm_quads = (uint32_t)((std::max<uint64_t>(dom / 32, 1) + 3) / 4);
  const unsigned ch_tiles = mirror_tiles(bm_quads * 4);
  const RuleC* doubling = doubling_rule_of(c, h, rs);
  Resident* R = doubling ? nullptr : resident_for(c, h, bits, slots, bm_quads, ch_tiles);
  if (doubling) c->resident.erase(h);
  // the mirror's own column order: for the grouped join the probed column is the major part of the index (group_join.cuh)
  KeyLayout M = H.layout;
  const bool grouped = !R && !(c->flags & XLOG_FLAG_NO_GROUPED_JOIN) && grouped_shape(c, h, rs);
  int carried_bits = 0;
  if (grouped) {
    carried_bits = bits - H.layout.shift[0];             // width of column 0
    M.shift[0] = 0;
    M.shift[1] = carried_bits;
  }
  const KeyLayout* ML = grouped ? &M : nullptr;
  DevBuf table_own, bitmap_own, present_own, ch_sums_own;
  if (!R) {
    table_own = DevBuf(c, slots * 4); bitmap_own = DevBuf(c, (size_t)bm_quads * 16); present_own = DevBuf(c, (size_t)bm_quads * 16);
    ch_sums_own = DevBuf(c, (size_t)ch_tiles * 4);
  }
  BitmapJoin bj;
  if (grouped) bitmap_join_setup(c, h, rs, M, carried_bits, slots, bj);
  DevBuf snap_own, rowstart_own;
  const int dense_bits1 = H.layout.shift[0];
  const uint32_t dense_rows = (uint32_t)(slots >> dense_bits1);
  if (doubling) { snap_own = DevBuf(c, slots * 4); rowstart_own = DevBuf(c, ((size_t)dense_rows + 2) * 4); }
  uint32_t* present = R ? R->present.as<uint32_t>() : present_own.as<uint32_t>();
  int32_t* table = R ? R->table.as<int32_t>() : table_own.as<int32_t>();
  uint4* bitmap = R ? R->bitmap.as<uint4>() : bitmap_own.as<uint4>();
  uint32_t* ch_sums = R ? R->ch_sums.as<uint32_t>() : ch_sums_own.as<uint32_t>();
  XLOG_LAUNCH(c, k_fill_i32, grid_for(slots, 256 * 8), 256, 0, table, slots, empty);
  XLOG_CUDA(cudaMemsetAsync(bitmap, 0, (size_t)bm_quads * 16, c->stream));
  XLOG_CUDA(cudaMemsetAsync(present, 0, (size_t)bm_quads * 16, c->stream));
  // what the relation holds now (its loaded facts, or the result of an earlier fixpoint) is the starting state
  const uint32_t n_start = H.n;
  if (n_start)
    XLOG_LAUNCH(c, (k_mirror_scatter<uint32_t>), grid_for(n_start, 256, 1 << 30), 256, 0, (const uint32_t*)H.keys(), (const float*)H.tags(), n_start, H.layout, M, table, present);
  zero_ctrl(c, kSlotMirNew, 2);
  const MirrorArgs mr{table, reinterpret_cast<uint32_t*>(bitmap), (unsigned long long*)(c->d_ctrl + kSlotMirNew), (uint32_t)(dom - 1),
                      ctrl_u32(c, kSlotErr)};
  c->unique_untracked = true;
  KeyTags delta_own;                       // host-driven rounds without persistent buffers keep their delta here
  const void* dk = nullptr; const float* dt = nullptr; uint32_t dn = 0;
  uint64_t total_new = 0;
  // count -> scan -> one control read -> join into the table, for a list of rule variants; returns the candidate total
  auto host_apply = [&](std::vector<Variant>& vs) -> uint64_t {
    if (vs.size() > 16) fail(XLOG_ERR_UNSUPPORTED, "too many rule variants for one head");
    std::vector<Counted> counted;
    counted.reserve(vs.size());
    uint64_t total = 0;
    for (Variant& v : vs) {
      if (v.outer.n == 0) continue;
      if (grouped && v.outer.keys == dk && v.rule->plan.atoms[v.outer_atom].rel == h) {
        // a delta variant of the grouped shape: the delta is ordered by the probed column
        const uint64_t t = grouped_apply(c, v, H, M, carried_bits, is_max, mr);
        if (t != UINT64_MAX) { total += t; c->r_candidates += (int64_t)t; continue; }
      }
      counted.emplace_back();
      count_variant(c, v, H, counted.back(), kSlotTotals + (int)counted.size() - 1, ML);
    }
    if (!counted.empty()) {
      sync_ctrl(c);
      for (Counted& q : counted) { q.total = c->h_ctrl[q.slot]; total += q.total; q.deg.reset(); q.sums.reset(); }
    }
    for (Counted& q : counted) c->r_candidates += (int64_t)q.total;
    for (Counted& q : counted) {
      if (q.total) {
        // per candidate: the looked-up atom's other columns and tag are read, and the key's slot is read (and now and then written)
        c->note_bytes = (int64_t)q.total * (4 + (q.spec.has_inner ? 4 * (q.spec.inner_free + 1) : 0));
        launch_expand_mirror(c, q, is_max, mr);
      }
      q.start.reset(); q.rowinfo.reset();
    }
    return total;
  };
  auto over_h = [&](const RuleC* r) {
    for (int j = 0; j < r->plan.n_atoms; ++j) if (r->plan.atoms[j].rel == h) return true;
    return false;
  };

  int64_t round = 0;
  bool plain_rules_done = false;           // the rules without an atom over H have had their one evaluation
  bool converged = false;
  if (R) {
    // Resident route.  Seed round, part one: rules without an atom over H are evaluated once, by the host (they scan whole
    // relations of known size).  Part two and every later round run on the device: for the rules over H the seed round
    // is a delta round whose delta is everything H holds now.
    std::vector<Variant> plain;
    for (const RuleC* r : rs)
      if (!over_h(r)) { const int outer = seed_outer(comp, r); plain.push_back(Variant{r, outer, full_source(*c->rels[r->plan.atoms[outer].rel])}); }
    host_apply(plain);
    plain_rules_done = true;
    if (n_start) {
      XLOG_CUDA(cudaMemcpyAsync(R->dkeys.p, H.keys(), (size_t)n_start * 4, cudaMemcpyDeviceToDevice, c->stream));
      XLOG_CUDA(cudaMemcpyAsync(R->dtags.p, H.tags(), (size_t)n_start * 4, cudaMemcpyDeviceToDevice, c->stream));
    }
    const ResState s = run_resident(c, *R, h, rs, is_max, mr, bm_quads, ch_tiles, n_start, c->max_iter, 0);
    round = s.rounds;
    c->r_iterations += s.rounds; c->r_candidates += (int64_t)s.candidates;
    c->r_new += (int64_t)s.n_new; c->r_improved += (int64_t)s.n_improved;
    total_new = s.new_seen;
    dk = R->dkeys.p; dt = R->dtags.as<float>(); dn = s.n_delta;
    if (s.status == kResCap) fail(XLOG_ERR_CONVERGENCE_FAILURE, "iteration cap reached before the fixpoint");
    if (s.status == kResOk) converged = true;             // the delta ran empty
    // kResOverflow: a round needs more expand tiles than planned; the host redoes that round and finishes the job
  }
  for (; !converged; ++round) {
    if (round >= c->max_iter) fail(XLOG_ERR_CONVERGENCE_FAILURE, "iteration cap reached before the fixpoint");
    ++c->r_iterations;
    std::vector<Variant> vs;
    for (const RuleC* r : rs) {
      if (round == 0) {
        if (plain_rules_done && !over_h(r)) continue;
        const int outer = seed_outer(comp, r);
        vs.push_back(Variant{r, outer, full_source(*c->rels[r->plan.atoms[outer].rel])});
      } else {
        if (r == doubling) continue;                      // both of its delta variants run in the dense round below
        for (int j = 0; j < r->plan.n_atoms; ++j)
          if (r->plan.atoms[j].rel == h && dn) vs.push_back(Variant{r, j, Source{dk, dt, dn, M, H.key_bytes}});
      }
    }
    uint64_t total = 0;
    const bool dense_round = doubling && round > 0 && dn > 0;
    if (dense_round) {
      // path doubling: snapshot the matrix, then one block per row applies both delta variants (dense_closure.cuh)
      XLOG_CUDA(cudaMemcpyAsync(snap_own.p, table, slots * 4, cudaMemcpyDeviceToDevice, c->stream));
      zero_ctrl(c, kSlotDense);
      XLOG_LAUNCH(c, k_dense_rowstart, (dense_rows + 1 + 255) / 256, 256, 0, (const uint32_t*)dk, dn, dense_bits1, dense_rows, rowstart_own.as<uint32_t>());
      const DenseRound D{snap_own.as<int32_t>(), table, reinterpret_cast<uint32_t*>(bitmap), (const uint32_t*)dk, dt, rowstart_own.as<uint32_t>(), dense_rows,
                         dense_bits1, (unsigned long long*)(c->d_ctrl + kSlotDense)};
      c->note_bytes = (int64_t)slots * 8 + (int64_t)dn * 8;
#define XLOG_DENSE_ROUND(COLS)                                                                                                  \
  do {                                                                                                                          \
    if (is_max) XLOG_LAUNCH(c, (k_dense_round<kSinkMax, COLS>), dense_rows, kDenseRoundBlock, dense_round_smem(dense_bits1), D); \
    else XLOG_LAUNCH(c, (k_dense_round<kSinkMin, COLS>), dense_rows, kDenseRoundBlock, dense_round_smem(dense_bits1), D);        \
  } while (0)
      switch (std::max(dense_bits1 - 8, 0)) {              // columns per thread = row length / 256
        case 0: XLOG_DENSE_ROUND(1); break;
        case 1: XLOG_DENSE_ROUND(2); break;
        case 2: XLOG_DENSE_ROUND(4); break;
        case 3: XLOG_DENSE_ROUND(8); break;
        default: XLOG_DENSE_ROUND(16); break;
      }
#undef XLOG_DENSE_ROUND
      total = 1;                                         // the candidate count arrives with the round's control read
    }
    total += host_apply(vs);
    if (total == 0 && !(round == 0 && plain_rules_done)) break;
    if (bj.valid) {
      // Every later round is  k_bm_plan -> one control read -> k_bm_expand : the plan kernel closes the round just joined
      // (changed / new keys, bitmap cleared, the changed keys' tags set aside) and lays out the next one's work items.
      const uint32_t nwords = bm_quads * 4;
      BmPlan P{reinterpret_cast<uint32_t*>(bitmap), present, nwords, table, bj.pairs.as<uint2>(), carried_bits - 5, bj.spec.inner_off,
               (uint32_t)std::min<int64_t>(bj.spec.inner_domain, 0xffffffffll), bj.items.as<uint4>(), (unsigned long long*)(c->d_ctrl + kSlotBm)};
      BmExpand E{bj.items.as<uint4>(), 0, bj.spec.inner_col[0], bj.spec.inner_tag, H.layout.mask[1], carried_bits,
                 bj.pairs.as<uint2>(), table, reinterpret_cast<uint32_t*>(bitmap), ctrl_u32(c, kSlotErr)};
      for (;;) {
        zero_ctrl(c, kSlotBm, kBmTotals);
        c->note_bytes = (int64_t)nwords * 4;              // plus 12 bytes per changed key and 16 per item, not known yet
        XLOG_LAUNCH(c, k_bm_plan, (nwords + kBmPlanTile - 1) / kBmPlanTile, kBmPlanBlock, 0, P);
        sync_ctrl(c);
        const uint64_t changed = c->h_ctrl[kSlotBm + kBmChanged], n_new = c->h_ctrl[kSlotBm + kBmNew], cand = c->h_ctrl[kSlotBm + kBmCandidates];
        const uint64_t n_items = c->h_ctrl[kSlotBm + kBmReserve] >> 32, nbrs = c->h_ctrl[kSlotBm + kBmNeighbours];
        total_new += n_new;
        c->r_new += (int64_t)n_new; c->r_improved += (int64_t)changed - (int64_t)n_new;
        if (changed == 0) break;
        ++round;
        if (round >= c->max_iter) fail(XLOG_ERR_CONVERGENCE_FAILURE, "iteration cap reached before the fixpoint");
        ++c->r_iterations;
        if (cand == 0) break;
        c->r_candidates += (int64_t)cand;
        E.n_items = (uint32_t)n_items;
        // per candidate its slot; per (b, neighbour) the looked-up column and tag; per item its record; per changed key its pair
        c->note_bytes = (int64_t)cand * 4 + (int64_t)nbrs * 8 + (int64_t)n_items * 16 + (int64_t)changed * 8;
        const unsigned grid = (unsigned)std::min<uint64_t>((n_items + 7) / 8, (uint64_t)kSMs * 8 * 16);
        if (is_max) XLOG_LAUNCH(c, (k_bm_expand<kSinkMax>), grid, 256, 0, E);
        else XLOG_LAUNCH(c, (k_bm_expand<kSinkMin>), grid, 256, 0, E);
      }
      break;
    }
    launch_changed_count(c, reinterpret_cast<const uint32_t*>(bitmap), present, bm_quads * 4, ch_tiles, ch_sums, mr.n_new);
    XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, ch_sums, (int64_t)ch_tiles, ctrl_u32(c, kSlotMirChanged));
    sync_ctrl(c);
    const uint32_t changed = (uint32_t)c->h_ctrl[kSlotMirChanged];
    if (dense_round) c->r_candidates += (int64_t)c->h_ctrl[kSlotDense];
    const uint64_t n_new = c->h_ctrl[kSlotMirNew] - total_new;
    total_new += n_new;
    c->r_new += (int64_t)n_new; c->r_improved += (int64_t)changed - (int64_t)n_new;
    if (changed == 0) break;
    uint32_t* ek; float* et;
    if (R) { ek = R->dkeys.as<uint32_t>(); et = R->dtags.as<float>(); }
    else {
      delta_own = KeyTags();
      delta_own.keys = DevBuf(c, (size_t)changed * 4);
      delta_own.tags = DevBuf(c, (size_t)changed * 4);
      ek = delta_own.keys.as<uint32_t>(); et = delta_own.tags.as<float>();
    }
    c->note_bytes = (int64_t)bm_quads * 16 + (int64_t)changed * 12;
    launch_changed_emit(c, reinterpret_cast<uint32_t*>(bitmap), bm_quads * 4, ch_tiles, ch_sums, table, ek, et, nullptr);
    dk = ek; dt = et; dn = changed;
  }
  // the relation in sorted form: every occupied slot, in slot order
  const uint64_t n_out = (uint64_t)n_start + total_new;
  KeyTags full;
  full.n = (uint32_t)n_out;
  full.keys = DevBuf(c, (size_t)std::max<uint64_t>(n_out, 1) * 4);
  full.tags = DevBuf(c, (size_t)std::max<uint64_t>(n_out, 1) * 4);
  bool counted_slots = false;              // kSlotA holds the number of occupied slots (for the invariant check)
  if (n_out && grouped && carried_bits <= 6) {
    // the mirror is ordered (column 1, column 0) and column 0 has at most 64 values: every row goes straight to its place
    // in the relation's order (mirror.cuh), found from the bitmap of present keys; no pass over empty slots, no sort
    const int per_node = 1 << carried_bits;
    const uint32_t n_nodes = (uint32_t)(slots >> carried_bits);
    const uint32_t ntiles = (n_nodes + kMtNodes - 1) / kMtNodes;
    const int64_t len = (int64_t)per_node * ntiles;
    const unsigned stiles = (unsigned)((len + kScanTile - 1) / kScanTile);
    DevBuf cnt(c, (size_t)len * 4), base(c, (size_t)len * 4), sums(c, (size_t)stiles * 4);
    c->note_bytes = (int64_t)slots / 8;
    XLOG_LAUNCH(c, k_mirror_t_count, ntiles, kMtNodes, 0, (const uint32_t*)present, n_nodes, ntiles, per_node, cnt.as<uint32_t>());
    XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint32_t>), stiles, kScanBlock, 0, (const uint32_t*)cnt.as<uint32_t>(), len, sums.as<uint32_t>());
    XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, sums.as<uint32_t>(), (int64_t)stiles, ctrl_u32(c, kSlotA));
    XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint32_t>), stiles, kScanBlock, 0, (const uint32_t*)cnt.as<uint32_t>(), len, (const uint32_t*)sums.as<uint32_t>(),
                base.as<uint32_t>());
    c->note_bytes = (int64_t)slots / 8 + (int64_t)n_out * 12;
    XLOG_LAUNCH(c, (k_mirror_t_emit<uint32_t>), ntiles, kMtNodes, 0, (const uint32_t*)present, (const int32_t*)table, n_nodes, ntiles, per_node,
                (const uint32_t*)base.as<uint32_t>(), H.layout.shift[0], H.layout.shift[1], full.keys.as<uint32_t>(), full.tags.as<float>());
    counted_slots = true;
  } else if (n_out) {
    const uint64_t nquads = slots / 4;
    const unsigned tiles = (unsigned)((slots + kMirSlotsPerTile - 1) / kMirSlotsPerTile);
    DevBuf sums(c, (size_t)tiles * 4);
    c->note_bytes = (int64_t)slots * 4;
    XLOG_LAUNCH(c, k_mirror_full_count, tiles, kMirBlock, 0, (const int4*)table, nquads, empty, sums.as<uint32_t>());
    XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, sums.as<uint32_t>(), (int64_t)tiles, ctrl_u32(c, kSlotA));
    c->note_bytes = (int64_t)slots * 4 + (int64_t)n_out * 8;
    XLOG_LAUNCH(c, (k_mirror_full_emit<uint32_t>), tiles, kMirBlock, 0, (const int4*)table, nquads, empty, (const uint32_t*)sums.as<uint32_t>(), M, H.layout,
                full.keys.as<uint32_t>(), full.tags.as<float>());
    counted_slots = true;
    if (grouped && n_out > 1) {
      // rows came out in the mirror's order, (column 1, column 0) ascending: a stable sort on column 0's bits alone puts
      // them in the relation's key order
      table_own.reset(); bitmap_own.reset(); present_own.reset(); bj.pairs.reset(); bj.items.reset();
      DevBuf ak(c, (size_t)n_out * 4), at(c, (size_t)n_out * 4);
      uint32_t* pk = full.keys.as<uint32_t>(); uint32_t* qk = ak.as<uint32_t>();
      float* pt = full.tags.as<float>(); float* qt = at.as<float>();
      sort_pairs<uint32_t>(c, pk, pt, qk, qt, n_out, bits, H.layout.shift[0]);
      if ((void*)pk != full.keys.p) { std::swap(full.keys, ak); std::swap(full.tags, at); }
    }
  }
  set_current(H, std::move(full));
  if (c->flags & XLOG_FLAG_CHECK_INVARIANTS) {
    XLOG_LAUNCH(c, (k_check_sorted<uint32_t>), grid_for(H.n, 256), 256, 0, (const uint32_t*)H.keys(), (int64_t)H.n, ctrl_u32(c, kSlotErr));
    sync_ctrl(c);
    if (n_out && counted_slots && (uint64_t)(uint32_t)c->h_ctrl[kSlotA] != n_out) fail(XLOG_ERR_INTERNAL, "tag mirror: occupied slots disagree with the tuple count");
  }
}

// ---- several heads in one component (mutual recursion) ----------------------------------------------------------------

// Mutually recursive max / min heads, each over its own tag mirror, when every rule reads at most one relation of the
// component (so the looked-up side of every join is a relation of a lower stratum, indexed once).
bool mirror_multi_applies(Ctx* c, const std::vector<int>& comp, const std::vector<const RuleC*>& rs) {
  if ((c->flags & XLOG_FLAG_NO_TAG_MIRROR) || comp.size() < 2 || comp.size() > (size_t)kMultiMaxHeads) return false;
  uint64_t need = 1u << 20;
  for (int h : comp) {
    const Relation& H = *c->rels[h];
    if (H.sr != XLOG_SR_MAXPLUS && H.sr != XLOG_SR_MINPLUS) return false;
    if (H.layout.total_bits > kMirrorMaxBits || H.key_bytes != 4) return false;
    need += ((uint64_t)4 << H.layout.total_bits) + ((uint64_t)1 << H.layout.total_bits) / 4 + (1u << 16);
  }
  for (const RuleC* r : rs) {
    if (r->plan.emit_count_column || (r->kind != 1 && r->kind != 2)) return false;
    int in = 0, pos = 0;
    for (int j = 0; j < r->plan.n_atoms; ++j)
      if (in_set(comp, r->plan.atoms[j].rel)) { if (r->plan.atoms[j].negated) return false; ++in; pos = j; }
    if (in > 1) return false;
    if (in == 1 && r->kind == 2 && !r->shape[pos].ok) return false;
    if (in == 1 && r->kind != 2 && pos != 0) return false;
    if (in == 0 && r->kind == 2 && !r->shape[0].ok && !r->shape[1].ok) return false;
  }
  return need <= c->arena.largest_free() / 2;
}

// Algorithm 1 over one tag mirror per head.  A round applies every delta variant of every rule to its head's table (the
// deltas are lists written at the end of the round before, so all heads see the same state), then each head's changed
// bitmap becomes its next delta.  Two control reads per round: the variants' candidate totals, the heads' changed counts.
void stratum_recursive_mirror_multi(Ctx* c, const std::vector<int>& comp, const std::vector<const RuleC*>& rs) {
  {
    std::vector<RowRule> row_rules;
    if (row_fixpoint_applies(c, comp, rs, row_rules)) { stratum_row_fixpoint(c, comp, rs, row_rules); return; }
  }
  struct Head {
    int h; Relation* H; bool is_max; int32_t empty; uint64_t slots; uint32_t bm_quads; unsigned ch_tiles;
    DevBuf table, bitmap, present, ch_sums;
    KeyTags delta; uint32_t n_start; uint64_t total_new; MirrorArgs mr;
  };
  std::vector<Head> heads(comp.size());
  zero_ctrl(c, kSlotMultiChanged, 2 * kMultiMaxHeads);
  for (size_t i = 0; i < comp.size(); ++i) {
    Head& X = heads[i];
    X.h = comp[i]; X.H = c->rels[comp[i]];
    Relation& H = *X.H;
    const uint64_t dom = (uint64_t)1 << H.layout.total_bits;
    X.is_max = H.sr == XLOG_SR_MAXPLUS;
    X.empty = X.is_max ? kMirrorEmptyMax : kMirrorEmptyMin;
    X.slots = std::max<uint64_t>(dom, 4);
    X.bm_quads = (uint32_t)((std::max<uint64_t>(dom / 32, 1) + 3) / 4);
    X.ch_tiles = mirror_tiles(X.bm_quads * 4);
    X.table = DevBuf(c, X.slots * 4); X.bitmap = DevBuf(c, (size_t)X.bm_quads * 16); X.present = DevBuf(c, (size_t)X.bm_quads * 16);
    X.ch_sums = DevBuf(c, (size_t)X.ch_tiles * 4);
    X.n_start = H.n; X.total_new = 0;
    XLOG_LAUNCH(c, k_fill_i32, grid_for(X.slots, 256 * 8), 256, 0, X.table.as<int32_t>(), X.slots, X.empty);
    XLOG_CUDA(cudaMemsetAsync(X.bitmap.p, 0, (size_t)X.bm_quads * 16, c->stream));
    XLOG_CUDA(cudaMemsetAsync(X.present.p, 0, (size_t)X.bm_quads * 16, c->stream));
    if (X.n_start)
      XLOG_LAUNCH(c, (k_mirror_scatter<uint32_t>), grid_for(X.n_start, 256, 1 << 30), 256, 0, (const uint32_t*)H.keys(), (const float*)H.tags(), X.n_start, H.layout,
                  H.layout, X.table.as<int32_t>(), X.present.as<uint32_t>());
    X.mr = MirrorArgs{X.table.as<int32_t>(), X.bitmap.as<uint32_t>(), (unsigned long long*)(c->d_ctrl + kSlotMultiNew + i), (uint32_t)(dom - 1),
                      ctrl_u32(c, kSlotErr)};
  }
  c->unique_untracked = true;
  auto head_of = [&](int rel) -> Head& { for (Head& X : heads) if (X.h == rel) return X; return heads[0]; };
  for (int64_t round = 0;; ++round) {
    if (round >= c->max_iter) fail(XLOG_ERR_CONVERGENCE_FAILURE, "iteration cap reached before the fixpoint");
    ++c->r_iterations;
    std::vector<Variant> vs;
    for (const RuleC* r : rs) {
      if (round == 0) {                                     // seed: every atom reads the full relation
        const int outer = seed_outer(comp, r);
        vs.push_back(Variant{r, outer, full_source(*c->rels[r->plan.atoms[outer].rel])});
      } else {
        for (int j = 0; j < r->plan.n_atoms; ++j) {
          const int ar = r->plan.atoms[j].rel;
          if (!in_set(comp, ar)) continue;
          const Head& D = head_of(ar);
          if (D.delta.n) vs.push_back(Variant{r, j, Source{D.delta.keys.p, D.delta.tags.as<float>(), D.delta.n, D.H->layout, D.H->key_bytes}});
        }
      }
    }
    // the candidate totals of a round's variants are settled sixteen at a time, by one control read
    uint64_t total = 0;
    for (size_t v0 = 0; v0 < vs.size(); v0 += 16) {
      std::vector<Counted> counted;
      std::vector<Head*> target;
      counted.reserve(16);
      for (size_t v = v0; v < std::min(vs.size(), v0 + 16); ++v) {
        if (vs[v].outer.n == 0) continue;
        Head& T = head_of(vs[v].rule->plan.head_rel);
        counted.emplace_back();
        count_variant(c, vs[v], *T.H, counted.back(), kSlotTotals + (int)counted.size() - 1);
        target.push_back(&T);
      }
      if (counted.empty()) continue;
      sync_ctrl(c);
      for (size_t i = 0; i < counted.size(); ++i) {
        Counted& q = counted[i];
        q.total = c->h_ctrl[q.slot];
        q.deg.reset(); q.sums.reset();
        total += q.total;
        c->r_candidates += (int64_t)q.total;
        if (q.total) {
          c->note_bytes = (int64_t)q.total * (4 + (q.spec.has_inner ? 4 * (q.spec.inner_free + 1) : 0));
          launch_expand_mirror(c, q, target[i]->is_max, target[i]->mr);
        }
      }
    }
    if (total == 0) break;
    for (size_t i = 0; i < heads.size(); ++i) {
      Head& X = heads[i];
      launch_changed_count(c, X.bitmap.as<uint32_t>(), X.present.as<uint32_t>(), X.bm_quads * 4, X.ch_tiles, X.ch_sums.as<uint32_t>(), X.mr.n_new);
      XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, X.ch_sums.as<uint32_t>(), (int64_t)X.ch_tiles, ctrl_u32(c, kSlotMultiChanged + (int)i));
    }
    sync_ctrl(c);
    uint64_t changed_all = 0;
    for (size_t i = 0; i < heads.size(); ++i) {
      Head& X = heads[i];
      const uint32_t changed = (uint32_t)c->h_ctrl[kSlotMultiChanged + i];
      const uint64_t n_new = c->h_ctrl[kSlotMultiNew + i] - X.total_new;
      X.total_new += n_new;
      c->r_new += (int64_t)n_new; c->r_improved += (int64_t)changed - (int64_t)n_new;
      changed_all += changed;
      X.delta = KeyTags();
      X.delta.n = changed;
      if (changed == 0) continue;
      X.delta.keys = DevBuf(c, (size_t)changed * 4);
      X.delta.tags = DevBuf(c, (size_t)changed * 4);
      c->note_bytes = (int64_t)X.bm_quads * 16 + (int64_t)changed * 12;
      launch_changed_emit(c, X.bitmap.as<uint32_t>(), X.bm_quads * 4, X.ch_tiles, X.ch_sums.as<uint32_t>(), X.table.as<int32_t>(), X.delta.keys.as<uint32_t>(),
                          X.delta.tags.as<float>(), nullptr);
    }
    if (changed_all == 0) break;
  }
  // every head in sorted form: the occupied slots in slot order
  for (Head& X : heads) {
    Relation& H = *X.H;
    X.delta = KeyTags();
    const uint64_t n_out = (uint64_t)X.n_start + X.total_new;
    KeyTags full;
    full.n = (uint32_t)n_out;
    full.keys = DevBuf(c, (size_t)std::max<uint64_t>(n_out, 1) * 4);
    full.tags = DevBuf(c, (size_t)std::max<uint64_t>(n_out, 1) * 4);
    if (n_out) {
      const uint64_t nquads = X.slots / 4;
      const unsigned tiles = (unsigned)((X.slots + kMirSlotsPerTile - 1) / kMirSlotsPerTile);
      DevBuf sums(c, (size_t)tiles * 4);
      c->note_bytes = (int64_t)X.slots * 4;
      XLOG_LAUNCH(c, k_mirror_full_count, tiles, kMirBlock, 0, (const int4*)X.table.as<int4>(), nquads, X.empty, sums.as<uint32_t>());
      XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, sums.as<uint32_t>(), (int64_t)tiles, ctrl_u32(c, kSlotA));
      c->note_bytes = (int64_t)X.slots * 4 + (int64_t)n_out * 8;
      XLOG_LAUNCH(c, (k_mirror_full_emit<uint32_t>), tiles, kMirBlock, 0, (const int4*)X.table.as<int4>(), nquads, X.empty, (const uint32_t*)sums.as<uint32_t>(), H.layout,
                  H.layout, full.keys.as<uint32_t>(), full.tags.as<float>());
    }
    set_current(H, std::move(full));
    X.table.reset(); X.bitmap.reset(); X.present.reset(); X.ch_sums.reset();
    if (c->flags & XLOG_FLAG_CHECK_INVARIANTS) {
      XLOG_LAUNCH(c, (k_check_sorted<uint32_t>), grid_for(H.n, 256), 256, 0, (const uint32_t*)H.keys(), (int64_t)H.n, ctrl_u32(c, kSlotErr));
      sync_ctrl(c);
      if (n_out && (uint64_t)(uint32_t)c->h_ctrl[kSlotA] != n_out) fail(XLOG_ERR_INTERNAL, "tag mirror: occupied slots disagree with the tuple count");
    }
  }
}

}  // namespace
}  // namespace xlog
