// Cyclic joins: the fused triangle aggregate, the materialised triangle join (two plans + skew test) and the four-cycle join.
// Host-side driver code of the engine; included by xlog_api.cu only (one translation unit).
#pragma once
#include "host_eval.cuh"
#include "triangle.cuh"
#include "cycle4.cuh"

namespace xlog {
namespace {

// Turn groups keyed by the declared head columns into rows of the counted head relation:
// (declared columns..., group size), tag unchanged.  `counts` has one entry per group.
void append_counts(Ctx* c, Relation& H, KeyTags& u, const KeyLayout& cl, const uint32_t* counts, uint32_t max_count) {
  if (max_count > (uint32_t)INT32_MAX) fail(XLOG_ERR_CAPACITY_EXCEEDED, "count exceeds INT32_MAX");
  const int nd = cl.arity;
  H.col_max[nd] = (int32_t)max_count;
  const KeyLayout L = make_layout(H.arity, H.col_max);
  if (L.total_bits > 64) fail(XLOG_ERR_CAPACITY_EXCEEDED, "packed key of relation '" + H.name + "' needs more than 64 bits");
  const int kb_in = cl.total_bits <= 32 ? 4 : 8, kb_out = L.total_bits <= 32 ? 4 : 8;
  const int cbits = L.shift[nd - 1];               // bits of the count column = shift of the column before it
  KeyTags out;
  out.n = u.n;
  out.keys = DevBuf(c, (size_t)std::max(u.n, 1u) * kb_out);
  out.tags = std::move(u.tags);
  if (u.n) {
    const unsigned g = grid_for(u.n, 256);
    if (kb_in == 4 && kb_out == 4) XLOG_LAUNCH(c, (k_append_count<uint32_t, uint32_t>), g, 256, 0, u.keys.as<uint32_t>(), counts, u.n, cbits, out.keys.as<uint32_t>());
    else if (kb_in == 4) XLOG_LAUNCH(c, (k_append_count<uint32_t, uint64_t>), g, 256, 0, u.keys.as<uint32_t>(), counts, u.n, cbits, out.keys.as<uint64_t>());
    else XLOG_LAUNCH(c, (k_append_count<uint64_t, uint64_t>), g, 256, 0, u.keys.as<uint64_t>(), counts, u.n, cbits, out.keys.as<uint64_t>());
  }
  H.layout = L;
  H.key_bytes = kb_out;
  set_current(H, std::move(out));
}

void append_count_column(Ctx* c, Relation& H, KeyTags& u, const KeyLayout& cl) {
  DevBuf counts(c, (size_t)std::max(u.n, 1u) * 4);
  zero_ctrl(c, kSlotD);
  if (u.n) XLOG_LAUNCH(c, k_group_sizes, grid_for(u.n, 256), 256, 0, (const uint32_t*)u.head_pos.as<uint32_t>(), u.n, counts.as<uint32_t>(), ctrl_u32(c, kSlotD));
  sync_ctrl(c);
  append_counts(c, H, u, cl, counts.as<uint32_t>(), (uint32_t)c->h_ctrl[kSlotD]);
}

// h(x[, count]) :- e(x,y), e(y,z), e(z,x): per-edge sorted-list intersection, then per-x combination.
template <typename Op>
void triangle_aggregate_t(Ctx* c, Relation& H, const RuleC& r) {
  typedef typename Op::A A;
  Relation& E = *c->rels[r.plan.atoms[0].rel];
  const bool counted = r.plan.emit_count_column != 0;
  int32_t mx[kMaxArity] = {H.col_max[0], 0, 0, 0};
  const KeyLayout cl = make_layout(1, mx);
  if (E.n == 0) { KeyTags empty; set_current(H, std::move(empty)); return; }
  Index& out_ix = ensure_index(c, E, 0);
  Index& in_ix = ensure_index(c, E, 1);
  TriGraph G{};
  G.n_edges = E.n;
  G.src = E.cols[0].as<int32_t>(); G.dst = E.cols[1].as<int32_t>(); G.w = E.tags();
  G.out_domain = out_ix.domain; G.in_domain = in_ix.domain;
  G.out_off = out_ix.off.as<uint32_t>(); G.in_off = in_ix.off.as<uint32_t>();
  G.in_src = in_ix.other[0]; G.in_w = in_ix.tags;
  G.s_dst = G.dst; G.s_w = G.w;
  const int64_t domain = out_ix.domain;
  // work items: edges cut into slices of the walked list (count -> scan -> one control read for the item total)
  const uint32_t ne1 = E.n + 1;
  DevBuf items(c, (size_t)ne1 * 4), item_off(c, (size_t)ne1 * 4);
  const unsigned it_tiles = (ne1 + kScanTile - 1) / kScanTile;
  DevBuf it_sums(c, (size_t)it_tiles * 4);
  zero_ctrl(c, kSlotA, 4);
  // per x: search the longer list, or mark in(x) in a shared-memory bitmap and walk every out(y) against it (triangle.cuh)
  // the bitmap holds sources of edges into x (values of column 0) and is probed with targets (values of column 1): both ranges must fit
  const int64_t node_domain = std::max(in_ix.domain, out_ix.domain);
  const bool bitmap_ok = !(c->flags & XLOG_FLAG_NO_TRIANGLE_BITMAP) && node_domain <= kTriBitmapMaxDomain;
  const int64_t sum_n = std::max<int64_t>(in_ix.domain, 1);
  DevBuf route_sums(c, bitmap_ok ? (size_t)sum_n * 16 : 16);
  TriRoute RT{route_sums.as<unsigned long long>(), route_sums.as<unsigned long long>() + (bitmap_ok ? sum_n : 0), bitmap_ok ? 1 : 0};
  if (bitmap_ok) {
    XLOG_CUDA(cudaMemsetAsync(route_sums.p, 0, (size_t)sum_n * 16, c->stream));
    XLOG_LAUNCH(c, k_tri_route_sums, grid_for(E.n, 256), 256, 0, G, route_sums.as<unsigned long long>(), route_sums.as<unsigned long long>() + sum_n);
  }
  XLOG_LAUNCH(c, k_tri_plan, grid_for(ne1, 256), 256, 0, G, RT, items.as<uint32_t>(), (unsigned long long*)(c->d_ctrl + kSlotC),
              (unsigned long long*)(c->d_ctrl + kSlotD));
  XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint32_t>), it_tiles, kScanBlock, 0, (const uint32_t*)items.as<uint32_t>(), (int64_t)ne1, it_sums.as<uint32_t>());
  XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, it_sums.as<uint32_t>(), (int64_t)it_tiles, ctrl_u32(c, kSlotB));
  XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint32_t>), it_tiles, kScanBlock, 0, (const uint32_t*)items.as<uint32_t>(), (int64_t)ne1,
              (const uint32_t*)it_sums.as<uint32_t>(), item_off.as<uint32_t>());
  // the bitmap kernel's units: the work items of one x in slices (count -> scan; the total arrives with the same control read)
  const int64_t nd1 = domain + 1;
  const unsigned un_tiles = (unsigned)((nd1 + kScanTile - 1) / kScanTile);
  DevBuf units(c, bitmap_ok ? (size_t)nd1 * 4 : 4), unit_off(c, bitmap_ok ? (size_t)nd1 * 4 : 4), un_sums(c, (size_t)un_tiles * 4);
  if (bitmap_ok) {
    XLOG_LAUNCH(c, k_tri_unit_count, grid_for(nd1, 256), 256, 0, G, RT, G.out_off, domain, (const uint32_t*)item_off.as<uint32_t>(), units.as<uint32_t>());
    XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint32_t>), un_tiles, kScanBlock, 0, (const uint32_t*)units.as<uint32_t>(), nd1, un_sums.as<uint32_t>());
    XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, un_sums.as<uint32_t>(), (int64_t)un_tiles, ctrl_u32(c, kSlotA));
    XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint32_t>), un_tiles, kScanBlock, 0, (const uint32_t*)units.as<uint32_t>(), nd1, (const uint32_t*)un_sums.as<uint32_t>(),
                unit_off.as<uint32_t>());
  }
  sync_ctrl(c);
  const uint32_t n_items = (uint32_t)c->h_ctrl[kSlotB];
  const uint32_t n_units = bitmap_ok ? (uint32_t)c->h_ctrl[kSlotA] : 0u;
  const uint64_t walked = c->h_ctrl[kSlotC];               // list entries walked by the whole join (one probe each)
  const uint64_t walked_bitmap = c->h_ctrl[kSlotD];        // those of them the bitmap kernel walks
  items.reset(); it_sums.reset(); units.reset(); un_sums.reset();
  DevBuf item_edge(c, (size_t)std::max(n_items, 1u) * 4), ecnt(c, (size_t)std::max(n_items, 1u) * 4), eacc(c, (size_t)std::max(n_items, 1u) * sizeof(A));
  DevBuf gcnt(c, (size_t)domain * 4), gtag(c, (size_t)domain * 4), flag(c, (size_t)domain * 4);
  const unsigned scan_tiles = (unsigned)((domain + kScanTile - 1) / kScanTile);
  DevBuf spine(c, ((size_t)scan_tiles + 1) * 4);
  zero_ctrl(c, kSlotA, 4);
  XLOG_LAUNCH(c, k_tri_item_edges, grid_for(E.n, 256), 256, 0, E.n, (const uint32_t*)item_off.as<uint32_t>(), item_edge.as<uint32_t>());
  // declared work: one 4-byte entry per probe (the walked lists) plus the edge rows; the searches themselves hit L1 / L2
  c->note_bytes = (int64_t)(walked - walked_bitmap) * 4 + (int64_t)E.n * 12;
  c->r_candidates += (int64_t)walked;
  XLOG_LAUNCH(c, (k_tri_edges<Op>), kSMs * 8, 256, 0, G, RT, H.sr == XLOG_SR_SUMPROD ? 1 : 0, n_items, (const uint32_t*)item_off.as<uint32_t>(),
              (const uint32_t*)item_edge.as<uint32_t>(), ecnt.as<uint32_t>(), eacc.as<A>());
  if (n_units) {
    DevBuf unit(c, (size_t)n_units * 8);
    XLOG_LAUNCH(c, k_tri_unit_fill, grid_for(domain, 256), 256, 0, G.out_off, domain, (const uint32_t*)item_off.as<uint32_t>(), (const uint32_t*)unit_off.as<uint32_t>(),
                unit.as<uint2>());
    const uint32_t words = (uint32_t)((node_domain + 31) / 32);
    const size_t smem = (size_t)words * 8;
    c->note_bytes = (int64_t)walked_bitmap * 4;
    XLOG_CUDA(cudaFuncSetAttribute(k_tri_bitmap<Op>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kTriBitmapMaxDomain / 32 * 8)));
    XLOG_LAUNCH(c, (k_tri_bitmap<Op>), std::min<unsigned>(n_units, kSMs * 16), 256, smem, G, H.sr == XLOG_SR_SUMPROD ? 1 : 0, n_units, (const uint2*)unit.as<uint2>(),
                G.out_off, (const uint32_t*)item_off.as<uint32_t>(), (const uint32_t*)item_edge.as<uint32_t>(), words, ecnt.as<uint32_t>(), eacc.as<A>());
  }
  XLOG_LAUNCH(c, (k_tri_groups<Op>), grid_for((uint64_t)domain * 32, 256, kSMs * 8), 256, 0, G.out_off, domain, (const uint32_t*)item_off.as<uint32_t>(),
              (const uint32_t*)ecnt.as<uint32_t>(), (const A*)eacc.as<A>(), gcnt.as<uint32_t>(), gtag.as<float>(), flag.as<uint32_t>(), ctrl_u32(c, kSlotD),
              ctrl_u32(c, kSlotErr));
  // positions of the surviving x: exclusive scan of the flags (kept in a second buffer)
  DevBuf pos(c, (size_t)domain * 4);
  XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint32_t>), scan_tiles, kScanBlock, 0, (const uint32_t*)flag.as<uint32_t>(), domain, spine.as<uint32_t>());
  XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, spine.as<uint32_t>(), (int64_t)scan_tiles, ctrl_u32(c, kSlotA));
  XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint32_t>), scan_tiles, kScanBlock, 0, (const uint32_t*)flag.as<uint32_t>(), domain,
              (const uint32_t*)spine.as<uint32_t>(), pos.as<uint32_t>());
  sync_ctrl(c);
  const uint32_t u = (uint32_t)c->h_ctrl[kSlotA], max_count = (uint32_t)c->h_ctrl[kSlotD];
  c->r_unique += u;
  KeyTags kt;
  kt.n = u;
  const int kb = cl.total_bits <= 32 ? 4 : 8;
  kt.keys = DevBuf(c, (size_t)std::max(u, 1u) * kb);
  kt.tags = DevBuf(c, (size_t)std::max(u, 1u) * 4);
  DevBuf counts(c, (size_t)std::max(u, 1u) * 4);
  DISPATCH_K(kb, XLOG_LAUNCH(c, (k_tri_compact<K>), grid_for(domain, 256), 256, 0, (const uint32_t*)flag.as<uint32_t>(), (const uint32_t*)pos.as<uint32_t>(), domain,
                              (const uint32_t*)gcnt.as<uint32_t>(), (const float*)gtag.as<float>(), kt.keys.as<K>(), counts.as<uint32_t>(), kt.tags.as<float>()));
  if (counted) append_counts(c, H, kt, cl, counts.as<uint32_t>(), max_count);
  else set_current(H, std::move(kt));
}

// tri(x,y,z) :- e(x,y), e(y,z), e(z,x): count per edge -> scan -> materialise; the result is born sorted.
// tri(x,y,z) :- r(x,y), s(y,z), t(z,x), materialised.  Two plans (paper: "Worst-case-optimal joins"):
//  - multiway: for every r row intersect s's out-list of y with t's in-list of x (count -> scan -> write);
//  - binary chain: materialise every two-path of r and s with the ordinary join, then keep those t closes.
// A skew test picks one per evaluation: the chain when its intermediate (the two-paths, counted exactly by the join's
// count step) stays within a small multiple of the inputs, the multiway join otherwise.
constexpr uint64_t kChainMaxBlowup = 4;      // two-paths per input row up to which the chain is chosen

void triangle_chain(Ctx* c, Relation& H, const Relation& H2, Counted& q, Relation& T) {
  const int times = H.sr == XLOG_SR_SUMPROD ? 1 : 0;
  const int ckb = H2.key_bytes;
  const uint64_t n2 = q.total;
  // step one: all two-paths (x,y,z) with tag w_xy otimes w_yz, in (x,y,z) order
  DevBuf k0(c, std::max<uint64_t>(n2, 1) * ckb), t0(c, std::max<uint64_t>(n2, 1) * 4);
  c->note_bytes = (int64_t)n2 * (ckb + 4 + 8);
  launch_expand<false>(c, q, 0, n2, ckb, k0.p, t0.as<float>(), BwdArgs{});
  q.start.reset(); q.rowinfo.reset();
  // step two: probe t with (z, x)
  Index& tix = ensure_index(c, T, 0);
  ChainProbe P{};
  P.last = 2;
  P.L = H2.layout; P.out = H.layout;
  P.t_domain = tix.domain; P.t_off = tix.off.as<uint32_t>(); P.t_col1 = tix.other[0]; P.t_w = tix.tags; P.times = times;
  DevBuf hit(c, std::max<uint64_t>(n2, 1) * 4), off(c, std::max<uint64_t>(n2, 1) * 8);
  const unsigned tiles = (unsigned)((n2 + kScanTile - 1) / kScanTile);
  DevBuf sums(c, (size_t)std::max(tiles, 1u) * 8);
  zero_ctrl(c, kSlotTotals);
  c->note_bytes = (int64_t)n2 * (ckb + 4);
  DISPATCH_K(ckb, XLOG_LAUNCH(c, (k_chain_probe_count<K>), grid_for(n2, 256), 256, 0, P, (const K*)k0.p, n2, hit.as<uint32_t>()));
  XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint64_t>), tiles, kScanBlock, 0, (const uint32_t*)hit.as<uint32_t>(), (int64_t)n2, sums.as<uint64_t>());
  XLOG_LAUNCH(c, (k_scan_spine<uint64_t>), 1, 1024, 0, sums.as<uint64_t>(), (int64_t)tiles, (uint64_t*)(c->d_ctrl + kSlotTotals));
  XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint64_t>), tiles, kScanBlock, 0, (const uint32_t*)hit.as<uint32_t>(), (int64_t)n2,
              (const uint64_t*)sums.as<uint64_t>(), off.as<uint64_t>());
  sync_ctrl(c);
  const uint64_t total = c->h_ctrl[kSlotTotals];
  if (total > kSortMaxN) fail(XLOG_ERR_CAPACITY_EXCEEDED, "materialised triangle relation exceeds 2^30 - 1 rows");
  c->r_unique += (int64_t)total;
  KeyTags kt;
  kt.n = (uint32_t)total;
  kt.keys = DevBuf(c, (size_t)std::max<uint64_t>(total, 1) * H.key_bytes);
  kt.tags = DevBuf(c, (size_t)std::max<uint64_t>(total, 1) * 4);
  c->note_bytes = (int64_t)n2 * (ckb + 4 + 12) + (int64_t)total * (H.key_bytes + 4);
#define XLOG_CHAIN_EMIT(K2, KH)                                                                                                     \
  XLOG_LAUNCH(c, (k_chain_probe_emit<K2, KH>), grid_for(n2, 256), 256, 0, P, (const K2*)k0.p, (const float*)t0.as<float>(), n2,    \
              (const uint32_t*)hit.as<uint32_t>(), (const uint64_t*)off.as<uint64_t>(), kt.keys.as<KH>(), kt.tags.as<float>())
  if (n2) {
    if (ckb == 4 && H.key_bytes == 4) XLOG_CHAIN_EMIT(uint32_t, uint32_t);
    else if (ckb == 4) XLOG_CHAIN_EMIT(uint32_t, uint64_t);
    else if (H.key_bytes == 4) XLOG_CHAIN_EMIT(uint64_t, uint32_t);
    else XLOG_CHAIN_EMIT(uint64_t, uint64_t);
  }
#undef XLOG_CHAIN_EMIT
  set_current(H, std::move(kt));
}

void triangle_materialise(Ctx* c, Relation& H, const RuleC& r) {
  Relation& R = *c->rels[r.plan.atoms[0].rel];
  Relation& S = *c->rels[r.plan.atoms[1].rel];
  Relation& T = *c->rels[r.plan.atoms[2].rel];
  if (H.n_facts) fail(XLOG_ERR_UNSUPPORTED, "a materialised triangle relation cannot also hold loaded facts");
  if (R.n == 0 || S.n == 0 || T.n == 0) { KeyTags empty; set_current(H, std::move(empty)); c->last_triangle_plan = XLOG_PLAN_CHAIN; return; }
  const int times = H.sr == XLOG_SR_SUMPROD ? 1 : 0;

  // skew test: count the two-paths of r and s exactly (the chain's intermediate); this is the chain's own count step
  bool chain = (c->flags & XLOG_FLAG_FORCE_CHAIN) != 0;
  if (!(c->flags & (XLOG_FLAG_FORCE_CHAIN | XLOG_FLAG_FORCE_WCOJ)) || chain) {
    RuleC two;                                           // tmp(x,y,z) :- r(x,y), s(y,z)
    two.plan = r.plan;
    two.plan.n_atoms = 2;
    two.kind = 2;
    two.shape[0] = join_shape(c, two.plan, 0);
    if (!two.shape[0].ok) fail(XLOG_ERR_INTERNAL, "triangle chain: no join path");
    Relation H2;                                         // the two-paths' own layout: bounds from r and s alone
    H2.arity = 3; H2.sr = H.sr;
    H2.col_max[0] = R.val_max[0] ? R.val_max[0] : R.col_max[0]; H2.col_max[1] = R.val_max[1] ? R.val_max[1] : R.col_max[1];
    H2.col_max[2] = S.val_max[1] ? S.val_max[1] : S.col_max[1];
    H2.layout = make_layout(3, H2.col_max);
    H2.key_bytes = H2.layout.total_bits <= 32 ? 4 : 8;
    Variant v{&two, 0, full_source(R)};
    Counted q;
    count_variant(c, v, H2, q, kSlotTotals);
    sync_ctrl(c);
    q.total = c->h_ctrl[kSlotTotals];
    q.deg.reset(); q.sums.reset();
    const uint64_t biggest = std::max<uint64_t>(R.n, std::max<uint64_t>(S.n, T.n));
    const size_t need = (size_t)q.total * (H2.key_bytes + 4 + 12) + (16u << 20);
    const bool fits = q.total <= kSortMaxN && need <= c->arena.largest_free() / 2;
    if (!(c->flags & XLOG_FLAG_FORCE_CHAIN)) chain = fits && q.total <= kChainMaxBlowup * biggest;
    else if (!fits) fail(XLOG_ERR_RESOURCE_EXHAUSTED, "triangle chain: the two-path intermediate does not fit the arena");
    if (chain) {
      c->r_candidates += (int64_t)q.total;
      c->last_triangle_plan = XLOG_PLAN_CHAIN;
      if (q.total == 0) { KeyTags empty; set_current(H, std::move(empty)); return; }      // no two-path at all
      triangle_chain(c, H, H2, q, T);
      return;
    }
  }
  c->last_triangle_plan = XLOG_PLAN_WCOJ;
  Index& out_ix = ensure_index(c, S, 0);
  Index& in_ix = ensure_index(c, T, 1);
  ensure_soa(c, R);
  ensure_soa(c, S);
  TriGraph G{};
  G.n_edges = R.n;
  G.src = R.cols[0].as<int32_t>(); G.dst = R.cols[1].as<int32_t>(); G.w = R.tags();
  G.out_domain = out_ix.domain; G.in_domain = in_ix.domain;
  G.out_off = out_ix.off.as<uint32_t>(); G.in_off = in_ix.off.as<uint32_t>();
  G.s_dst = out_ix.other[0]; G.s_w = out_ix.tags;
  G.in_src = in_ix.other[0]; G.in_w = in_ix.tags;
  DevBuf ecnt(c, (size_t)R.n * 4), eoff(c, (size_t)R.n * 8);
  const unsigned tiles = (R.n + kScanTile - 1) / kScanTile;
  DevBuf sums(c, (size_t)tiles * 8);
  c->note_bytes = (int64_t)(R.n + S.n + T.n) * 12;
  XLOG_LAUNCH(c, k_tri_count_edges, kSMs * 8, 256, 0, G, ecnt.as<uint32_t>());
  XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint64_t>), tiles, kScanBlock, 0, (const uint32_t*)ecnt.as<uint32_t>(), (int64_t)R.n, sums.as<uint64_t>());
  XLOG_LAUNCH(c, (k_scan_spine<uint64_t>), 1, 1024, 0, sums.as<uint64_t>(), (int64_t)tiles, (uint64_t*)(c->d_ctrl + kSlotTotals));
  XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint64_t>), tiles, kScanBlock, 0, (const uint32_t*)ecnt.as<uint32_t>(), (int64_t)R.n,
              (const uint64_t*)sums.as<uint64_t>(), eoff.as<uint64_t>());
  sync_ctrl(c);                                            // the one small metadata read that sizes the output
  const uint64_t total = c->h_ctrl[kSlotTotals];
  if (total > kSortMaxN) fail(XLOG_ERR_CAPACITY_EXCEEDED, "materialised triangle relation exceeds 2^30 - 1 rows");
  c->r_candidates += (int64_t)total; c->r_unique += (int64_t)total;
  KeyTags kt;
  kt.n = (uint32_t)total;
  kt.keys = DevBuf(c, (size_t)std::max<uint64_t>(total, 1) * H.key_bytes);
  kt.tags = DevBuf(c, (size_t)std::max<uint64_t>(total, 1) * 4);
  c->note_bytes = (int64_t)total * (H.key_bytes + 4);
  DISPATCH_K(H.key_bytes, XLOG_LAUNCH(c, (k_tri_materialise<K>), kSMs * 8, 256, 0, G, times, (const uint64_t*)eoff.as<uint64_t>(), H.layout,
                                       kt.keys.as<K>(), kt.tags.as<float>()));
  set_current(H, std::move(kt));
}

// c4(x,y,z,w) :- r(x,y), s(y,z), t(z,w), u(w,x): the two-paths of r and s through the ordinary join, then either the
// multiway step (per two-path the intersection of t's out-list of z with u's in-list of x: count -> scan -> write; see
// cycle4.cuh) or the rest of the binary-join chain (every three-path written out, then a probe of u), as the skew test says.
void cycle4_materialise(Ctx* c, Relation& H, const RuleC& r) {
  Relation& R = *c->rels[r.plan.atoms[0].rel];
  Relation& S = *c->rels[r.plan.atoms[1].rel];
  Relation& T = *c->rels[r.plan.atoms[2].rel];
  Relation& U = *c->rels[r.plan.atoms[3].rel];
  if (H.n_facts) fail(XLOG_ERR_UNSUPPORTED, "a materialised four-cycle relation cannot also hold loaded facts");
  // empty inputs take the chain (nothing to intersect), as for the triangle
  const int empty_plan = (c->flags & XLOG_FLAG_FORCE_WCOJ) ? XLOG_PLAN_WCOJ : XLOG_PLAN_CHAIN;
  c->last_triangle_plan = empty_plan;
  if (R.n == 0 || S.n == 0 || T.n == 0 || U.n == 0) { KeyTags empty; set_current(H, std::move(empty)); return; }
  RuleC two;                                             // tmp(x,y,z) :- r(x,y), s(y,z)
  two.plan = r.plan;
  two.plan.n_atoms = 2;
  two.plan.n_head_cols = 3;
  two.kind = 2;
  two.shape[0] = join_shape(c, two.plan, 0);
  if (!two.shape[0].ok) fail(XLOG_ERR_INTERNAL, "four-cycle: no join path");
  Relation H2;
  H2.arity = 3; H2.sr = H.sr;
  H2.col_max[0] = R.val_max[0] ? R.val_max[0] : R.col_max[0]; H2.col_max[1] = R.val_max[1] ? R.val_max[1] : R.col_max[1];
  H2.col_max[2] = S.val_max[1] ? S.val_max[1] : S.col_max[1];
  H2.layout = make_layout(3, H2.col_max);
  H2.key_bytes = H2.layout.total_bits <= 32 ? 4 : 8;
  Variant v{&two, 0, full_source(R)};
  Counted q;
  count_variant(c, v, H2, q, kSlotTotals);
  sync_ctrl(c);
  q.total = c->h_ctrl[kSlotTotals];
  q.deg.reset(); q.sums.reset();
  const uint64_t n2 = q.total;
  const int ckb = H2.key_bytes;
  const size_t need = (size_t)n2 * (ckb + 4 + 12) + (16u << 20);
  if (n2 > kSortMaxN) fail(XLOG_ERR_CAPACITY_EXCEEDED, "four-cycle: more than 2^30 - 1 two-paths");
  if (need > c->arena.largest_free() / 2) fail(XLOG_ERR_RESOURCE_EXHAUSTED, "four-cycle: the two-paths do not fit the arena");
  c->r_candidates += (int64_t)n2;
  if (n2 == 0) { KeyTags empty; set_current(H, std::move(empty)); return; }
  c->last_triangle_plan = XLOG_PLAN_WCOJ;
  DevBuf k0(c, n2 * ckb), t0(c, n2 * 4);
  c->note_bytes = (int64_t)n2 * (ckb + 4 + 8);
  launch_expand<false>(c, q, 0, n2, ckb, k0.p, t0.as<float>(), BwdArgs{});
  q.start.reset(); q.rowinfo.reset();
  Index& tix = ensure_index(c, T, 0);
  Index& uix = ensure_index(c, U, 1);
  Cycle4 P{};
  P.L2 = H2.layout; P.L = H.layout;
  P.t_domain = tix.domain; P.t_off = tix.off.as<uint32_t>(); P.t_w = tix.other[0]; P.t_tag = tix.tags;
  P.u_domain = uix.domain; P.u_off = uix.off.as<uint32_t>(); P.u_w = uix.other[0]; P.u_tag = uix.tags;
  P.times = H.sr == XLOG_SR_SUMPROD ? 1 : 0;
  DevBuf cnt(c, n2 * 4), off(c, n2 * 8);
  const unsigned tiles = (unsigned)((n2 + kScanTile - 1) / kScanTile);
  DevBuf sums(c, (size_t)tiles * 8);
  zero_ctrl(c, kSlotTotals);
  const unsigned grid = (unsigned)std::min<uint64_t>((n2 + 255) / 256, (uint64_t)kSMs * 8);
  KeyTags kt;
  // skew test (as for the triangle): count the three-paths of r, s and t exactly, the chain's intermediate; the chain is taken
  // when they number at most kChainMaxBlowup per row of the largest input and fit the arena, the multiway plan otherwise
  if (!(c->flags & XLOG_FLAG_FORCE_WCOJ)) {
    int32_t mx3[kMaxArity] = {H2.col_max[0], H2.col_max[1], H2.col_max[2], T.val_max[1] ? T.val_max[1] : T.col_max[1]};
    const KeyLayout L3 = make_layout(4, mx3);
    const int kb3 = L3.total_bits <= 32 ? 4 : 8;
    Cycle4 P3 = P;
    P3.L = L3;
    DISPATCH_K(ckb, XLOG_LAUNCH(c, (k_c4_chain_count<K>), grid, 256, 0, P3, (const K*)k0.p, n2, cnt.as<uint32_t>()));
    XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint64_t>), tiles, kScanBlock, 0, (const uint32_t*)cnt.as<uint32_t>(), (int64_t)n2, sums.as<uint64_t>());
    XLOG_LAUNCH(c, (k_scan_spine<uint64_t>), 1, 1024, 0, sums.as<uint64_t>(), (int64_t)tiles, (uint64_t*)(c->d_ctrl + kSlotTotals));
    XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint64_t>), tiles, kScanBlock, 0, (const uint32_t*)cnt.as<uint32_t>(), (int64_t)n2,
                (const uint64_t*)sums.as<uint64_t>(), off.as<uint64_t>());
    sync_ctrl(c);
    const uint64_t n3 = c->h_ctrl[kSlotTotals];
    const uint64_t biggest = std::max<uint64_t>(std::max<uint64_t>(R.n, S.n), std::max<uint64_t>(T.n, U.n));
    const size_t need3 = (size_t)n3 * (kb3 + 4 + 12) + (16u << 20);
    const bool fits = L3.total_bits <= 64 && n3 <= kSortMaxN && need3 <= c->arena.largest_free() / 2;
    bool chain = fits && n3 <= kChainMaxBlowup * biggest;
    if (c->flags & XLOG_FLAG_FORCE_CHAIN) {
      if (!fits) fail(XLOG_ERR_RESOURCE_EXHAUSTED, "four-cycle chain: the three-path intermediate does not fit the arena");
      chain = true;
    }
    if (chain) {
      c->last_triangle_plan = XLOG_PLAN_CHAIN;
      c->r_candidates += (int64_t)n3;
      if (n3 == 0) { KeyTags empty; set_current(H, std::move(empty)); return; }
      DevBuf k3(c, n3 * kb3), t3(c, n3 * 4);
      c->note_bytes = (int64_t)n2 * (ckb + 4 + 8) + (int64_t)n3 * (kb3 + 4 + 8);
#define XLOG_C4_CHAIN(K2, K3) \
  XLOG_LAUNCH(c, (k_c4_chain_expand<K2, K3>), grid, 256, 0, P3, (const K2*)k0.p, (const float*)t0.as<float>(), n2, (const uint64_t*)off.as<uint64_t>(), k3.as<K3>(), t3.as<float>())
      if (ckb == 4 && kb3 == 4) XLOG_C4_CHAIN(uint32_t, uint32_t);
      else if (ckb == 4) XLOG_C4_CHAIN(uint32_t, uint64_t);
      else if (kb3 == 4) XLOG_C4_CHAIN(uint64_t, uint32_t);
      else XLOG_C4_CHAIN(uint64_t, uint64_t);
#undef XLOG_C4_CHAIN
      k0.reset(); t0.reset(); cnt.reset(); off.reset(); sums.reset();
      // probe u with (w, x)
      Index& ux = ensure_index(c, U, 0);
      ChainProbe Q{};
      Q.last = 3;
      Q.L = L3; Q.out = H.layout;
      Q.t_domain = ux.domain; Q.t_off = ux.off.as<uint32_t>(); Q.t_col1 = ux.other[0]; Q.t_w = ux.tags; Q.times = P.times;
      DevBuf hit(c, n3 * 4), hoff(c, n3 * 8);
      const unsigned tiles3 = (unsigned)((n3 + kScanTile - 1) / kScanTile);
      DevBuf sums3(c, (size_t)tiles3 * 8);
      zero_ctrl(c, kSlotTotals);
      c->note_bytes = (int64_t)n3 * (kb3 + 4);
      DISPATCH_K(kb3, XLOG_LAUNCH(c, (k_chain_probe_count<K>), grid_for(n3, 256), 256, 0, Q, (const K*)k3.p, n3, hit.as<uint32_t>()));
      XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint64_t>), tiles3, kScanBlock, 0, (const uint32_t*)hit.as<uint32_t>(), (int64_t)n3, sums3.as<uint64_t>());
      XLOG_LAUNCH(c, (k_scan_spine<uint64_t>), 1, 1024, 0, sums3.as<uint64_t>(), (int64_t)tiles3, (uint64_t*)(c->d_ctrl + kSlotTotals));
      XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint64_t>), tiles3, kScanBlock, 0, (const uint32_t*)hit.as<uint32_t>(), (int64_t)n3,
                  (const uint64_t*)sums3.as<uint64_t>(), hoff.as<uint64_t>());
      sync_ctrl(c);
      const uint64_t total = c->h_ctrl[kSlotTotals];
      if (total > kSortMaxN) fail(XLOG_ERR_CAPACITY_EXCEEDED, "materialised four-cycle relation exceeds 2^30 - 1 rows");
      c->r_unique += (int64_t)total;
      kt.n = (uint32_t)total;
      kt.keys = DevBuf(c, (size_t)std::max<uint64_t>(total, 1) * H.key_bytes);
      kt.tags = DevBuf(c, (size_t)std::max<uint64_t>(total, 1) * 4);
      c->note_bytes = (int64_t)n3 * (kb3 + 4 + 12) + (int64_t)total * (H.key_bytes + 4);
#define XLOG_C4_EMIT(K3, KH) \
  XLOG_LAUNCH(c, (k_chain_probe_emit<K3, KH>), grid_for(n3, 256), 256, 0, Q, (const K3*)k3.p, (const float*)t3.as<float>(), n3, \
              (const uint32_t*)hit.as<uint32_t>(), (const uint64_t*)hoff.as<uint64_t>(), kt.keys.as<KH>(), kt.tags.as<float>())
      if (kb3 == 4 && H.key_bytes == 4) XLOG_C4_EMIT(uint32_t, uint32_t);
      else if (kb3 == 4) XLOG_C4_EMIT(uint32_t, uint64_t);
      else if (H.key_bytes == 4) XLOG_C4_EMIT(uint64_t, uint32_t);
      else XLOG_C4_EMIT(uint64_t, uint64_t);
#undef XLOG_C4_EMIT
      set_current(H, std::move(kt));
      return;
    }
    zero_ctrl(c, kSlotTotals);
  }
  // long runs of equal x and small w values: the bitmap kernel (see cycle4.cuh)
  const uint64_t w_max = (uint64_t)(U.val_max[0] ? U.val_max[0] : U.col_max[0]);
  const uint64_t x_values = std::min<uint64_t>(R.n, (uint64_t)(R.val_max[0] ? R.val_max[0] : R.col_max[0]) + 1);
  const bool bitmap = w_max < (uint64_t)kC4BmWords * 32 && n2 >= 16 * x_values;
  const unsigned bgrid = (unsigned)std::min<uint64_t>((n2 + kC4Chunk - 1) / kC4Chunk, (uint64_t)kSMs * 6);
#define XLOG_C4(K2, KH, EMIT, KEYS, TAGS)                                                                                          \
  do {                                                                                                                             \
    if (bitmap) {                                                                                                                  \
      XLOG_CUDA(cudaFuncSetAttribute(k_cycle4_bitmap<K2, KH, EMIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kC4BmSmem));   \
      XLOG_LAUNCH(c, (k_cycle4_bitmap<K2, KH, EMIT>), bgrid, 256, kC4BmSmem, P, (const K2*)k0.p, (const float*)t0.as<float>(), n2,         \
                  cnt.as<uint32_t>(), (const uint64_t*)off.as<uint64_t>(), (KH*)(KEYS), (float*)(TAGS));                           \
    } else                                                                                                                         \
      XLOG_LAUNCH(c, (k_cycle4<K2, KH, EMIT>), grid, 256, 0, P, (const K2*)k0.p, (const float*)t0.as<float>(), n2,                 \
                  cnt.as<uint32_t>(), (const uint64_t*)off.as<uint64_t>(), (KH*)(KEYS), (float*)(TAGS));                           \
  } while (0)
#define XLOG_C4_DISPATCH(EMIT, KEYS, TAGS)                                        \
  do {                                                                            \
    if (ckb == 4 && H.key_bytes == 4) XLOG_C4(uint32_t, uint32_t, EMIT, KEYS, TAGS); \
    else if (ckb == 4) XLOG_C4(uint32_t, uint64_t, EMIT, KEYS, TAGS);             \
    else if (H.key_bytes == 4) XLOG_C4(uint64_t, uint32_t, EMIT, KEYS, TAGS);     \
    else XLOG_C4(uint64_t, uint64_t, EMIT, KEYS, TAGS);                           \
  } while (0)
  c->note_bytes = (int64_t)n2 * (ckb + 4) + (int64_t)(T.n + U.n) * 4;
  XLOG_C4_DISPATCH(false, nullptr, nullptr);
  XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint64_t>), tiles, kScanBlock, 0, (const uint32_t*)cnt.as<uint32_t>(), (int64_t)n2, sums.as<uint64_t>());
  XLOG_LAUNCH(c, (k_scan_spine<uint64_t>), 1, 1024, 0, sums.as<uint64_t>(), (int64_t)tiles, (uint64_t*)(c->d_ctrl + kSlotTotals));
  XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint64_t>), tiles, kScanBlock, 0, (const uint32_t*)cnt.as<uint32_t>(), (int64_t)n2,
              (const uint64_t*)sums.as<uint64_t>(), off.as<uint64_t>());
  sync_ctrl(c);                                            // the one small metadata read that sizes the output
  const uint64_t total = c->h_ctrl[kSlotTotals];
  if (total > kSortMaxN) fail(XLOG_ERR_CAPACITY_EXCEEDED, "materialised four-cycle relation exceeds 2^30 - 1 rows");
  c->r_unique += (int64_t)total;
  kt.n = (uint32_t)total;
  kt.keys = DevBuf(c, (size_t)std::max<uint64_t>(total, 1) * H.key_bytes);
  kt.tags = DevBuf(c, (size_t)std::max<uint64_t>(total, 1) * 4);
  c->note_bytes = (int64_t)n2 * (ckb + 4 + 8) + (int64_t)(T.n + U.n) * 8 + (int64_t)total * (H.key_bytes + 4);
  XLOG_C4_DISPATCH(true, kt.keys.p, kt.tags.p);
#undef XLOG_C4_DISPATCH
#undef XLOG_C4
  set_current(H, std::move(kt));
}

void triangle_aggregate(Ctx* c, Relation& H, const RuleC& r) {
  if (c->rels[r.plan.atoms[0].rel]->is_head && r.plan.atoms[0].rel == r.plan.head_rel) fail(XLOG_ERR_UNSUPPORTED, "recursive triangle rule");
  switch (H.sr) {
    case XLOG_SR_MAXPLUS: triangle_aggregate_t<OpMax>(c, H, r); break;
    case XLOG_SR_MINPLUS: triangle_aggregate_t<OpMin>(c, H, r); break;
    case XLOG_SR_LOGSUMEXP: triangle_aggregate_t<OpLse>(c, H, r); break;
    default: triangle_aggregate_t<OpSum>(c, H, r); break;
  }
}

}  // namespace
}  // namespace xlog
