// Recursive components over a tag mirror, building blocks: when the mirror applies, resident rounds (CUDA graph with a WHILE node),
// grouped and bitmap-driven joins.  The strata themselves are in host_mirror_strata.cuh.
// Host-side driver code of the engine; included by xlog_api.cu only (one translation unit).
#pragma once
#include "host_eval.cuh"
#include "bitmap_join.cuh"
#include "dense_closure.cuh"
#include "group_join.cuh"
#include "mirror.cuh"
#include "resident.cuh"

namespace xlog {
namespace {

constexpr int kSlotMirNew = 12, kSlotMirChanged = 13;
constexpr int kMirrorMaxBits = 30;

// The tag mirror serves a component of one max/min relation whose rules are all linear (at most one atom over the
// relation itself, and that atom is the scanned side): then the relation is only ever read through its delta, and
// its sorted form is needed again only after the last round.
// Path doubling  h(x,z) :- h(x,y), h(y,z)  (dense_closure.cuh): the one rule shape with two atoms over the relation that a
// tag mirror serves, because both of its delta variants can read the looked-up side from the mirror itself.  It must be
// the only rule with atoms over h, h binary without dictionaries, and a row of the matrix must fit shared memory.
constexpr int kDenseMaxColumnBits = 12;
constexpr int kSlotDense = 90;             // candidate counter of the dense path-doubling rounds

bool is_doubling_rule(Ctx* c, int h, const RuleC* r) {
  const xlog_plan& p = r->plan;
  if (r->kind != 2 || p.n_atoms != 2 || p.atoms[0].rel != h || p.atoms[1].rel != h || p.atoms[0].negated || p.atoms[1].negated) return false;
  const xlog_arg* a = p.atoms[0].args; const xlog_arg* b = p.atoms[1].args;
  if (!is_plain_var(a[0]) || !is_plain_var(a[1]) || !is_plain_var(b[0]) || !is_plain_var(b[1])) return false;
  const int x = a[0].var, y = a[1].var, z = b[1].var;
  if (b[0].var != y || x == y || y == z || x == z || p.n_head_cols != 2 || p.emit_count_column) return false;
  const int hv[2] = {x, z};
  for (int col = 0; col < 2; ++col) {
    if (p.head[col].c0 != 0) return false;
    for (int v = 0; v < XLOG_MAX_VARS; ++v) if (p.head[col].coef[v] != (v == hv[col] ? 1 : 0)) return false;
  }
  return true;
}
const RuleC* doubling_rule_of(Ctx* c, int h, const std::vector<const RuleC*>& rs) {
  if (c->flags & XLOG_FLAG_NO_DENSE_DOUBLING) return nullptr;
  const Relation& H = *c->rels[h];
  if (H.arity != 2 || H.dict_n[0] || H.dict_n[1] || H.layout.shift[1] != 0) return nullptr;
  if (H.layout.shift[0] > kDenseMaxColumnBits) return nullptr;             // shift of column 0 = bits of column 1 = log2 of the row length
  const RuleC* found = nullptr;
  for (const RuleC* r : rs) {
    int in = 0;
    for (int j = 0; j < r->plan.n_atoms; ++j) if (r->plan.atoms[j].rel == h) ++in;
    if (in == 0) continue;
    if (found || !is_doubling_rule(c, h, r)) return nullptr;
    found = r;
  }
  return found;
}

bool mirror_applies(Ctx* c, const std::vector<int>& comp, const std::vector<const RuleC*>& rs) {
  if ((c->flags & XLOG_FLAG_NO_TAG_MIRROR) || comp.size() != 1) return false;
  const Relation& H = *c->rels[comp[0]];
  if (H.sr != XLOG_SR_MAXPLUS && H.sr != XLOG_SR_MINPLUS) return false;
  if (H.layout.total_bits > kMirrorMaxBits || H.key_bytes != 4) return false;
  for (const RuleC* r : rs) {
    if (r->plan.emit_count_column || r->kind == 3 || r->kind == 4 || r->kind == 6) return false;
    int in = 0, pos = 0;
    for (int j = 0; j < r->plan.n_atoms; ++j)
      if (r->plan.atoms[j].rel == comp[0]) { if (r->plan.atoms[j].negated) return false; ++in; pos = j; }
    if (in > 1 && !(c->rels[comp[0]]->layout.total_bits <= kMirrorMaxBits && doubling_rule_of(c, comp[0], rs) == r)) return false;
    if (in == 1 && r->kind == 2 && !r->shape[pos].ok) return false;
    if (in == 1 && r->kind != 2 && pos != 0) return false;
    if (in == 0 && r->kind == 2 && !r->shape[0].ok && !r->shape[1].ok) return false;
  }
  uint64_t need = ((uint64_t)4 << H.layout.total_bits) + ((uint64_t)1 << H.layout.total_bits) / 4 + (1u << 20);
  if (doubling_rule_of(c, comp[0], rs)) need += (uint64_t)4 << H.layout.total_bits;       // the snapshot of the matrix
  return need <= c->arena.largest_free() / 2;
}

// ---- resident rounds (resident.cuh) --------------------------------------------------------------------
constexpr int kResidentMaxBits = 24;
constexpr uint32_t kResidentMaxTiles = 1u << 20;

ResState* res_state(Ctx* c) { return reinterpret_cast<ResState*>(c->d_ctrl + kSlotResState); }
static_assert(sizeof(ResState) <= (kCtrlSlots - kSlotResState) * sizeof(uint64_t), "state block must fit the control words");

// The persistent buffers of head relation h at their fixed capacities, or nullptr when the resident rounds do not
// apply (domain too large for fixed-capacity buffers, not enough arena, or switched off).
Resident* resident_for(Ctx* c, int h, int bits, uint64_t slots, uint32_t bm_quads, unsigned ch_tiles) {
  if ((c->flags & XLOG_FLAG_NO_RESIDENT_LOOP) || bits > kResidentMaxBits) { c->resident.erase(h); return nullptr; }
  uint32_t max_tiles = kResidentMaxTiles;
  if (c->chunk_bytes) max_tiles = (uint32_t)std::max<uint64_t>(1, std::min<uint64_t>(max_tiles, c->chunk_bytes / 16 / kExpTileMirror));
  auto it = c->resident.find(h);
  if (it != c->resident.end() && it->second->slots == slots && it->second->max_tiles == max_tiles) return it->second.get();
  c->resident.erase(h);
  const uint64_t dom = (uint64_t)1 << bits;
  const uint64_t need = slots * 4 + (uint64_t)bm_quads * 32 + dom * 32 + (uint64_t)max_tiles * 8 + (4u << 20);
  if (need > c->arena.largest_free() / 3) return nullptr;
  std::unique_ptr<Resident> R(new Resident());
  R->slots = slots; R->max_tiles = max_tiles;
  R->table = DevBuf(c, slots * 4);
  R->bitmap = DevBuf(c, (size_t)bm_quads * 16);
  R->present = DevBuf(c, (size_t)bm_quads * 16);
  R->ch_sums = DevBuf(c, (size_t)ch_tiles * 4);
  R->dkeys = DevBuf(c, dom * 4); R->dtags = DevBuf(c, dom * 4);
  R->rowinfo = DevBuf(c, dom * 16); R->start = DevBuf(c, dom * 8);
  R->scan_tiles_cap = (uint32_t)(dom / kResScanTile + 2);
  R->scan_status = DevBuf(c, (size_t)kResMaxVariants * R->scan_tiles_cap * 8);
  R->tickets = DevBuf(c, kResTickets * 4);
  R->tile_rows = DevBuf(c, (size_t)max_tiles * 8);
  Resident* out = R.get();
  c->resident[h] = std::move(R);
  return out;
}

// bitmap tiles: one sweep of 256 words per tile for domains up to 2^22 keys (so that small domains still give hundreds of
// blocks), four sweeps above that
int mirror_sweeps(uint32_t nwords) { return nwords <= (1u << 17) ? 1 : 4; }
unsigned mirror_tiles(uint32_t nwords) { const uint32_t per = kMirBlock * mirror_sweeps(nwords); return (nwords + per - 1) / per; }
void launch_changed_count(Ctx* c, const uint32_t* words, uint32_t* present, uint32_t nwords, unsigned tiles, uint32_t* sums, unsigned long long* new_total) {
  if (mirror_sweeps(nwords) == 1) XLOG_LAUNCH(c, (k_mirror_changed_count<1>), tiles, kMirBlock, 0, words, present, nwords, sums, new_total);
  else XLOG_LAUNCH(c, (k_mirror_changed_count<4>), tiles, kMirBlock, 0, words, present, nwords, sums, new_total);
}
void launch_changed_emit(Ctx* c, uint32_t* words, uint32_t nwords, unsigned tiles, const uint32_t* base, const int32_t* table, uint32_t* keys,
                         float* tags, const uint32_t* skip) {
  if (mirror_sweeps(nwords) == 1) XLOG_LAUNCH(c, (k_mirror_changed_emit<uint32_t, 1>), tiles, kMirBlock, 0, words, nwords, base, table, keys, tags, skip);
  else XLOG_LAUNCH(c, (k_mirror_changed_emit<uint32_t, 4>), tiles, kMirBlock, 0, words, nwords, base, table, keys, tags, skip);
}

template <typename T> void sig_add(std::vector<char>& sig, const T& v) {
  const char* p = reinterpret_cast<const char*>(&v);
  sig.insert(sig.end(), p, p + sizeof(T));
}

// Count, scan and partition of rule v over the current delta (resident.cuh).
void resident_count(Ctx* c, Resident& R, const JoinSpec& S, size_t v) {
  XLOG_LAUNCH(c, (k_res_count_scan<uint32_t>), kSMs * 4, kScanBlock, 0, S, (const uint32_t*)R.dkeys.as<uint32_t>(), (const float*)R.dtags.as<float>(), res_state(c),
              R.rowinfo.as<uint4>(), R.start.as<uint64_t>(), R.tile_rows.as<uint2>(), R.scan_status.as<unsigned long long>() + v * R.scan_tiles_cap,
              R.tickets.as<uint32_t>() + v, ctrl_u32(c, kSlotErr), c->spin_limit);
}

// One round's launches.  Nothing here allocates, copies or waits: the same calls are either captured into the WHILE
// body or issued directly (host-driven rounds, used when launches are being timed one by one).
void resident_body(Ctx* c, Resident& R, const std::vector<JoinSpec>& specs, bool is_max, const MirrorArgs& mr, uint32_t bm_quads, unsigned ch_tiles,
                   cudaGraphConditionalHandle handle, int use_handle) {
  ResState* st = res_state(c);
  uint32_t* err = ctrl_u32(c, kSlotErr);
  const uint32_t* dk = R.dkeys.as<uint32_t>();
  const ResScratch sc{R.scan_status.as<unsigned long long>(), R.scan_tiles_cap, R.tickets.as<uint32_t>()};
  const bool fused = specs.size() == 1;                  // the count of the next round rides on the emit kernel; the first round's is launched before the loop
  for (size_t v = 0; v < specs.size(); ++v) {
    const JoinSpec& S = specs[v];
    if (!fused) resident_count(c, R, S, v);
// four waves of blocks: the hardware hands a new block to whichever SM finishes first, which evens out skewed tiles
#define XLOG_RES_EXPAND(MODE, SINK)                                                                                                         \
  XLOG_LAUNCH(c, (k_res_expand<uint32_t, MODE, SINK>), kSMs * kExpMirrorBlocksPerSM * 4, kExpBlock, 0, S, dk, (const ResState*)st, (const uint64_t*)R.start.as<uint64_t>(), \
              (const uint4*)R.rowinfo.as<uint4>(), (const uint2*)R.tile_rows.as<uint2>(), err, mr)
    if (S.fast) { if (is_max) XLOG_RES_EXPAND(kExpFast, kSinkMax); else XLOG_RES_EXPAND(kExpFast, kSinkMin); }
    else { if (is_max) XLOG_RES_EXPAND(kExpGeneric, kSinkMax); else XLOG_RES_EXPAND(kExpGeneric, kSinkMin); }
#undef XLOG_RES_EXPAND
  }
  uint32_t* ctr = sc.tickets + kResTkEmit;
  if (fused) {
#define XLOG_RES_EMIT_COUNT(SW)                                                                                                            \
  XLOG_LAUNCH(c, (k_res_emit_count<SW>), (bm_quads * 4 + kResEcWords * SW - 1) / (kResEcWords * SW), kMirBlock, 0, R.bitmap.as<uint32_t>(), R.present.as<uint32_t>(), bm_quads * 4, mr.n_new,  \
              (const int32_t*)R.table.as<int32_t>(), R.dkeys.as<uint32_t>(), R.dtags.as<float>(), st, sc, (const unsigned long long*)mr.n_new, \
              ctr, handle, use_handle, specs[0], R.rowinfo.as<uint4>(), R.start.as<uint64_t>(), R.tile_rows.as<uint2>(), err)
    if (mirror_sweeps(bm_quads * 4) == 1) XLOG_RES_EMIT_COUNT(1); else XLOG_RES_EMIT_COUNT(4);
#undef XLOG_RES_EMIT_COUNT
    return;
  }
#define XLOG_RES_EMIT(SW)                                                                                                                  \
  XLOG_LAUNCH(c, (k_res_emit<SW>), ch_tiles, kMirBlock, 0, R.bitmap.as<uint32_t>(), R.present.as<uint32_t>(), bm_quads * 4, mr.n_new,        \
              (const int32_t*)R.table.as<int32_t>(),                                                                                        \
              R.dkeys.as<uint32_t>(), R.dtags.as<float>(), st, sc, (uint32_t)specs.size(), (const unsigned long long*)mr.n_new, ctr, handle, use_handle)
  if (mirror_sweeps(bm_quads * 4) == 1) XLOG_RES_EMIT(1); else XLOG_RES_EMIT(4);
#undef XLOG_RES_EMIT
}

// Run rounds on the device until the delta is empty, the round budget is used up or a round needs more tiles than
// planned.  Returns the final state block (read once, after the loop).
ResState run_resident(Ctx* c, Resident& R, int h, const std::vector<const RuleC*>& rs, bool is_max, const MirrorArgs& mr_host, uint32_t bm_quads,
                      unsigned ch_tiles, uint32_t n_delta, int64_t rounds_left, uint64_t new_seen) {
  Relation& H = *c->rels[h];
  std::vector<JoinSpec> specs;
  for (const RuleC* r : rs)
    for (int j = 0; j < r->plan.n_atoms; ++j)
      if (r->plan.atoms[j].rel == h) {
        const Variant v{r, j, Source{R.dkeys.p, R.dtags.as<float>(), n_delta, H.layout, H.key_bytes}};
        specs.push_back(make_spec(c, v, H));              // builds the looked-up relation's index if it is missing
      }
  if (specs.size() > 16) fail(XLOG_ERR_UNSUPPORTED, "too many rule variants for one head");
  const uint32_t budget = (uint32_t)std::min<int64_t>(rounds_left, 0x7fffffff);
  const ResScratch sc{R.scan_status.as<unsigned long long>(), R.scan_tiles_cap, R.tickets.as<uint32_t>()};
  XLOG_LAUNCH(c, k_res_init, 1, 1024, 0, res_state(c), sc, (uint32_t)specs.size(), n_delta, budget, R.max_tiles, (unsigned long long)new_seen);
  const MirrorArgs& mr = mr_host;
  const bool fused = specs.size() == 1;
  if (fused) resident_count(c, R, specs[0], 0);          // the first round's count; every later one rides on the emit kernel
  const int64_t l0 = c->launches;
  const bool use_graph = !(c->flags & (XLOG_FLAG_PROFILE | XLOG_FLAG_NO_GRAPH));
  ResState out{};
  auto read_state = [&]() {
    sync_ctrl(c);
    memcpy(&out, c->h_ctrl + kSlotResState, sizeof out);
  };
  if (use_graph) {
    std::vector<char> sig;
    for (const JoinSpec& S : specs) sig_add(sig, S);
    sig_add(sig, mr.table); sig_add(sig, mr.changed); sig_add(sig, mr.n_new); sig_add(sig, mr.key_max); sig_add(sig, mr.err); sig_add(sig, R.present.p);
    sig_add(sig, is_max); sig_add(sig, bm_quads); sig_add(sig, ch_tiles); sig_add(sig, c->d_ctrl); sig_add(sig, c->spin_limit);
    if (!R.exec || sig != R.sig) {
      if (R.exec) { cudaGraphExecDestroy(R.exec); R.exec = nullptr; }
      if (R.graph) { cudaGraphDestroy(R.graph); R.graph = nullptr; }
      XLOG_CUDA(cudaGraphCreate(&R.graph, 0));
      cudaGraphConditionalHandle handle;
      XLOG_CUDA(cudaGraphConditionalHandleCreate(&handle, R.graph, 1, cudaGraphCondAssignDefault));
      cudaGraphNodeParams np = {};
      np.type = cudaGraphNodeTypeConditional;
      np.conditional.handle = handle;
      np.conditional.type = cudaGraphCondTypeWhile;
      np.conditional.size = 1;
      cudaGraphNode_t node;
      XLOG_CUDA(cudaGraphAddNode(&node, R.graph, nullptr, 0, &np));
      cudaGraph_t body = np.conditional.phGraph_out[0];
      // the body is recorded on a stream of the context's own (the caller's stream may be the legacy default stream,
      // which cannot capture); the instantiated graph is launched on the caller's stream like everything else
      if (!c->capture_stream) XLOG_CUDA(cudaStreamCreateWithFlags(&c->capture_stream, cudaStreamNonBlocking));
      XLOG_CUDA(cudaStreamBeginCaptureToGraph(c->capture_stream, body, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal));
      cudaStream_t caller = c->stream;
      c->stream = c->capture_stream;
      const int64_t b0 = c->launches;
      try {
        resident_body(c, R, specs, is_max, mr, bm_quads, ch_tiles, handle, 1);
      } catch (...) {
        c->stream = caller;
        cudaGraph_t dummy = nullptr;
        cudaStreamEndCapture(c->capture_stream, &dummy);
        throw;
      }
      c->stream = caller;
      R.body_launches = c->launches - b0;
      XLOG_CUDA(cudaStreamEndCapture(c->capture_stream, nullptr));
      XLOG_CUDA(cudaGraphInstantiate(&R.exec, R.graph, 0));
      R.sig = std::move(sig);
    }
    XLOG_CUDA(cudaGraphLaunch(R.exec, c->stream));
    read_state();
    c->launches = l0 + R.body_launches * (int64_t)out.rounds + (out.status == kResOverflow && !fused ? R.body_launches : 0);
  } else {
    unsigned long long seen = 0;
    uint32_t rows = n_delta;
    double expand_ms_seen = 0.0;
    int64_t expand_launches_seen = 0;
    {
      auto it0 = c->prof_index.find("k_res_expand");
      if (it0 != c->prof_index.end()) { expand_ms_seen = c->prof[it0->second].ms; expand_launches_seen = c->prof[it0->second].launches; }
    }
    for (;;) {
      resident_body(c, R, specs, is_max, mr, bm_quads, ch_tiles, cudaGraphConditionalHandle{}, 0);
      read_state();
      if (c->flags & XLOG_FLAG_PROFILE) {
        // per delta row and rule: key and tag read, two offsets probed, 16-byte row record and 8-byte start offset written
        auto cs = c->prof_index.find(fused ? "k_res_emit_count" : "k_res_count_scan");
        if (cs != c->prof_index.end()) c->prof[cs->second].bytes += (int64_t)(fused ? out.n_delta : rows) * 40 * (int64_t)specs.size() + (fused ? (int64_t)bm_quads * 16 : 0);
        rows = out.n_delta;
        // algorithmic bytes of the round's expand launches (per candidate: the looked-up columns and tag, and the slot)
        auto it = c->prof_index.find("k_res_expand");
        if (it != c->prof_index.end()) {
          const int64_t bytes = (int64_t)(out.candidates - seen) * (4 + (specs[0].has_inner ? 4 * (specs[0].inner_free + 1) : 0));
          Ctx::ProfEntry& pe = c->prof[it->second];
          pe.bytes += bytes;
          if (bytes >= kProfLargeBytes) {                // this round's launches, totalled on their own like any large launch
            const double round_ms = pe.ms - expand_ms_seen;
            const int64_t round_launches = pe.launches - expand_launches_seen;
            auto bt = c->prof_index.find("k_res_expand (large)");
            if (bt == c->prof_index.end()) {
              bt = c->prof_index.emplace("k_res_expand (large)", (int)c->prof.size()).first;
              c->prof.push_back(Ctx::ProfEntry{"k_res_expand (large)", 0, 0.0, 0});
            }
            Ctx::ProfEntry& be = c->prof[bt->second];
            be.ms += round_ms; be.launches += round_launches; be.bytes += bytes;
          }
          expand_ms_seen = c->prof[it->second].ms; expand_launches_seen = c->prof[it->second].launches;
        }
        seen = out.candidates;
      }
      if (out.status != kResOk || out.n_delta == 0) break;
    }
  }
  return out;
}

// ---- grouped join (group_join.cuh) -----------------------------------------------------------------------
// The shape  h(a, c) :- h(a, b), r(b, c)  for every rule over h (binary h; a and b bare variables; c the looked-up
// relation's other column).
bool grouped_shape(Ctx* c, int h, const std::vector<const RuleC*>& rs) {
  const Relation& H = *c->rels[h];
  if (H.arity != 2) return false;
  bool any = false;
  for (const RuleC* r : rs) {
    int j = -1;
    for (int k = 0; k < r->plan.n_atoms; ++k) if (r->plan.atoms[k].rel == h) j = k;
    if (j < 0) continue;
    if (r->kind != 2 || !r->shape[j].ok) return false;
    const xlog_plan& p = r->plan;
    const xlog_atom& A = p.atoms[j];
    const xlog_atom& B = p.atoms[1 - j];
    if (!is_plain_var(A.args[0]) || !is_plain_var(A.args[1]) || A.args[0].var == A.args[1].var) return false;
    if (c->rels[B.rel]->arity != 2 || r->shape[j].probe_col != 0 || r->shape[j].probe_var != A.args[1].var || r->shape[j].probe_mul != 1 ||
        r->shape[j].probe_add != 0 || !is_plain_var(B.args[1]))
      return false;
    const int hv[2] = {A.args[0].var, B.args[1].var};
    for (int col = 0; col < 2; ++col) {
      if (p.head[col].c0 != 0) return false;
      for (int v = 0; v < XLOG_MAX_VARS; ++v) if (p.head[col].coef[v] != (v == hv[col] ? 1 : 0)) return false;
    }
    any = true;
  }
  return any;
}

constexpr int kSlotSeg = 80;               // grouped join: segments, candidates, work items, neighbour rows read

// One delta variant through the grouped join.  Returns the candidate total, or UINT64_MAX when the compiled rule turns
// out not to have the linear-key form (the caller then takes the row-wise join).
uint64_t grouped_apply(Ctx* c, const Variant& v, const Relation& H, const KeyLayout& M, int carried_bits, bool is_max, const MirrorArgs& mr) {
  const JoinSpec S = make_spec(c, v, H, &M);
  if (!S.fast || !S.has_inner || S.inner_free != 1 || v.outer.key_bytes != 4) return UINT64_MAX;
  const uint32_t n = v.outer.n;
  const unsigned tiles = (n + kScanTile - 1) / kScanTile;
  DevBuf deg(c, (size_t)n * 4), rowinfo(c, (size_t)n * 16), flags(c, (size_t)n * 4), idx(c, (size_t)n * 4), sums(c, (size_t)tiles * 4);
  zero_ctrl(c, kSlotSeg, 4);
  XLOG_LAUNCH(c, (k_join_count_flags<uint32_t>), grid_for(n, 256, kSMs * 32), 256, 0, S, (const uint32_t*)v.outer.keys, v.outer.tags, n, carried_bits, deg.as<uint32_t>(),
              rowinfo.as<uint4>(), flags.as<uint32_t>(), (unsigned long long*)(c->d_ctrl + kSlotSeg + 1), ctrl_u32(c, kSlotErr));
  XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint32_t>), tiles, kScanBlock, 0, (const uint32_t*)flags.as<uint32_t>(), (int64_t)n, sums.as<uint32_t>());
  XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, sums.as<uint32_t>(), (int64_t)tiles, ctrl_u32(c, kSlotSeg));
  XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint32_t>), tiles, kScanBlock, 0, (const uint32_t*)flags.as<uint32_t>(), (int64_t)n,
              (const uint32_t*)sums.as<uint32_t>(), idx.as<uint32_t>());
  sync_ctrl(c);
  const uint32_t n_seg = (uint32_t)c->h_ctrl[kSlotSeg];
  const uint64_t total = c->h_ctrl[kSlotSeg + 1];
  if (total == 0) return 0;
  if (total / n_seg < 128) return UINT64_MAX;            // small segments: the row-wise join does as well, with fewer passes
  const uint32_t ns1 = n_seg + 1;
  DevBuf seg_first(c, (size_t)ns1 * 4);
  XLOG_LAUNCH(c, k_seg_first, grid_for((uint64_t)n + 1, 256), 256, 0, (const uint32_t*)flags.as<uint32_t>(), (const uint32_t*)idx.as<uint32_t>(), n, n_seg,
              seg_first.as<uint32_t>());
  flags.reset(); idx.reset(); sums.reset();
  const unsigned ittiles = (ns1 + kScanTile - 1) / kScanTile;
  DevBuf items(c, (size_t)ns1 * 4), item_off(c, (size_t)ns1 * 4), itsums(c, (size_t)ittiles * 4);
  XLOG_LAUNCH(c, k_seg_items, grid_for(ns1, 256, kSMs * 16), 256, 0, (const uint32_t*)seg_first.as<uint32_t>(), n_seg, (const uint32_t*)deg.as<uint32_t>(), items.as<uint32_t>(),
              (unsigned long long*)(c->d_ctrl + kSlotSeg + 3));
  XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint32_t>), ittiles, kScanBlock, 0, (const uint32_t*)items.as<uint32_t>(), (int64_t)ns1, itsums.as<uint32_t>());
  XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, itsums.as<uint32_t>(), (int64_t)ittiles, ctrl_u32(c, kSlotSeg + 2));
  XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint32_t>), ittiles, kScanBlock, 0, (const uint32_t*)items.as<uint32_t>(), (int64_t)ns1,
              (const uint32_t*)itsums.as<uint32_t>(), item_off.as<uint32_t>());
  sync_ctrl(c);
  const uint32_t n_items = (uint32_t)c->h_ctrl[kSlotSeg + 2];
  items.reset(); itsums.reset();
  DevBuf item_seg(c, (size_t)std::max(n_items, 1u) * 4);
  XLOG_LAUNCH(c, k_seg_item_fill, grid_for(n_seg, 256), 256, 0, n_seg, (const uint32_t*)item_off.as<uint32_t>(), item_seg.as<uint32_t>());
  // per candidate: its slot; per segment and neighbour: the looked-up column and tag, read once for all the segment's rows;
  // per delta row: its count record
  c->note_bytes = (int64_t)total * 4 + (int64_t)c->h_ctrl[kSlotSeg + 3] * 8 + (int64_t)n * 16;
  const unsigned grid = (unsigned)std::min<uint64_t>(((uint64_t)n_items + 7) / 8, (uint64_t)kSMs * 8 * 16);
  if (is_max)
    XLOG_LAUNCH(c, (k_seg_expand<kSinkMax>), grid, 256, 0, S, n_items, (const uint32_t*)item_off.as<uint32_t>(), (const uint32_t*)item_seg.as<uint32_t>(),
                (const uint32_t*)seg_first.as<uint32_t>(), (const uint32_t*)deg.as<uint32_t>(), (const uint4*)rowinfo.as<uint4>(), mr);
  else
    XLOG_LAUNCH(c, (k_seg_expand<kSinkMin>), grid, 256, 0, S, n_items, (const uint32_t*)item_off.as<uint32_t>(), (const uint32_t*)item_seg.as<uint32_t>(),
                (const uint32_t*)seg_first.as<uint32_t>(), (const uint32_t*)deg.as<uint32_t>(), (const uint4*)rowinfo.as<uint4>(), mr);
  return total;
}

constexpr int kSlotBm = 84;                // bitmap-driven grouped join: the kBmTotals counters of k_bm_plan
static_assert(kSlotBm + kBmTotals <= kCtrlSlots, "control block too small");

// What the bitmap-driven grouped join (bitmap_join.cuh) needs beyond the mirror itself; valid == false: not applicable.
struct BitmapJoin {
  bool valid = false;
  JoinSpec spec;
  DevBuf pairs, items;
  int carried_bits = 0;
};

// Applicable when exactly one rule has an atom over h (so a round is one join), that rule has the grouped shape with the
// linear-key form, a value of the probed column owns 1 to 32 whole bitmap words, and the pair list and the item list
// (sized for every key changing in one round) fit the arena.
void bitmap_join_setup(Ctx* c, int h, const std::vector<const RuleC*>& rs, const KeyLayout& M, int carried_bits, uint64_t slots, BitmapJoin& bj) {
  if ((c->flags & XLOG_FLAG_NO_BITMAP_JOIN) || carried_bits < 5 || carried_bits > 5 + kBmMaxWordsLog2) return;
  Relation& H = *c->rels[h];
  if (H.dict_n[1]) return;
  const RuleC* rule = nullptr; int pos = -1, n_over = 0;
  for (const RuleC* r : rs)
    for (int j = 0; j < r->plan.n_atoms; ++j)
      if (r->plan.atoms[j].rel == h) { ++n_over; rule = r; pos = j; }
  if (n_over != 1) return;
  const Variant v{rule, pos, Source{nullptr, nullptr, 0, M, H.key_bytes}};
  const JoinSpec S = make_spec(c, v, H, &M);               // builds the looked-up relation's index if it is missing
  if (!S.fast || !S.has_inner || S.inner_free != 1 || S.outer_decode[0] || S.outer_decode[1] || S.head_encode[0] || S.head_encode[1] ||
      S.inner_mult[0] != ((uint64_t)1 << carried_bits))
    return;
  const Relation& RB = *c->rels[rule->plan.atoms[1 - pos].rel];
  const uint64_t passes = (uint64_t)1 << (carried_bits - 5);             // at most one pass per 32 carried values
  const uint64_t values = std::min<uint64_t>((uint64_t)S.inner_domain, slots >> carried_bits);
  const uint64_t max_items = ((uint64_t)RB.n / kBmSlice + values + 1) * passes;
  if (max_items >= ((uint64_t)1 << 32)) return;
  const uint64_t need = slots * 8 + max_items * 16 + (1u << 20);          // a round can change every key: one (tag, carried value) pair each
  if (need > c->arena.largest_free() / 2) return;
  bj.pairs = DevBuf(c, slots * 8);
  bj.items = DevBuf(c, max_items * 16);
  bj.spec = S;
  bj.carried_bits = carried_bits;
  bj.valid = true;
}

}  // namespace
}  // namespace xlog
