// Recursive components over a tag mirror: host-driven rounds, resident rounds (CUDA graph with a WHILE node), grouped and bitmap-driven joins.
// Host-side driver code of the engine; included by xlog_api.cu only (one translation unit).
#pragma once
#include "host_eval.cuh"
#include "bitmap_join.cuh"
#include "dense_closure.cuh"
#include "group_join.cuh"
#include "mirror.cuh"
#include "resident.cuh"
#include "row_fixpoint.cuh"

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
