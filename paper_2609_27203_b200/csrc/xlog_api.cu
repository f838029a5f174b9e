// C ABI of the engine (see include/xlog.h) and the host-side fixpoint driver.
#include "engine.cuh"
#include "bitmap_join.cuh"
#include "group_join.cuh"
#include "mirror.cuh"
#include "resident.cuh"
#include "triangle.cuh"
#include "cycle4.cuh"

using namespace xlog;

struct xlog_ctx : public xlog::Ctx {};

namespace {

template <typename F>
xlog_status guarded(xlog_ctx* c, F&& f) {
  if (!c) return XLOG_ERR_INVALID_ARGUMENT;
  try {
    cudaSetDevice(c->device);
    f();
    c->err.clear();
    return XLOG_OK;
  } catch (const Fail& e) {
    c->err = e.msg;
    return e.st;
  } catch (const std::exception& e) {
    c->err = e.what();
    return XLOG_ERR_INTERNAL;
  }
}

// the sort pass needs more than 48 KB of dynamic shared memory and the largest carve-out
template <typename K, int B>
void set_sort_attributes_b() {
  XLOG_CUDA(cudaFuncSetAttribute(k_sort_pass<K, B>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sort_pass_smem<K>()));
  XLOG_CUDA(cudaFuncSetAttribute(k_sort_pass<K, B>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
}
template <typename K>
void set_sort_attributes() {
  set_sort_attributes_b<K, 1>(); set_sort_attributes_b<K, 2>(); set_sort_attributes_b<K, 3>(); set_sort_attributes_b<K, 4>();
  set_sort_attributes_b<K, 5>(); set_sort_attributes_b<K, 6>(); set_sort_attributes_b<K, 7>(); set_sort_attributes_b<K, 8>();
}

Relation& rel_of(Ctx* c, xlog_rel r) {
  if (r < 0 || r >= (int)c->rels.size()) fail(XLOG_ERR_INVALID_ARGUMENT, "bad relation handle");
  return *c->rels[r];
}

float one_of(int sr) { return sr == XLOG_SR_SUMPROD ? 1.f : 0.f; }

#define DISPATCH_K(key_bytes, ...)                        \
  do {                                                    \
    if ((key_bytes) == 4) { typedef uint32_t K; __VA_ARGS__; } \
    else { typedef uint64_t K; __VA_ARGS__; }             \
  } while (0)

void drop_indices(Relation& R) {
  for (int i = 0; i < kMaxArity; ++i) R.idx[i] = Index();
}

void drop_current(Relation& R) {
  R.cur_keys.reset(); R.cur_tags.reset();
  R.cur_owned = false;
  R.n = R.n_facts;
  R.soa_valid = false;
  for (int i = 0; i < kMaxArity; ++i) R.cols[i].reset();
  drop_indices(R);
}

void set_current(Relation& R, KeyTags&& kt) {
  R.cur_keys = std::move(kt.keys);
  R.cur_tags = std::move(kt.tags);
  R.cur_owned = true;
  R.n = kt.n;
  R.soa_valid = false;
  drop_indices(R);
}

// Column-major int32 view of the current contents.
void ensure_soa(Ctx* c, Relation& R) {
  if (R.soa_valid) return;
  ColPtrsMut out{};
  for (int i = 0; i < R.arity; ++i) {
    R.cols[i] = DevBuf(c, (size_t)std::max(R.n, 1u) * 4);
    out.c[i] = R.cols[i].as<int32_t>();
  }
  if (R.n) DISPATCH_K(R.key_bytes, XLOG_LAUNCH(c, (k_unpack<K>), grid_for(R.n, 256), 256, 0, (const K*)R.keys(), (int64_t)R.n, R.layout, R.dicts(), out));
  R.soa_valid = true;
}

// Repack the loaded facts under a wider layout (derived tuples need more bits than the facts).
void relayout_facts(Ctx* c, Relation& R, const KeyLayout& L) {
  if (same_layout(R.layout, L)) return;
  const int nkb = L.total_bits <= 32 ? 4 : 8;
  if (R.n_facts) {
    ColPtrsMut tmp{}; ColPtrs tmpc{};
    DevBuf cols[kMaxArity];
    for (int i = 0; i < R.arity; ++i) { cols[i] = DevBuf(c, (size_t)R.n_facts * 4); tmp.c[i] = cols[i].as<int32_t>(); tmpc.c[i] = tmp.c[i]; }
    DISPATCH_K(R.key_bytes, XLOG_LAUNCH(c, (k_unpack<K>), grid_for(R.n_facts, 256), 256, 0, R.fact_keys.as<K>(), (int64_t)R.n_facts, R.layout, DictSet{}, tmp));
    DevBuf nk(c, (size_t)R.n_facts * nkb);
    DISPATCH_K(nkb, XLOG_LAUNCH(c, (k_pack<K>), grid_for(R.n_facts, 256), 256, 0, tmpc, R.fact_tags.as<float>(), (int64_t)R.n_facts, L,
                                 DictSet{}, 0.f, nk.as<K>(), R.fact_tags.as<float>()));
    R.fact_keys = std::move(nk);
  }
  R.layout = L;
  R.key_bytes = nkb;
  drop_current(R);
}

// ---- load ------------------------------------------------------------------------
void load_relation(Ctx* c, Relation& R, const int32_t* const* cols, const float* tags, int64_t n, xlog_memspace space) {
  if (n < 0 || n > (int64_t)kSortMaxN) fail(XLOG_ERR_CAPACITY_EXCEEDED, "row count must be in [0, 2^30)");
  if (n > 0 && !cols) fail(XLOG_ERR_INVALID_ARGUMENT, "cols is NULL");
  // drop everything the relation held
  drop_current(R);
  R.fact_keys.reset(); R.fact_tags.reset();
  R.n_facts = R.n = 0;
  for (int i = 0; i < kMaxArity; ++i) { R.col_max[i] = R.fact_max[i] = R.val_max[i] = 0; R.dict[i].reset(); R.dict_n[i] = 0; }
  R.layout = make_layout(R.arity, R.col_max);
  R.key_bytes = 4;
  c->idb_dirty = true;
  if (n == 0) return;

  // stage the input columns on the device
  DevBuf stage[kMaxArity], stage_t;
  ColPtrs in{};
  const float* dtags = nullptr;
  if (space == XLOG_MEM_HOST) {
    for (int i = 0; i < R.arity; ++i) {
      if (!cols[i]) fail(XLOG_ERR_INVALID_ARGUMENT, "column pointer is NULL");
      stage[i] = DevBuf(c, (size_t)n * 4);
      XLOG_CUDA(cudaMemcpyAsync(stage[i].p, cols[i], (size_t)n * 4, cudaMemcpyHostToDevice, c->stream));
      in.c[i] = stage[i].as<int32_t>();
    }
    if (tags) {
      stage_t = DevBuf(c, (size_t)n * 4);
      XLOG_CUDA(cudaMemcpyAsync(stage_t.p, tags, (size_t)n * 4, cudaMemcpyHostToDevice, c->stream));
      dtags = stage_t.as<float>();
    }
    c->h2d_bytes += (int64_t)n * 4 * (R.arity + (tags ? 1 : 0));
  } else {
    for (int i = 0; i < R.arity; ++i) { if (!cols[i]) fail(XLOG_ERR_INVALID_ARGUMENT, "column pointer is NULL"); in.c[i] = cols[i]; }
    dtags = tags;
  }

  // validate, find the column maxima (they fix the key layout)
  zero_ctrl(c, kSlotErr);
  zero_ctrl(c, kSlotA, 4);
  XLOG_LAUNCH(c, k_col_stats, grid_for(n, 256, kSMs * 8), 256, 0, in, dtags, n, R.arity, R.sr,
              reinterpret_cast<int32_t*>(c->d_ctrl + kSlotA), ctrl_u32(c, kSlotErr), ctrl_u32(c, kSlotC));
  sync_ctrl(c);
  const bool in_order = (uint32_t)c->h_ctrl[kSlotC] == 0;     // rows arrived strictly increasing: nothing to sort or combine
  const int32_t* mx = reinterpret_cast<const int32_t*>(c->h_ctrl + kSlotA);
  for (int i = 0; i < R.arity; ++i) R.col_max[i] = R.fact_max[i] = R.val_max[i] = mx[i];
  zero_ctrl(c, kSlotA, 4);
  R.layout = make_layout(R.arity, R.col_max);
  if (R.layout.total_bits > 64) fail(XLOG_ERR_CAPACITY_EXCEEDED, "packed key of relation '" + R.name + "' needs more than 64 bits");
  R.key_bytes = R.layout.total_bits <= 32 ? 4 : 8;

  // pack -> sort -> combine duplicates
  if (in_order) {
    DISPATCH_K(R.key_bytes, {
      R.fact_keys = DevBuf(c, (size_t)n * sizeof(K));
      R.fact_tags = DevBuf(c, (size_t)n * 4);
      XLOG_LAUNCH(c, (k_pack<K>), grid_for(n, 256), 256, 0, in, dtags, n, R.layout, DictSet{}, one_of(R.sr), R.fact_keys.as<K>(), R.fact_tags.as<float>());
      R.n_facts = R.n = (uint32_t)n;
    });
    // the pack kernel reads the caller's columns: the load has copied them only once it has run
    XLOG_CUDA(cudaStreamSynchronize(c->stream));
  } else DISPATCH_K(R.key_bytes, {
    DevBuf k0(c, (size_t)n * sizeof(K)), t0(c, (size_t)n * 4), k1(c, (size_t)n * sizeof(K)), t1(c, (size_t)n * 4);
    XLOG_LAUNCH(c, (k_pack<K>), grid_for(n, 256), 256, 0, in, dtags, n, R.layout, DictSet{}, one_of(R.sr), k0.as<K>(), t0.as<float>());
    for (int i = 0; i < kMaxArity; ++i) stage[i].reset();
    stage_t.reset();
    KeyTags kt = sort_reduce<K>(c, R.sr, k0, t0, k1, t1, (uint64_t)n, R.layout.total_bits, false);
    R.fact_keys = std::move(kt.keys);
    R.fact_tags = std::move(kt.tags);
    R.n_facts = R.n = kt.n;
  });
  if (c->flags & XLOG_FLAG_CHECK_INVARIANTS) {
    DISPATCH_K(R.key_bytes, XLOG_LAUNCH(c, (k_check_sorted<K>), grid_for(R.n, 256), 256, 0, R.fact_keys.as<K>(), (int64_t)R.n, ctrl_u32(c, kSlotErr)));
    sync_ctrl(c);
  }
}

// ---- rules -----------------------------------------------------------------------
bool is_plain_var(const xlog_arg& a) { return a.kind == XLOG_ARG_VAR && a.mul == 1 && a.add == 0; }

JoinShape join_shape(Ctx* c, const xlog_plan& p, int outer) {
  JoinShape s;
  s.outer = outer; s.inner = 1 - outer;
  const xlog_atom& A = p.atoms[s.outer];
  const xlog_atom& B = p.atoms[s.inner];
  const int ka = c->rels[A.rel]->arity, kb = c->rels[B.rel]->arity;
  bool bound[XLOG_MAX_VARS] = {false};
  for (int i = 0; i < ka; ++i) if (A.args[i].kind == XLOG_ARG_VAR) bound[A.args[i].var] = true;
  int probe = -1;
  for (int i = 0; i < kb && probe < 0; ++i)
    if (B.args[i].kind == XLOG_ARG_VAR && bound[B.args[i].var]) probe = i;
  if (probe < 0) return s;                       // cross product: not supported
  bool seen[XLOG_MAX_VARS] = {false};
  for (int i = 0; i < kb; ++i) {
    if (i == probe) continue;
    const xlog_arg& a = B.args[i];
    // every other inner column must introduce a fresh variable (filters on the inner side are not supported)
    if (a.kind != XLOG_ARG_VAR || a.mul != 1 || bound[a.var] || seen[a.var]) return s;
    seen[a.var] = true;
  }
  s.probe_col = probe;
  s.probe_var = B.args[probe].var; s.probe_mul = B.args[probe].mul; s.probe_add = B.args[probe].add;
  s.ok = true;
  return s;
}

void add_rule(Ctx* c, const xlog_plan* p, xlog_rule* out) {
  if (!p || !out) fail(XLOG_ERR_INVALID_ARGUMENT, "plan or out is NULL");
  if (p->struct_size != sizeof(xlog_plan)) fail(XLOG_ERR_INVALID_ARGUMENT, "xlog_plan.struct_size mismatch");
  Relation& H = rel_of(c, p->head_rel);
  if (p->n_atoms < 1 || p->n_atoms > XLOG_MAX_ATOMS) fail(XLOG_ERR_INVALID_ARGUMENT, "n_atoms must be 1..4");
  if (p->n_head_cols < 1 || p->n_head_cols + (p->emit_count_column ? 1 : 0) != H.arity)
    fail(XLOG_ERR_INVALID_ARGUMENT, "head columns do not match the head relation's arity");
  bool bound[XLOG_MAX_VARS] = {false};
  for (int j = 0; j < p->n_atoms; ++j) {
    Relation& R = rel_of(c, p->atoms[j].rel);
    if ((R.sr == XLOG_SR_SUMPROD) != (H.sr == XLOG_SR_SUMPROD))
      fail(XLOG_ERR_INVALID_ARGUMENT, "body relation '" + R.name + "' does not share the head's otimes");
    for (int i = 0; i < R.arity; ++i) {
      const xlog_arg& a = p->atoms[j].args[i];
      if (a.kind == XLOG_ARG_VAR) {
        if (a.var < 0 || a.var >= XLOG_MAX_VARS || a.mul <= 0) fail(XLOG_ERR_INVALID_ARGUMENT, "bad variable pattern");
        bound[a.var] = true;
      } else if (a.kind != XLOG_ARG_CONST) fail(XLOG_ERR_INVALID_ARGUMENT, "bad argument kind");
    }
  }
  for (int h = 0; h < p->n_head_cols; ++h)
    for (int v = 0; v < XLOG_MAX_VARS; ++v)
      if (p->head[h].coef[v] != 0 && !bound[v]) fail(XLOG_ERR_INVALID_ARGUMENT, "head uses a variable no body atom binds");
  RuleC r;
  r.plan = *p;
  for (int j = 0; j < p->n_atoms; ++j)
    if (p->atoms[j].negated && !(p->n_atoms == 2 && j == 1)) fail(XLOG_ERR_UNSUPPORTED, "negation is supported as  h :- a(..), not b(..)  only");
  if (p->n_atoms == 1) r.kind = 1;
  else if (p->n_atoms == 2 && p->atoms[1].negated) {
    // the negated atom: a fixed prefix of one or two columns, then wildcards
    const xlog_atom& A = p->atoms[0];
    const xlog_atom& B = p->atoms[1];
    bool in_a[XLOG_MAX_VARS] = {false};
    for (int i = 0; i < c->rels[A.rel]->arity; ++i) if (A.args[i].kind == XLOG_ARG_VAR) in_a[A.args[i].var] = true;
    const int kb = c->rels[B.rel]->arity;
    int prefix = 0;
    for (; prefix < kb && prefix < 2; ++prefix) {
      const xlog_arg& g = B.args[prefix];
      if (!(g.kind == XLOG_ARG_CONST || in_a[g.var])) break;
    }
    bool ok = prefix >= 1;
    for (int i = prefix; i < kb && ok; ++i) {
      const xlog_arg& g = B.args[i];
      ok = g.kind == XLOG_ARG_VAR && !in_a[g.var];
      for (int k = 0; k < kb && ok; ++k) if (k != i && B.args[k].kind == XLOG_ARG_VAR && B.args[k].var == g.var) ok = false;
      for (int hcol = 0; hcol < p->n_head_cols && ok; ++hcol) if (p->head[hcol].coef[g.var] != 0) ok = false;
    }
    if (!ok) fail(XLOG_ERR_UNSUPPORTED, "negated atom: its first one or two columns must be fixed by the positive atom, the rest wildcards");
    r.kind = 5;
    r.neg_prefix = prefix;
  } else if (p->n_atoms == 2) {
    r.kind = 2;
    r.shape[0] = join_shape(c, *p, 0);
    r.shape[1] = join_shape(c, *p, 1);
    if (!r.shape[0].ok && !r.shape[1].ok)
      fail(XLOG_ERR_UNSUPPORTED, "two-atom rule must join on one variable with the looked-up side's other columns plain fresh variables");
  } else if (p->n_atoms == 4) {
    // four-cycle  h(x,y,z,w) :- r(x,y), s(y,z), t(z,w), u(w,x)
    const xlog_atom* a = p->atoms;
    bool ok = p->n_head_cols == 4 && !p->emit_count_column;
    for (int j = 0; j < 4 && ok; ++j) ok = c->rels[a[j].rel]->arity == 2 && is_plain_var(a[j].args[0]) && is_plain_var(a[j].args[1]);
    if (ok) {
      const int hv[4] = {a[0].args[0].var, a[0].args[1].var, a[1].args[1].var, a[2].args[1].var};
      for (int i = 0; i < 4 && ok; ++i) for (int k = i + 1; k < 4 && ok; ++k) ok = hv[i] != hv[k];
      ok = ok && a[1].args[0].var == hv[1] && a[2].args[0].var == hv[2] && a[3].args[0].var == hv[3] && a[3].args[1].var == hv[0];
      for (int h = 0; h < 4 && ok; ++h) {
        ok = p->head[h].c0 == 0;
        for (int v = 0; v < XLOG_MAX_VARS; ++v) ok = ok && p->head[h].coef[v] == (v == hv[h] ? 1 : 0);
      }
    }
    if (!ok) fail(XLOG_ERR_UNSUPPORTED, "four-atom rules are supported only as the four-cycle join h(x,y,z,w) :- r(x,y), s(y,z), t(z,w), u(w,x)");
    r.kind = 6;
  } else {
    // directed triangle  h(x) :- e(x,y), e(y,z), e(z,x)
    const xlog_atom* a = p->atoms;
    const bool one_rel = a[0].rel == a[1].rel && a[1].rel == a[2].rel;
    bool ok = c->rels[a[0].rel]->arity == 2 && c->rels[a[1].rel]->arity == 2 && c->rels[a[2].rel]->arity == 2;
    for (int j = 0; j < 3 && ok; ++j) ok = is_plain_var(a[j].args[0]) && is_plain_var(a[j].args[1]);
    if (ok) {
      const int x = a[0].args[0].var, y = a[0].args[1].var, z = a[1].args[1].var;
      ok = x != y && y != z && x != z && a[1].args[0].var == y && a[2].args[0].var == z && a[2].args[1].var == x;
      const int hv[3] = {x, y, z};
      bool agg = ok && one_rel && p->n_head_cols == 1, mat = ok && p->n_head_cols == 3 && !p->emit_count_column;
      for (int h = 0; h < p->n_head_cols && h < 3; ++h) {
        bool id = p->head[h].c0 == 0;
        for (int v = 0; v < XLOG_MAX_VARS; ++v) id = id && p->head[h].coef[v] == (v == hv[h] ? 1 : 0);
        agg = agg && id; mat = mat && id;
      }
      ok = agg || mat;
      r.kind = mat ? 4 : 3;
    }
    if (!ok) fail(XLOG_ERR_UNSUPPORTED, "three-atom rules are supported only as the triangle join h(x,y,z) :- r(x,y), s(y,z), t(z,x) or its per-x aggregate h(x) over one relation");
  }
  c->rules.push_back(r);
  H.is_head = true;
  c->idb_dirty = true;
  *out = (xlog_rule)c->rules.size() - 1;
}

// ---- indices ---------------------------------------------------------------------
// Sorted access path on column `col` of R's current contents: offsets over that column plus the
// remaining columns and tags in (col, others...) order.  Column 0 reuses the store itself.
Index& ensure_index(Ctx* c, Relation& R, int col) {
  Index& ix = R.idx[col];
  if (ix.valid) return ix;
  ++c->r_index_builds;
  ensure_soa(c, R);
  ix = Index();
  ix.domain = (int64_t)R.val_max[col] + 1;
  ix.n_other = R.arity - 1;
  const int32_t* lead = nullptr;
  if (col == 0 || R.n == 0) {
    lead = R.cols[col].as<int32_t>();
    for (int i = 1; i < R.arity; ++i) { ix.other_src[i - 1] = i; ix.other[i - 1] = R.cols[i].as<int32_t>(); }
    if (col != 0) { int k = 0; for (int i = 0; i < R.arity; ++i) if (i != col) { ix.other_src[k] = i; ix.other[k] = R.cols[i].as<int32_t>(); ++k; } }
    ix.tags = R.tags();
  } else {
    // permuted copy sorted by (col, remaining columns in order)
    int perm[kMaxArity] = {0, 1, 2, 3};
    perm[0] = col;
    { int k = 1; for (int i = 0; i < R.arity; ++i) if (i != col) perm[k++] = i; }
    int32_t pmax[kMaxArity] = {0, 0, 0, 0};
    for (int i = 0; i < R.arity; ++i) pmax[i] = R.val_max[perm[i]];
    const KeyLayout PL = make_layout(R.arity, pmax);
    const int kb = PL.total_bits <= 32 ? 4 : 8;
    ColPtrs in{};
    for (int i = 0; i < R.arity; ++i) in.c[i] = R.cols[perm[i]].as<int32_t>();
    DevBuf lead_buf(c, (size_t)R.n * 4);
    for (int i = 1; i < R.arity; ++i) { ix.own_cols[i - 1] = DevBuf(c, (size_t)R.n * 4); ix.other_src[i - 1] = perm[i]; }
    ix.own_tags = DevBuf(c, (size_t)R.n * 4);
    DISPATCH_K(kb, {
      DevBuf k0(c, (size_t)R.n * sizeof(K)), t0(c, (size_t)R.n * 4), k1(c, (size_t)R.n * sizeof(K)), t1(c, (size_t)R.n * 4);
      XLOG_LAUNCH(c, (k_pack<K>), grid_for(R.n, 256), 256, 0, in, (const float*)R.tags(), (int64_t)R.n, PL, DictSet{}, 0.f, k0.as<K>(), t0.as<float>());
      K* ka = k0.as<K>(); K* kbuf = k1.as<K>();
      float* ta = t0.as<float>(); float* tb = t1.as<float>();
      sort_pairs<K>(c, ka, ta, kbuf, tb, R.n, PL.total_bits);
      ColPtrsMut out{};
      out.c[0] = lead_buf.as<int32_t>();
      for (int i = 1; i < R.arity; ++i) out.c[i] = ix.own_cols[i - 1].as<int32_t>();
      XLOG_LAUNCH(c, (k_unpack<K>), grid_for(R.n, 256), 256, 0, (const K*)ka, (int64_t)R.n, PL, DictSet{}, out);
      XLOG_CUDA(cudaMemcpyAsync(ix.own_tags.p, ta, (size_t)R.n * 4, cudaMemcpyDeviceToDevice, c->stream));
    });
    for (int i = 1; i < R.arity; ++i) ix.other[i - 1] = ix.own_cols[i - 1].as<int32_t>();
    ix.tags = ix.own_tags.as<float>();
    ix.off = DevBuf(c, ((size_t)ix.domain + 1) * 4);
    XLOG_LAUNCH(c, k_build_offsets, grid_for(ix.domain + 1, 256), 256, 0, (const int32_t*)lead_buf.as<int32_t>(), R.n, ix.domain, ix.off.as<uint32_t>());
    ix.valid = true;
    return ix;
  }
  ix.off = DevBuf(c, ((size_t)ix.domain + 1) * 4);
  XLOG_LAUNCH(c, k_build_offsets, grid_for(ix.domain + 1, 256), 256, 0, lead, R.n, ix.domain, ix.off.as<uint32_t>());
  ix.valid = true;
  return ix;
}

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
    // Leading head columns that are the leading columns of the scanned atom, in the same order, are carried over
    // unchanged; the scanned relation is sorted by them (dictionary codes keep the order of the values), so the
    // candidate stream is already ordered by those key bits.
    const xlog_plan& p = v.rule->plan;
    const xlog_atom& A = p.atoms[v.outer_atom];
    const int ka = c->rels[A.rel]->arity;
    int k = 0;
    for (; k < p.n_head_cols && k < ka; ++k) {
      if (!is_plain_var(A.args[k])) break;
      const int var = A.args[k].var;
      bool id = p.head[k].c0 == 0;
      for (int w = 0; w < kMaxVars; ++w) id = id && p.head[k].coef[w] == (w == var ? 1 : 0);
      if (!id) break;
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

// ---- strata ------------------------------------------------------------------------
std::vector<std::vector<int>> components(Ctx* c) {
  const int n = (int)c->rels.size();
  std::vector<std::set<int>> dep(n);
  for (const RuleC& r : c->rules) for (int j = 0; j < r.plan.n_atoms; ++j) dep[r.plan.head_rel].insert(r.plan.atoms[j].rel);
  std::vector<int> idx(n, -1), low(n, 0), stack; std::vector<char> on(n, 0);
  std::vector<std::vector<int>> out; int counter = 0;
  std::function<void(int)> visit = [&](int v) {
    idx[v] = low[v] = counter++; stack.push_back(v); on[v] = 1;
    for (int w : dep[v]) {
      if (idx[w] < 0) { visit(w); low[v] = std::min(low[v], low[w]); }
      else if (on[w]) low[v] = std::min(low[v], idx[w]);
    }
    if (low[v] == idx[v]) {
      std::vector<int> comp;
      for (;;) { int w = stack.back(); stack.pop_back(); on[w] = 0; comp.push_back(w); if (w == v) break; }
      std::sort(comp.begin(), comp.end());
      out.push_back(comp);                 // emitted after everything it depends on
    }
  };
  for (int v = 0; v < n; ++v) if (idx[v] < 0) visit(v);
  return out;
}

// Sorted distinct values of column `col` of (non-derived) relation S: the dictionary of a head column fed by it.
DevBuf distinct_values(Ctx* c, Relation& S, int col, uint32_t* n_out) {
  ensure_soa(c, S);
  const uint32_t n = S.n;
  DevBuf k0(c, (size_t)n * 4), t0(c, (size_t)n * 4), k1(c, (size_t)n * 4), t1(c, (size_t)n * 4);
  XLOG_CUDA(cudaMemcpyAsync(k0.p, S.cols[col].p, (size_t)n * 4, cudaMemcpyDeviceToDevice, c->stream));
  XLOG_CUDA(cudaMemsetAsync(t0.p, 0, (size_t)n * 4, c->stream));
  KeyTags u = sort_reduce<uint32_t>(c, XLOG_SR_MAXPLUS, k0, t0, k1, t1, n, bit_length(S.val_max[col]), false);
  *n_out = u.n;
  return std::move(u.keys);
}

// Upper bounds of every column of every relation (loaded maxima pushed through the rules), which fix
// the packed-key layouts before any kernel runs; and dictionaries for head columns that only ever
// carry values of one small stored column (e.g. reach(s, .) with s drawn from 64 sources).
void propagate_bounds(Ctx* c) {
  const int n = (int)c->rels.size();
  std::vector<std::array<int64_t, kMaxArity>> ub(n);
  for (int r = 0; r < n; ++r) for (int i = 0; i < kMaxArity; ++i) ub[r][i] = c->rels[r]->n_facts ? c->rels[r]->fact_max[i] : 0;
  for (int round = 0; round < n + 3; ++round) {
    bool changed = false;
    for (const RuleC& rc : c->rules) {
      const xlog_plan& p = rc.plan;
      int64_t vub[XLOG_MAX_VARS];
      for (int v = 0; v < XLOG_MAX_VARS; ++v) vub[v] = INT32_MAX;
      for (int j = 0; j < p.n_atoms; ++j) {
        const Relation& R = *c->rels[p.atoms[j].rel];
        if (p.atoms[j].negated) continue;                  // binds nothing
        for (int i = 0; i < R.arity; ++i) {
          const xlog_arg& a = p.atoms[j].args[i];
          if (a.kind != XLOG_ARG_VAR) continue;
          const int64_t b = (ub[p.atoms[j].rel][i] - a.add) / a.mul;
          vub[a.var] = std::min(vub[a.var], std::max<int64_t>(b, 0));
        }
      }
      for (int h = 0; h < p.n_head_cols; ++h) {
        int64_t b = p.head[h].c0;
        for (int v = 0; v < XLOG_MAX_VARS; ++v) if (p.head[h].coef[v] > 0) b += (int64_t)p.head[h].coef[v] * vub[v];
        b = std::min<int64_t>(std::max<int64_t>(b, 0), INT32_MAX);
        if (round >= n + 1 && b > ub[p.head_rel][h]) b = INT32_MAX;      // still growing: recursive arithmetic
        if (b > ub[p.head_rel][h]) { ub[p.head_rel][h] = b; changed = true; }
      }
    }
    if (!changed) break;
  }
  for (int r = 0; r < n; ++r) {
    Relation& R = *c->rels[r];
    if (!R.is_head) continue;
    int32_t mx[kMaxArity] = {0, 0, 0, 0};
    for (int i = 0; i < R.arity; ++i) { mx[i] = (int32_t)ub[r][i]; R.val_max[i] = mx[i]; R.dict[i].reset(); R.dict_n[i] = 0; }
    // dictionary candidates: every rule writes the column as a bare variable that is bound either by the
    // same column of this relation (carried along) or by a column of a stored, non-derived relation
    bool plain_rules = R.n_facts == 0;
    for (const RuleC& rc : c->rules) if (rc.plan.head_rel == r && (rc.kind >= 3 || rc.plan.emit_count_column)) plain_rules = false;
    for (int col = 0; col < R.arity && plain_rules; ++col) {
      int src_rel = -1, src_col = -1;
      bool ok = true;
      for (const RuleC& rc : c->rules) {
        const xlog_plan& p = rc.plan;
        if (p.head_rel != r) continue;
        int v = -1;
        bool identity = p.head[col].c0 == 0;
        for (int k = 0; k < XLOG_MAX_VARS; ++k) if (p.head[col].coef[k] != 0) { if (v >= 0 || p.head[col].coef[k] != 1) identity = false; v = k; }
        if (!identity || v < 0) { ok = false; break; }
        // where the variable comes from: a carry of this very column, else the smallest stored relation binding it plainly
        bool carried = false;
        int best_rel = -1, best_col = -1;
        for (int j = 0; j < p.n_atoms; ++j)
          for (int k = 0; k < c->rels[p.atoms[j].rel]->arity; ++k) {
            const xlog_arg& g = p.atoms[j].args[k];
            if (p.atoms[j].negated || g.kind != XLOG_ARG_VAR || g.var != v || g.mul != 1 || g.add != 0) continue;
            if (p.atoms[j].rel == r && k == col) carried = true;
            else if (!c->rels[p.atoms[j].rel]->is_head && (best_rel < 0 || c->rels[p.atoms[j].rel]->n < c->rels[best_rel]->n)) { best_rel = p.atoms[j].rel; best_col = k; }
          }
        if (carried && best_rel < 0) continue;                         // pure carry: adds no values
        if (best_rel < 0) { ok = false; break; }
        if (src_rel >= 0 && (src_rel != best_rel || src_col != best_col)) { ok = false; break; }   // one source column only
        src_rel = best_rel; src_col = best_col;
      }
      if (!ok || src_rel < 0) continue;
      Relation& S = *c->rels[src_rel];
      // worth it only if the codes are clearly narrower than the values
      if (S.n == 0 || S.n > (1u << 16) || bit_length((int64_t)S.n - 1) + 2 > bit_length(mx[col])) continue;
      uint32_t dn = 0;
      R.dict[col] = distinct_values(c, S, src_col, &dn);
      R.dict_n[col] = dn;
      mx[col] = (int32_t)dn - 1;
    }
    const KeyLayout L = make_layout(R.arity, mx);
    if (L.total_bits > 64) fail(XLOG_ERR_CAPACITY_EXCEEDED, "packed key of relation '" + R.name + "' needs more than 64 bits");
    for (int i = 0; i < R.arity; ++i) R.col_max[i] = mx[i];
    relayout_facts(c, R, L);
  }
}

void reset_idb(Ctx* c) {
  for (Relation* R : c->rels) if (R->is_head) drop_current(*R);
  c->poisoned = false;
  c->evaluated = false;
}

bool in_set(const std::vector<int>& comp, int r) { return std::binary_search(comp.begin(), comp.end(), r); }

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
  XLOG_LAUNCH(c, k_tri_plan, grid_for(ne1, 256), 256, 0, G, items.as<uint32_t>(), (unsigned long long*)(c->d_ctrl + kSlotC));
  XLOG_LAUNCH(c, (k_scan_tile_sums<uint32_t, uint32_t>), it_tiles, kScanBlock, 0, (const uint32_t*)items.as<uint32_t>(), (int64_t)ne1, it_sums.as<uint32_t>());
  XLOG_LAUNCH(c, (k_scan_spine<uint32_t>), 1, 1024, 0, it_sums.as<uint32_t>(), (int64_t)it_tiles, ctrl_u32(c, kSlotB));
  XLOG_LAUNCH(c, (k_scan_apply<uint32_t, uint32_t>), it_tiles, kScanBlock, 0, (const uint32_t*)items.as<uint32_t>(), (int64_t)ne1,
              (const uint32_t*)it_sums.as<uint32_t>(), item_off.as<uint32_t>());
  sync_ctrl(c);
  const uint32_t n_items = (uint32_t)c->h_ctrl[kSlotB];
  const uint64_t walked = c->h_ctrl[kSlotC];               // sorted-list probes of the whole join
  items.reset(); it_sums.reset();
  DevBuf item_edge(c, (size_t)std::max(n_items, 1u) * 4), ecnt(c, (size_t)std::max(n_items, 1u) * 4), eacc(c, (size_t)std::max(n_items, 1u) * sizeof(A));
  DevBuf gcnt(c, (size_t)domain * 4), gtag(c, (size_t)domain * 4), flag(c, (size_t)domain * 4);
  const unsigned scan_tiles = (unsigned)((domain + kScanTile - 1) / kScanTile);
  DevBuf spine(c, ((size_t)scan_tiles + 1) * 4);
  zero_ctrl(c, kSlotA, 4);
  XLOG_LAUNCH(c, k_tri_item_edges, grid_for(E.n, 256), 256, 0, E.n, (const uint32_t*)item_off.as<uint32_t>(), item_edge.as<uint32_t>());
  // declared work: one 4-byte entry per probe (the walked lists) plus the edge rows; the searches themselves hit L1 / L2
  c->note_bytes = (int64_t)walked * 4 + (int64_t)E.n * 12;
  c->r_candidates += (int64_t)walked;
  XLOG_LAUNCH(c, (k_tri_edges<Op>), kSMs * 8, 256, 0, G, H.sr == XLOG_SR_SUMPROD ? 1 : 0, n_items, (const uint32_t*)item_off.as<uint32_t>(),
              (const uint32_t*)item_edge.as<uint32_t>(), ecnt.as<uint32_t>(), eacc.as<A>());
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
    if (bitmap)                                                                                                                    \
      XLOG_LAUNCH(c, (k_cycle4_bitmap<K2, KH, EMIT>), bgrid, 256, 0, P, (const K2*)k0.p, (const float*)t0.as<float>(), n2,         \
                  cnt.as<uint32_t>(), (const uint64_t*)off.as<uint64_t>(), (KH*)(KEYS), (float*)(TAGS));                           \
    else                                                                                                                           \
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

// Gradient of a non-recursive logsumexp / sum rule with respect to its body tags: enumerate the
// bindings again (count -> scan -> tiled walk) and scatter g[h] * weight to the body rows.
void rule_backward(Ctx* c, const RuleC& r, const float* g, float* const* grads) {
  Relation& H = *c->rels[r.plan.head_rel];
  if (H.sr != XLOG_SR_LOGSUMEXP && H.sr != XLOG_SR_SUMPROD) fail(XLOG_ERR_UNSUPPORTED, "backward is defined for logsumexp and sum heads only");
  if (r.kind == 3 || r.kind == 4 || r.kind == 6) fail(XLOG_ERR_UNSUPPORTED, "backward of the triangle and four-cycle rules is not built");
  for (int j = 0; j < r.plan.n_atoms; ++j) {
    if (!grads[j] && c->rels[r.plan.atoms[j].rel]->n) fail(XLOG_ERR_INVALID_ARGUMENT, "NULL gradient buffer");
    if (r.plan.atoms[j].rel == r.plan.head_rel) fail(XLOG_ERR_UNSUPPORTED, "backward of a recursive rule");
  }
  int outer = 0;
  if (r.kind == 2 && !r.shape[0].ok) outer = 1;
  if (r.kind == 2 && r.shape[outer].probe_col != 0) fail(XLOG_ERR_UNSUPPORTED, "backward needs the looked-up atom probed on its first column");
  // zero-fill each distinct buffer once
  for (int j = 0; j < r.plan.n_atoms; ++j) {
    bool seen = false;
    for (int i = 0; i < j; ++i) seen = seen || grads[i] == grads[j];
    if (!seen && grads[j]) XLOG_CUDA(cudaMemsetAsync(grads[j], 0, (size_t)c->rels[r.plan.atoms[j].rel]->n * 4, c->stream));
  }
  Relation& RA = *c->rels[r.plan.atoms[outer].rel];
  if (RA.n == 0 || H.n == 0) { XLOG_CUDA(cudaStreamSynchronize(c->stream)); return; }
  Variant v{&r, outer, full_source(RA)};
  Counted q;
  count_variant(c, v, H, q, kSlotTotals);
  sync_ctrl(c);
  q.total = c->h_ctrl[q.slot];
  const int ckb = q.spec.head.total_bits <= 32 ? 4 : 8;
  if (ckb != H.key_bytes) fail(XLOG_ERR_UNSUPPORTED, "backward: head key width differs from the declared-column key width");
  BwdArgs bw{};
  bw.head_keys = H.keys(); bw.head_tags = H.tags(); bw.n_head = H.n;
  bw.count_bits = r.plan.emit_count_column ? H.layout.shift[r.plan.n_head_cols - 1] : 0;
  bw.grad_head = g;
  bw.grad_outer = grads[outer];
  bw.grad_inner = r.kind == 2 ? grads[1 - outer] : nullptr;     // a negated atom (kind 5) carries no tag: its buffer stays zero
  bw.lse = H.sr == XLOG_SR_LOGSUMEXP ? 1 : 0;
  if (q.total) launch_expand<true>(c, q, 0, q.total, ckb, nullptr, nullptr, bw);
  sync_ctrl(c);
}

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

constexpr int kSlotMirNew = 12, kSlotMirChanged = 13;
constexpr int kMirrorMaxBits = 30;

// The tag mirror serves a component of one max/min relation whose rules are all linear (at most one atom over the
// relation itself, and that atom is the scanned side): then the relation is only ever read through its delta, and
// its sorted form is needed again only after the last round.
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
    if (in > 1) return false;
    if (in == 1 && r->kind == 2 && !r->shape[pos].ok) return false;
    if (in == 1 && r->kind != 2 && pos != 0) return false;
    if (in == 0 && r->kind == 2 && !r->shape[0].ok && !r->shape[1].ok) return false;
  }
  const uint64_t need = ((uint64_t)4 << H.layout.total_bits) + ((uint64_t)1 << H.layout.total_bits) / 4 + (1u << 20);
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
  R->tickets = DevBuf(c, (kResMaxVariants + 2) * 4);
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

// One round's launches.  Nothing here allocates, copies or waits: the same calls are either captured into the WHILE
// body or issued directly (host-driven rounds, used when launches are being timed one by one).
void resident_body(Ctx* c, Resident& R, const std::vector<JoinSpec>& specs, bool is_max, const MirrorArgs& mr, uint32_t bm_quads, unsigned ch_tiles,
                   cudaGraphConditionalHandle handle, int use_handle) {
  ResState* st = res_state(c);
  uint32_t* err = ctrl_u32(c, kSlotErr);
  const uint32_t* dk = R.dkeys.as<uint32_t>();
  const ResScratch sc{R.scan_status.as<unsigned long long>(), R.scan_tiles_cap, R.tickets.as<uint32_t>()};
  for (size_t v = 0; v < specs.size(); ++v) {
    const JoinSpec& S = specs[v];
    XLOG_LAUNCH(c, (k_res_count_scan<uint32_t>), kSMs * 4, kScanBlock, 0, S, dk, (const float*)R.dtags.as<float>(), st, R.rowinfo.as<uint4>(),
                R.start.as<uint64_t>(), R.tile_rows.as<uint2>(), sc.scan_status + v * R.scan_tiles_cap, sc.tickets + v, err, c->spin_limit);
// four waves of blocks: the hardware hands a new block to whichever SM finishes first, which evens out skewed tiles
#define XLOG_RES_EXPAND(MODE, SINK)                                                                                                         \
  XLOG_LAUNCH(c, (k_res_expand<uint32_t, MODE, SINK>), kSMs * kExpMirrorBlocksPerSM * 4, kExpBlock, 0, S, dk, (const ResState*)st, (const uint64_t*)R.start.as<uint64_t>(), \
              (const uint4*)R.rowinfo.as<uint4>(), (const uint2*)R.tile_rows.as<uint2>(), err, mr)
    if (S.fast) { if (is_max) XLOG_RES_EXPAND(kExpFast, kSinkMax); else XLOG_RES_EXPAND(kExpFast, kSinkMin); }
    else { if (is_max) XLOG_RES_EXPAND(kExpGeneric, kSinkMax); else XLOG_RES_EXPAND(kExpGeneric, kSinkMin); }
#undef XLOG_RES_EXPAND
  }
  uint32_t* ctr = sc.tickets + kResMaxVariants;
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
    c->launches = l0 + R.body_launches * (int64_t)out.rounds + (out.status == kResOverflow ? R.body_launches : 0);
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
        auto cs = c->prof_index.find("k_res_count_scan");
        if (cs != c->prof_index.end()) c->prof[cs->second].bytes += (int64_t)rows * 40 * (int64_t)specs.size();
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

// Algorithm 1 over a tag mirror (mirror.cuh): per round  count -> scan -> join straight into the table -> compact the
// changed bitmap into the next delta.  No candidate is ever written to memory.  The seed round is driven by the host
// (its rules scan whole relations of known size); the delta rounds run resident where the fixed-capacity buffers fit.
void stratum_recursive_mirror(Ctx* c, int h, const std::vector<const RuleC*>& rs) {
  Relation& H = *c->rels[h];
  const std::vector<int> comp{h};
  const int bits = H.layout.total_bits;
  const uint64_t dom = (uint64_t)1 << bits;
  const bool is_max = H.sr == XLOG_SR_MAXPLUS;
  const int32_t empty = is_max ? kMirrorEmptyMax : kMirrorEmptyMin;
  const uint64_t slots = std::max<uint64_t>(dom, 4);
  const uint32_t bm_quads = (uint32_t)((std::max<uint64_t>(dom / 32, 1) + 3) / 4);
  const unsigned ch_tiles = mirror_tiles(bm_quads * 4);
  Resident* R = resident_for(c, h, bits, slots, bm_quads, ch_tiles);
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
        for (int j = 0; j < r->plan.n_atoms; ++j)
          if (r->plan.atoms[j].rel == h && dn) vs.push_back(Variant{r, j, Source{dk, dt, dn, M, H.key_bytes}});
      }
    }
    const uint64_t total = host_apply(vs);
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
        if (getenv("XLOG_TRACE")) fprintf(stderr, "bm round %lld: changed %llu new %llu cand %llu items %llu nbrs %llu\n", (long long)round, (unsigned long long)changed,
                                          (unsigned long long)n_new, (unsigned long long)cand, (unsigned long long)n_items, (unsigned long long)nbrs);
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

// =====================================================================================
extern "C" {

xlog_status xlog_ctx_create(const xlog_config* cfg, xlog_ctx** out) {
  if (!cfg || !out || cfg->struct_size != sizeof(xlog_config) || !cfg->arena || cfg->arena_bytes < (1u << 16)) return XLOG_ERR_INVALID_ARGUMENT;
  xlog_ctx* c = new (std::nothrow) xlog_ctx();
  if (!c) return XLOG_ERR_INTERNAL;
  c->device = cfg->device;
  c->stream = (cudaStream_t)cfg->stream;
  c->max_iter = cfg->max_iterations > 0 ? cfg->max_iterations : (int64_t)1 << 20;
  c->chunk_bytes = cfg->candidate_chunk_bytes;
  c->flags = cfg->flags;
  c->arena.init(cfg->arena, cfg->arena_bytes);
  xlog_status st = guarded(c, [&] {
    c->d_ctrl = reinterpret_cast<uint64_t*>(c->arena.alloc(kCtrlSlots * sizeof(uint64_t)));
    if (!c->d_ctrl) fail(XLOG_ERR_RESOURCE_EXHAUSTED, "arena too small");
    XLOG_CUDA(cudaHostAlloc(&c->h_ctrl, kCtrlSlots * sizeof(uint64_t), cudaHostAllocDefault));
    XLOG_CUDA(cudaMemsetAsync(c->d_ctrl, 0, kCtrlSlots * sizeof(uint64_t), c->stream));
    XLOG_CUDA(cudaEventCreate(&c->ev0));
    XLOG_CUDA(cudaEventCreate(&c->ev1));
    set_sort_attributes<uint32_t>();
    set_sort_attributes<uint64_t>();
    XLOG_CUDA(cudaStreamSynchronize(c->stream));
  });
  if (st != XLOG_OK) { if (c->h_ctrl) cudaFreeHost(c->h_ctrl); delete c; return st; }
  *out = c;
  return XLOG_OK;
}

xlog_status xlog_ctx_destroy(xlog_ctx* c) {
  if (!c) return XLOG_ERR_INVALID_ARGUMENT;
  cudaSetDevice(c->device);
  cudaStreamSynchronize(c->stream);
  for (Relation* R : c->rels) delete R;
  if (c->h_ctrl) cudaFreeHost(c->h_ctrl);
  if (c->ev0) cudaEventDestroy(c->ev0);
  if (c->ev1) cudaEventDestroy(c->ev1);
  c->resident.clear();
  if (c->capture_stream) cudaStreamDestroy(c->capture_stream);
  for (auto& p : c->prof_pending) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  delete c;
  return XLOG_OK;
}

const char* xlog_last_error(const xlog_ctx* c) { return c ? c->err.c_str() : "null context"; }

xlog_status xlog_relation_create(xlog_ctx* c, int32_t arity, xlog_semiring sr, const char* name, xlog_rel* out) {
  return guarded(c, [&] {
    if (!out || arity < 1 || arity > XLOG_MAX_ARITY || (int)sr < 0 || (int)sr > 3) fail(XLOG_ERR_INVALID_ARGUMENT, "bad arity or semiring");
    Relation* R = new Relation();
    R->arity = arity; R->sr = (int)sr; R->name = name ? name : "";
    R->layout = make_layout(arity, R->col_max);
    c->rels.push_back(R);
    *out = (xlog_rel)c->rels.size() - 1;
  });
}

xlog_status xlog_relation_load(xlog_ctx* c, xlog_rel rel, const int32_t* const* cols, const float* tags, int64_t n, xlog_memspace space) {
  return guarded(c, [&] {
    Relation& R = rel_of(c, rel);
    try { load_relation(c, R, cols, tags, n, space); }
    catch (...) {                          // a rejected load leaves the relation empty
      drop_current(R); R.fact_keys.reset(); R.fact_tags.reset(); R.n = R.n_facts = 0;
      for (int i = 0; i < kMaxArity; ++i) R.col_max[i] = 0;
      R.layout = make_layout(R.arity, R.col_max); R.key_bytes = 4;
      throw;
    }
  });
}

xlog_status xlog_relation_size(xlog_ctx* c, xlog_rel rel, int64_t* n) {
  return guarded(c, [&] {
    Relation& R = rel_of(c, rel);
    if (!n) fail(XLOG_ERR_INVALID_ARGUMENT, "n is NULL");
    if (R.is_head && c->poisoned) fail(XLOG_ERR_INVALID_STATE, "derived relations are poisoned");
    if (R.is_head && c->idb_dirty) { reset_idb(c); c->idb_dirty = false; }
    *n = R.n;
  });
}

xlog_status xlog_relation_view(xlog_ctx* c, xlog_rel rel, const int32_t** cols, const float** tags, int64_t* n) {
  return guarded(c, [&] {
    Relation& R = rel_of(c, rel);
    if (R.is_head && c->poisoned) fail(XLOG_ERR_INVALID_STATE, "derived relations are poisoned");
    if (R.is_head && c->idb_dirty) { reset_idb(c); c->idb_dirty = false; }
    ensure_soa(c, R);
    XLOG_CUDA(cudaStreamSynchronize(c->stream));
    if (cols) for (int i = 0; i < R.arity; ++i) cols[i] = R.cols[i].as<int32_t>();
    if (tags) *tags = R.tags();
    if (n) *n = R.n;
  });
}

xlog_status xlog_relation_read(xlog_ctx* c, xlog_rel rel, int32_t* const* cols_out, float* tags_out, int64_t capacity, int64_t* n_out,
                               xlog_memspace space) {
  return guarded(c, [&] {
    Relation& R = rel_of(c, rel);
    if (R.is_head && c->poisoned) fail(XLOG_ERR_INVALID_STATE, "derived relations are poisoned");
    if (R.is_head && c->idb_dirty) { reset_idb(c); c->idb_dirty = false; }
    if ((int64_t)R.n > capacity) { if (n_out) *n_out = R.n; fail(XLOG_ERR_BUFFER_TOO_SMALL, "capacity smaller than the relation"); }
    ensure_soa(c, R);
    const cudaMemcpyKind kind = space == XLOG_MEM_HOST ? cudaMemcpyDeviceToHost : cudaMemcpyDeviceToDevice;
    if (R.n) {
      if (cols_out) for (int i = 0; i < R.arity; ++i) if (cols_out[i]) XLOG_CUDA(cudaMemcpyAsync(cols_out[i], R.cols[i].p, (size_t)R.n * 4, kind, c->stream));
      if (tags_out) XLOG_CUDA(cudaMemcpyAsync(tags_out, R.tags(), (size_t)R.n * 4, kind, c->stream));
    }
    XLOG_CUDA(cudaStreamSynchronize(c->stream));
    if (space == XLOG_MEM_HOST) c->d2h_bytes += (int64_t)R.n * 4 * (R.arity + 1);
    if (n_out) *n_out = R.n;
  });
}

xlog_status xlog_rule_add(xlog_ctx* c, const xlog_plan* plan, xlog_rule* out) {
  return guarded(c, [&] { add_rule(c, plan, out); });
}

xlog_status xlog_ctx_reset_idb(xlog_ctx* c) {
  return guarded(c, [&] { XLOG_CUDA(cudaStreamSynchronize(c->stream)); reset_idb(c); c->idb_dirty = false; });
}

xlog_status xlog_fixpoint(xlog_ctx* c, xlog_receipt* receipt) {
  if (!c) return XLOG_ERR_INVALID_ARGUMENT;
  if (receipt && receipt->struct_size != sizeof(xlog_receipt)) return XLOG_ERR_INVALID_ARGUMENT;
  const int64_t l0 = c->launches, d0 = c->d2h_bytes, h0 = c->h2d_bytes;
  c->r_candidates = c->r_unique = c->r_new = c->r_improved = c->r_iterations = c->r_strata = c->r_index_builds = 0;
  c->unique_untracked = false;
  c->last_triangle_plan = XLOG_PLAN_NONE;
  c->arena.reset_peak();
  cudaSetDevice(c->device);
  cudaEventRecord(c->ev0, c->stream);
  xlog_status st = guarded(c, [&] { run_fixpoint(c); });
  cudaEventRecord(c->ev1, c->stream);
  cudaEventSynchronize(c->ev1);
  if (st != XLOG_OK) {
    // leave no work in flight and no error flag behind; the derived relations stay poisoned
    cudaStreamSynchronize(c->stream);
    cudaMemsetAsync(c->d_ctrl, 0, kCtrlSlots * sizeof(uint64_t), c->stream);
    cudaStreamSynchronize(c->stream);
  }
  if (receipt) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, c->ev0, c->ev1);
    receipt->status = st;
    receipt->strata = c->r_strata;
    receipt->iterations = c->r_iterations;
    int64_t derived = 0;
    if (st == XLOG_OK) for (Relation* R : c->rels) if (R->is_head) derived += (int64_t)R->n - R->n_facts;
    receipt->derived_tuples = derived;
    receipt->candidates = c->r_candidates;
    receipt->unique_candidates = c->unique_untracked ? -1 : c->r_unique;
    receipt->new_tuples = c->r_new;
    receipt->improved_tags = c->r_improved;
    receipt->h2d_bytes = c->h2d_bytes - h0;
    receipt->d2h_bytes = c->d2h_bytes - d0;
    receipt->kernel_launches = c->launches - l0;
    receipt->peak_arena_bytes = (int64_t)c->arena.peak();
    receipt->device_ms = ms;
    receipt->triangle_plan = c->last_triangle_plan;
    receipt->index_builds = (int32_t)std::min<int64_t>(c->r_index_builds, INT32_MAX);
  }
  return st;
}

xlog_status xlog_sort_pairs(xlog_ctx* c, void* keys, void* payload, int64_t n, int32_t key_bytes, int32_t key_bits) {
  return guarded(c, [&] {
    if (n < 0 || (n > 0 && (!keys || !payload)) || (key_bytes != 4 && key_bytes != 8) || key_bits < 0 || key_bits > key_bytes * 8)
      fail(XLOG_ERR_INVALID_ARGUMENT, "xlog_sort_pairs: bad argument");
    if (n <= 1) return;
    DevBuf k1(c, (size_t)n * key_bytes), t1(c, (size_t)n * 4);
    DISPATCH_K(key_bytes, {
      K* ka = (K*)keys; K* kb = k1.as<K>();
      float* ta = (float*)payload; float* tb = t1.as<float>();
      sort_pairs<K>(c, ka, ta, kb, tb, (uint64_t)n, key_bits);
      if ((void*)ka != keys) {
        XLOG_CUDA(cudaMemcpyAsync(keys, ka, (size_t)n * key_bytes, cudaMemcpyDeviceToDevice, c->stream));
        XLOG_CUDA(cudaMemcpyAsync(payload, ta, (size_t)n * 4, cudaMemcpyDeviceToDevice, c->stream));
      }
    });
    sync_ctrl(c);
  });
}

xlog_status xlog_debug_set_poll_limit(xlog_ctx* c, uint32_t polls) {
  return guarded(c, [&] {
    if (polls == 0) fail(XLOG_ERR_INVALID_ARGUMENT, "poll limit must be positive");
    c->spin_limit = polls;
  });
}

// One 8-bit sort pass whose first tile never runs: tiles 1 .. T-1 are launched (tickets start at 1), tile 0's status words
// stay empty, and every look-back that reaches them gives up after the context's poll limit.
xlog_status xlog_debug_sort_pass_without_first_tile(xlog_ctx* c, const void* keys, const void* payload, void* out_keys, void* out_payload, int64_t n,
                                                    int32_t key_bytes) {
  return guarded(c, [&] {
    if (!keys || !payload || !out_keys || !out_payload || (key_bytes != 4 && key_bytes != 8) || n <= 0 || n > (int64_t)kSortMaxN)
      fail(XLOG_ERR_INVALID_ARGUMENT, "xlog_debug_sort_pass_without_first_tile: bad argument");
    DISPATCH_K(key_bytes, {
      const uint32_t ntiles = (uint32_t)((n + sort_tile<K>() - 1) / sort_tile<K>());
      if (ntiles < 2) fail(XLOG_ERR_INVALID_ARGUMENT, "xlog_debug_sort_pass_without_first_tile: needs at least two tiles of rows");
      const SortPasses P = make_sort_passes(0, 8);
      const size_t head_words = (size_t)kSortMaxPasses * kSortMaxBins + kSortMaxPasses + 8;
      DevBuf scratch(c, (head_words + (size_t)ntiles * kSortMaxBins) * 4);
      uint32_t* hist = scratch.as<uint32_t>();
      uint32_t* tickets = hist + kSortMaxPasses * kSortMaxBins;
      uint32_t* done = tickets + kSortMaxPasses;
      XLOG_CUDA(cudaMemsetAsync(hist, 0, (head_words + (size_t)ntiles * kSortMaxBins) * 4, c->stream));
      zero_ctrl(c, kSlotErr);
      XLOG_LAUNCH(c, (k_sort_digit_hist<K>), grid_for(n, 256 * 8, kSMs * 8), 256, 0, (const K*)keys, (uint32_t)n, P, hist, done);
      const uint32_t one = 1;
      XLOG_CUDA(cudaMemcpyAsync(tickets, &one, 4, cudaMemcpyHostToDevice, c->stream));
      XLOG_LAUNCH(c, (k_sort_pass<K, 8>), ntiles - 1, kSortBlock, sort_pass_smem<K>(), (const K*)keys, (const uint32_t*)payload, (K*)out_keys, (uint32_t*)out_payload,
                  (uint32_t)n, 0, hist, hist + head_words, tickets, ctrl_u32(c, kSlotErr), c->spin_limit);
    });
    sync_ctrl(c);                          // raises INTERNAL when a wait gave up
  });
}

xlog_status xlog_profile_read(xlog_ctx* c, xlog_kernel_stat* out, int32_t capacity, int32_t* n_out) {
  return guarded(c, [&] {
    XLOG_CUDA(cudaStreamSynchronize(c->stream));
    prof_collect(c);
    if (n_out) *n_out = (int32_t)c->prof.size();
    if (!out) return;
    for (int i = 0; i < (int)c->prof.size() && i < capacity; ++i) {
      memset(&out[i], 0, sizeof(out[i]));
      strncpy(out[i].name, c->prof[i].name.c_str(), sizeof(out[i].name) - 1);
      out[i].launches = c->prof[i].launches;
      out[i].device_ms = c->prof[i].ms;
      out[i].algorithmic_bytes = c->prof[i].bytes;
    }
  });
}

xlog_status xlog_profile_reset(xlog_ctx* c) {
  return guarded(c, [&] {
    XLOG_CUDA(cudaStreamSynchronize(c->stream));
    prof_collect(c);
    c->prof.clear(); c->prof_index.clear();
  });
}

xlog_status xlog_rule_backward(xlog_ctx* c, xlog_rule rule, const float* grad_head, float* const* grad_atoms) {
  return guarded(c, [&] {
    if (rule < 0 || rule >= (int)c->rules.size()) fail(XLOG_ERR_INVALID_ARGUMENT, "bad rule handle");
    if (!grad_atoms) fail(XLOG_ERR_INVALID_ARGUMENT, "NULL gradient pointer");
    if (!grad_head && c->rels[c->rules[rule].plan.head_rel]->n) fail(XLOG_ERR_INVALID_ARGUMENT, "NULL gradient pointer");   // an empty head has no gradient rows
    if (c->poisoned || !c->evaluated || c->idb_dirty) fail(XLOG_ERR_INVALID_STATE, "xlog_rule_backward needs a successful xlog_fixpoint first");
    rule_backward(c, c->rules[rule], grad_head, grad_atoms);
  });
}

}  // extern "C"
