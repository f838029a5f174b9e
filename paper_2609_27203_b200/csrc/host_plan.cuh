// Rule plans: validation and join shapes, strongly connected components, column bounds and dictionaries.
// Host-side driver code of the engine; included by xlog_api.cu only (one translation unit).
#pragma once
#include "host_store.cuh"

namespace xlog {
namespace {

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

}  // namespace
}  // namespace xlog
