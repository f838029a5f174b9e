// CPU oracle for tagged-Datalog fixpoint evaluation.  TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, plain definition that the CUDA path is checked against.
// Only the tests, the smoke check and the benchmark's cpu-baseline leg may use
// it; the product never calls it and shares no code with it.
//
// What it computes (paper: "Semi-naive evaluation on GPU", Algorithm 1, read with
// the head aggregates of "Aggregations and constraints" as semiring tags):
//   * a relation of arity k is a finite map  int32^k -> fp32 tag;
//   * semirings (oplus, otimes, zero, one):  MAXPLUS (max,+,-inf,0),
//     MINPLUS (min,+,+inf,0), LOGSUMEXP (logaddexp,+,-inf,0), SUMPROD (+,*,0,1);
//   * a rule contributes, for every binding of its body variables whose atoms
//     are all present, the otimes-product of the atom tags (taken left to right
//     in atom order) to the head tuple; contributions to one head tuple combine
//     with the head relation's oplus; a tuple is present iff it has a derivation;
//   * strata are the strongly connected components of "head depends on body
//     relation", in dependency order.  A non-recursive stratum evaluates every
//     rule once:  I(P) = facts(P) oplus  (oplus over rules of T_r).  A recursive
//     component (only idempotent oplus, i.e. max/min: the paper's stratifier
//     rejects aggregation inside a recursive component) iterates
//     I_{k+1} = I_k oplus T(I_k) on a snapshot until nothing changes
//     (Algorithm 1's "until all Delta empty", naive form);
//   * a negated atom (stratified negation-as-failure over a relation of a lower stratum: paper sections
//     "Aggregations and constraints" and "Completeness over finite domains", Listing 7's constraint
//     `:- edge(X,_), not degree(X,_)`) holds for a binding iff no stored row matches it; variables that occur
//     nowhere else act as wildcards; it contributes the semiring one to the tag;
//   * otimes is evaluated in fp32 for MAXPLUS/MINPLUS (which makes tags
//     bit-comparable) and in fp64 with one final rounding for LOGSUMEXP/SUMPROD;
//     logsumexp of a group is  m + log(sum exp(v - m)), m = max v, in fp64.
//
// mode 0 (naive) is the definition.  mode 1 (semi-naive, Algorithm 1 with tag
// improvement) is a second, delta-driven evaluator used where naive is too slow;
// tests hold the two equal on every small case.
//
// Pins (tests/test_oracle_*.py): chain / complete-DAG / cycle closed forms, the
// paper's Listing 1 and Listing 7 examples, fp32 Dijkstra (bit-exact), fp64
// Floyd-Warshall, brute-force path enumeration, trace(A^3), O(n^3) triangle brute
// force, discrete convolution, finite differences, torch.logsumexp / autograd.

#include <algorithm>
#include <array>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>
#include <limits>
#include <map>
#include <set>
#include <string>
#include <vector>

namespace {

constexpr int MAXV = 8;       // variables per rule
constexpr int MAXA = 4;       // columns per relation
enum { SR_MAXPLUS = 0, SR_MINPLUS = 1, SR_LOGSUMEXP = 2, SR_SUMPROD = 3 };
enum { ST_OK = 0, ST_INVALID = 1, ST_UNSUPPORTED = 3, ST_CAPACITY = 5, ST_CONVERGENCE = 6 };

typedef std::array<int32_t, MAXA> Key;        // unused columns stay 0
typedef std::map<Key, float> Table;

struct Arg  { int kind; int var; int64_t mul, add, c; };          // kind 0: constant c; 1: column == mul*var+add
struct Atom { int rel; std::vector<Arg> args; bool neg = false; };
struct Expr { int64_t c0; int64_t coef[MAXV]; };
struct Rule { int head; std::vector<Atom> atoms; std::vector<Expr> head_cols; bool emit_count; };
struct Rel  { int arity; int sr; Table facts; Table rows; };

struct Acc {                       // contributions to one head tuple within one evaluation
  float best = 0.f; bool has = false;   // max / min
  std::vector<double> terms;            // logsumexp / sum
  int64_t count = 0;
};
typedef std::map<Key, Acc> AccTable;

struct Binding {                   // what the innermost loop level sees
  int64_t var[MAXV];
  const Table::value_type* row[4];
  float  tf;                       // fp32 left-to-right otimes
  double td;                       // fp64 left-to-right otimes
};

struct Engine {
  std::vector<Rel> rels;
  std::vector<Rule> rules;
  int status = ST_OK;
  int64_t iterations = 0, contributions = 0, delta_total = 0;
  std::vector<int64_t> delta_trace;          // |Delta| after the seed round and after every later round

  static bool better(int sr, float a, float b) {     // does a strictly improve on b ?
    return sr == SR_MAXPLUS ? a > b : a < b;
  }

  // Enumerate all bindings of `r`, atom j reading src[j].  Plain nested loops in
  // atom order; columns already fixed by constants / bound variables narrow the
  // scan with lower_bound on the sorted map (still the plain definition).
  void enumerate(const Rule& r, const Table* const* src, const std::function<void(const Binding&)>& cb) {
    Binding b;
    bool bound[MAXV];
    for (int v = 0; v < MAXV; ++v) { bound[v] = false; b.var[v] = 0; }
    const bool mul_sr = rels[r.head].sr == SR_SUMPROD;
    std::function<void(int, float, double)> level = [&](int j, float tf, double td) {
      if (j == (int)r.atoms.size()) { b.tf = tf; b.td = td; cb(b); return; }
      const Atom& a = r.atoms[j];
      const int k = rels[a.rel].arity;
      if (a.neg) {
        // negation as failure: does any stored row agree with every column that is fixed by now?
        bool exists = false;
        for (const auto& rowkv : *src[j]) {
          bool m = true;
          for (int c = 0; c < k && m; ++c) {
            const Arg& g = a.args[c];
            if (g.kind == 0) m = rowkv.first[c] == g.c;
            else if (bound[g.var]) m = g.mul * b.var[g.var] + g.add == rowkv.first[c];
          }
          if (m) { exists = true; break; }
        }
        if (!exists) { b.row[j] = nullptr; level(j + 1, tf, td); }
        return;
      }
      // leading columns whose value is already determined
      Key lo{}; int pre = 0;
      for (; pre < k; ++pre) {
        const Arg& g = a.args[pre];
        int64_t val;
        if (g.kind == 0) val = g.c;
        else if (bound[g.var]) val = g.mul * b.var[g.var] + g.add;
        else break;
        if (val < 0 || val > INT32_MAX) return;            // cannot match any stored row
        lo[pre] = (int32_t)val;
      }
      for (auto it = src[j]->lower_bound(lo); it != src[j]->end(); ++it) {
        const Key& row = it->first;
        bool in_prefix = true;
        for (int c = 0; c < pre; ++c) if (row[c] != lo[c]) { in_prefix = false; break; }
        if (!in_prefix) break;
        int newly[MAXA]; int n_new = 0; bool ok = true;
        for (int c = pre; c < k && ok; ++c) {
          const Arg& g = a.args[c];
          const int64_t val = row[c];
          if (g.kind == 0) ok = (val == g.c);
          else if (bound[g.var]) ok = (g.mul * b.var[g.var] + g.add == val);
          else {
            const int64_t d = val - g.add;
            if (d % g.mul != 0) ok = false;
            else { b.var[g.var] = d / g.mul; bound[g.var] = true; newly[n_new++] = g.var; }
          }
        }
        if (ok) {
          b.row[j] = &*it;
          const float t = it->second;
          if (j == 0) level(1, t, (double)t);
          else if (mul_sr) level(j + 1, tf * t, td * (double)t);
          else level(j + 1, tf + t, td + (double)t);
        }
        for (int i = 0; i < n_new; ++i) bound[newly[i]] = false;
      }
    };
    level(0, 0.f, 0.0);
  }

  bool head_key(const Rule& r, const Binding& b, Key& out) {
    out = Key{};
    for (size_t c = 0; c < r.head_cols.size(); ++c) {
      int64_t v = r.head_cols[c].c0;
      for (int i = 0; i < MAXV; ++i) v += r.head_cols[c].coef[i] * b.var[i];
      if (v < 0 || v > INT32_MAX) { status = ST_CAPACITY; return false; }
      out[c] = (int32_t)v;
    }
    return true;
  }

  void contribute(const Rule& r, const Table* const* src, AccTable& acc) {
    const int sr = rels[r.head].sr;
    enumerate(r, src, [&](const Binding& b) {
      Key k;
      if (!head_key(r, b, k)) return;
      Acc& a = acc[k];
      ++a.count; ++contributions;
      if (sr == SR_MAXPLUS || sr == SR_MINPLUS) {
        if (!a.has || better(sr, b.tf, a.best)) { a.best = b.tf; a.has = true; }
      } else {
        a.terms.push_back(b.td);
      }
    });
  }

  static float finish(int sr, const Acc& a) {
    if (sr == SR_MAXPLUS || sr == SR_MINPLUS) return a.best;
    if (sr == SR_LOGSUMEXP) {
      double m = -std::numeric_limits<double>::infinity();
      for (double v : a.terms) m = std::max(m, v);
      double s = 0.0;
      for (double v : a.terms) s += std::exp(v - m);
      return (float)(m + std::log(s));
    }
    double s = 0.0;
    for (double v : a.terms) s += v;
    return (float)s;
  }

  // ---- strata ---------------------------------------------------------------
  std::vector<std::vector<int>> components() {        // Tarjan; emitted in dependency order
    const int n = (int)rels.size();
    std::vector<std::set<int>> dep(n);                 // head -> body relations
    for (const Rule& r : rules) for (const Atom& a : r.atoms) dep[r.head].insert(a.rel);
    std::vector<int> idx(n, -1), low(n, 0), stack; std::vector<bool> on(n, false);
    std::vector<std::vector<int>> out; int counter = 0;
    std::function<void(int)> visit = [&](int v) {
      idx[v] = low[v] = counter++; stack.push_back(v); on[v] = true;
      for (int w : dep[v]) {
        if (idx[w] < 0) { visit(w); low[v] = std::min(low[v], low[w]); }
        else if (on[w]) low[v] = std::min(low[v], idx[w]);
      }
      if (low[v] == idx[v]) {
        std::vector<int> comp;
        for (;;) { int w = stack.back(); stack.pop_back(); on[w] = false; comp.push_back(w); if (w == v) break; }
        std::sort(comp.begin(), comp.end());
        out.push_back(comp);                           // a component is emitted after everything it depends on
      }
    };
    for (int v = 0; v < n; ++v) if (idx[v] < 0) visit(v);
    return out;
  }

  int run(int mode, int64_t max_iter) {
    status = ST_OK; iterations = contributions = delta_total = 0; delta_trace.clear();
    for (const std::vector<int>& comp : components()) {
      std::set<int> in(comp.begin(), comp.end());
      std::vector<const Rule*> rs;
      for (const Rule& r : rules) if (in.count(r.head)) rs.push_back(&r);
      if (rs.empty()) { for (int p : comp) rels[p].rows = rels[p].facts; continue; }   // loaded facts only
      bool recursive = comp.size() > 1;
      for (const Rule* r : rs) for (const Atom& a : r->atoms) if (in.count(a.rel)) { recursive = true; if (a.neg) return status = ST_UNSUPPORTED; }
      if (!recursive) stratum_once(comp[0], rs);
      else {
        int idem = 0, additive = 0;
        for (int p : comp) { if (rels[p].sr == SR_MAXPLUS || rels[p].sr == SR_MINPLUS) ++idem; else ++additive; }
        if (idem && additive) return status = ST_UNSUPPORTED;
        for (const Rule* r : rs) if (r->emit_count) return status = ST_UNSUPPORTED;
        if (additive) {
          if (mode == 0) additive_naive(in, rs, max_iter);
          else {
            // the delta form below needs T to be linear in the component's relations: at most one recursive atom per rule
            for (const Rule* r : rs) { int k = 0; for (const Atom& a : r->atoms) if (in.count(a.rel)) ++k; if (k > 1) return status = ST_UNSUPPORTED; }
            additive_seminaive(in, rs, max_iter);
          }
        } else if (mode == 0) recursive_naive(in, rs, max_iter); else recursive_seminaive(in, rs, max_iter);
      }
      if (status != ST_OK) return status;
    }
    return status;
  }

  std::vector<const Table*> full_sources(const Rule& r) {
    std::vector<const Table*> s;
    for (const Atom& a : r.atoms) s.push_back(&rels[a.rel].rows);
    return s;
  }

  // I(P) = facts(P) oplus (oplus_r T_r), every rule evaluated once.
  void stratum_once(int p, const std::vector<const Rule*>& rs) {
    Rel& P = rels[p];
    const bool counted = rs[0]->emit_count;
    for (const Rule* r : rs) if (r->emit_count != counted) { status = ST_UNSUPPORTED; return; }
    if (counted && !P.facts.empty()) { status = ST_UNSUPPORTED; return; }
    AccTable acc;
    for (const Rule* r : rs) { auto s = full_sources(*r); contribute(*r, s.data(), acc); if (status) return; }
    for (const auto& f : P.facts) {                        // loaded facts are one more contribution each
      Acc& a = acc[f.first];
      if (P.sr == SR_MAXPLUS || P.sr == SR_MINPLUS) { if (!a.has || better(P.sr, f.second, a.best)) { a.best = f.second; a.has = true; } }
      else a.terms.push_back((double)f.second);
    }
    P.rows.clear();
    for (const auto& e : acc) {
      Key k = e.first;
      if (counted) {
        if (e.second.count > INT32_MAX) { status = ST_CAPACITY; return; }
        k[rs[0]->head_cols.size()] = (int32_t)e.second.count;
      }
      P.rows.emplace_hint(P.rows.end(), k, finish(P.sr, e.second));
    }
    iterations += 1;
  }

  // Naive rounds on a snapshot:  I_{k+1} = I_k oplus T(I_k), until I_{k+1} == I_k.
  void recursive_naive(const std::set<int>& in, const std::vector<const Rule*>& rs, int64_t max_iter) {
    for (int64_t round = 0;; ++round) {
      if (round >= max_iter) { status = ST_CONVERGENCE; return; }
      std::map<int, AccTable> acc;
      for (const Rule* r : rs) { auto s = full_sources(*r); contribute(*r, s.data(), acc[r->head]); if (status) return; }
      bool changed = false;
      for (int p : in) {
        Rel& P = rels[p];
        for (const auto& e : acc[p]) {
          auto it = P.rows.find(e.first);
          if (it == P.rows.end()) { P.rows.emplace(e.first, e.second.best); changed = true; }
          else if (better(P.sr, e.second.best, it->second)) { it->second = e.second.best; changed = true; }
        }
      }
      ++iterations;
      if (!changed) return;
    }
  }

  // Algorithm 1 with tag improvement: seed with every atom reading the full
  // relation, then one Delta-variant per recursive atom occurrence per round.
  void recursive_seminaive(const std::set<int>& in, const std::vector<const Rule*>& rs, int64_t max_iter) {
    std::map<int, Table> delta;
    auto absorb = [&](std::map<int, AccTable>& acc) {
      std::map<int, Table> nd; int64_t n = 0;
      for (int p : in) {
        Rel& P = rels[p];
        for (const auto& e : acc[p]) {
          auto it = P.rows.find(e.first);
          if (it == P.rows.end()) { P.rows.emplace(e.first, e.second.best); nd[p].emplace(e.first, e.second.best); }
          else if (better(P.sr, e.second.best, it->second)) { it->second = e.second.best; nd[p].emplace(e.first, e.second.best); }
        }
        n += (int64_t)nd[p].size();
      }
      delta.swap(nd); delta_total += n; delta_trace.push_back(n);
      return n;
    };
    {
      std::map<int, AccTable> acc;
      for (const Rule* r : rs) { auto s = full_sources(*r); contribute(*r, s.data(), acc[r->head]); if (status) return; }
      ++iterations;
      if (absorb(acc) == 0) return;
    }
    for (int64_t round = 1;; ++round) {
      if (round >= max_iter) { status = ST_CONVERGENCE; return; }
      std::map<int, AccTable> acc;
      for (const Rule* r : rs)
        for (size_t i = 0; i < r->atoms.size(); ++i) {
          if (!in.count(r->atoms[i].rel) || r->atoms[i].neg) continue;
          auto s = full_sources(*r);
          s[i] = &delta[r->atoms[i].rel];
          contribute(*r, s.data(), acc[r->head]);
          if (status) return;
        }
      ++iterations;
      if (absorb(acc) == 0) return;
    }
  }

  // Non-idempotent oplus inside a recursive component, naive form:  I_0 = facts,  I_{k+1} = facts oplus T(I_k).
  void additive_naive(const std::set<int>& in, const std::vector<const Rule*>& rs, int64_t max_iter) {
    for (int p : in) rels[p].rows = rels[p].facts;
    for (int64_t round = 0;; ++round) {
      if (round >= max_iter) { status = ST_CONVERGENCE; return; }
      std::map<int, AccTable> acc;
      for (const Rule* r : rs) { auto s = full_sources(*r); contribute(*r, s.data(), acc[r->head]); if (status) return; }
      bool changed = false;
      for (int p : in) {
        Rel& P = rels[p];
        for (const auto& f : P.facts) acc[p][f.first].terms.push_back((double)f.second);
        Table next;
        for (const auto& e : acc[p]) next.emplace_hint(next.end(), e.first, finish(P.sr, e.second));
        if (next.size() != P.rows.size()) changed = true;
        else for (auto a = next.begin(), b = P.rows.begin(); a != next.end(); ++a, ++b)
          if (a->first != b->first || std::memcmp(&a->second, &b->second, sizeof(float)) != 0) { changed = true; break; }
        P.rows.swap(next);
      }
      ++iterations;
      if (!changed) return;
    }
  }

  // The same fixpoint in delta form (Algorithm 1 with the delta carrying tag DIFFERENCES).  T is linear in the
  // component's relations (one recursive atom per rule), so  I_{k+1} - I_k = T_rec(I_k - I_{k-1}):
  //   Delta_1 = T(facts)  (every atom reads the full relation),  Delta_{k+1} = T_rec(Delta_k),  I_{k+1} = I_k oplus Delta_{k+1},
  // until a round derives nothing at all.  Each round's sums are taken in fp64 and rounded once; the running relation is fp32.
  void additive_seminaive(const std::set<int>& in, const std::vector<const Rule*>& rs, int64_t max_iter) {
    for (int p : in) rels[p].rows = rels[p].facts;
    std::map<int, Table> delta;
    auto absorb = [&](std::map<int, AccTable>& acc) {
      std::map<int, Table> nd; int64_t n = 0;
      for (int p : in) {
        Rel& P = rels[p];
        for (const auto& e : acc[p]) {
          const float d = finish(P.sr, e.second);
          nd[p].emplace_hint(nd[p].end(), e.first, d);
          auto it = P.rows.find(e.first);
          if (it == P.rows.end()) P.rows.emplace(e.first, d);
          else {
            Acc two; two.terms.push_back((double)it->second); two.terms.push_back((double)d);
            it->second = finish(P.sr, two);
          }
        }
        n += (int64_t)nd[p].size();
      }
      delta.swap(nd); delta_total += n; delta_trace.push_back(n);
      return n;
    };
    {
      std::map<int, AccTable> acc;
      for (const Rule* r : rs) { auto s = full_sources(*r); contribute(*r, s.data(), acc[r->head]); if (status) return; }
      ++iterations;
      if (absorb(acc) == 0) return;
    }
    for (int64_t round = 1;; ++round) {
      if (round >= max_iter) { status = ST_CONVERGENCE; return; }
      std::map<int, AccTable> acc;
      for (const Rule* r : rs)
        for (size_t i = 0; i < r->atoms.size(); ++i) {
          if (!in.count(r->atoms[i].rel) || r->atoms[i].neg) continue;
          auto s = full_sources(*r);
          s[i] = &delta[r->atoms[i].rel];
          contribute(*r, s.data(), acc[r->head]);
          if (status) return;
        }
      ++iterations;
      if (absorb(acc) == 0) return;
    }
  }

  // Gradient of a non-recursive LOGSUMEXP / SUMPROD rule with respect to the tags
  // of its body atoms, given g over the head rows in stored order:
  //   LOGSUMEXP:  grad_j[row] += g[h] * exp(sum_i tag_i - out[h])
  //   SUMPROD:    grad_j[row] += g[h] * prod_{i != j} tag_i
  // accumulated in fp64, rounded once.  Rows follow each relation's sorted order.
  int backward(int rule_id, const float* g, float* const* grads) {
    const Rule& r = rules[rule_id];
    const Rel& H = rels[r.head];
    if (H.sr != SR_LOGSUMEXP && H.sr != SR_SUMPROD) return ST_UNSUPPORTED;
    const size_t nd = r.head_cols.size();
    std::map<Key, int64_t> head_index;                   // declared head columns -> stored row
    { int64_t i = 0; for (const auto& e : H.rows) { Key k = e.first; if (r.emit_count) k[nd] = 0; head_index[k] = i++; } }
    std::vector<std::map<Key, int64_t>> row_index(r.atoms.size());
    std::vector<std::vector<double>> acc(r.atoms.size());
    for (size_t j = 0; j < r.atoms.size(); ++j) {
      int64_t i = 0; for (const auto& e : rels[r.atoms[j].rel].rows) row_index[j][e.first] = i++;
      acc[j].assign(rels[r.atoms[j].rel].rows.size(), 0.0);
    }
    std::vector<double> out; for (const auto& e : H.rows) out.push_back((double)e.second);
    auto s = full_sources(r);
    status = ST_OK;
    enumerate(r, s.data(), [&](const Binding& b) {
      Key k; if (!head_key(r, b, k)) return;
      const int64_t h = head_index.at(k);
      for (size_t j = 0; j < r.atoms.size(); ++j) {
        if (r.atoms[j].neg) continue;                      // a negated atom carries no tag
        double w;
        if (H.sr == SR_LOGSUMEXP) w = std::exp(b.td - out[h]);
        else { w = 1.0; for (size_t i = 0; i < r.atoms.size(); ++i) if (i != j && !r.atoms[i].neg) w *= (double)b.row[i]->second; }
        acc[j][row_index[j].at(b.row[j]->first)] += (double)g[h] * w;
      }
    });
    for (size_t j = 0; j < r.atoms.size(); ++j)
      for (size_t i = 0; i < acc[j].size(); ++i) grads[j][i] = (float)acc[j][i];
    return status;
  }
};

float zero_of(int sr) {
  return sr == SR_MAXPLUS || sr == SR_LOGSUMEXP ? -std::numeric_limits<float>::infinity()
       : sr == SR_MINPLUS ? std::numeric_limits<float>::infinity() : 0.f;
}
float one_of(int sr) { return sr == SR_SUMPROD ? 1.f : 0.f; }

}  // namespace

extern "C" {

void* orc_create() { return new Engine(); }
void orc_destroy(void* e) { delete (Engine*)e; }

int orc_relation(void* e, int arity, int sr) {
  Engine* E = (Engine*)e;
  if (arity < 1 || arity > MAXA || sr < 0 || sr > 3) return -1;
  Rel r; r.arity = arity; r.sr = sr; E->rels.push_back(r);
  return (int)E->rels.size() - 1;
}

// rows: row-major [n, arity]; tags NULL => every tag is the semiring's one.
// Duplicate keys combine with the relation's oplus.  Replaces earlier contents.
int orc_load(void* e, int rel, const int32_t* rows, const float* tags, int64_t n) {
  Engine* E = (Engine*)e; Rel& R = E->rels[rel];
  std::map<Key, std::vector<double>> multi;
  R.facts.clear();
  for (int64_t i = 0; i < n; ++i) {
    Key k{}; for (int c = 0; c < R.arity; ++c) { k[c] = rows[i * R.arity + c]; if (k[c] < 0) return ST_INVALID; }
    float t = tags ? tags[i] : one_of(R.sr);
    if (std::isnan(t) || (t == zero_of(R.sr) && R.sr != SR_SUMPROD)) return ST_INVALID;
    if (t == 0.f) t = 0.f;                                // -0.0 -> +0.0
    if (R.sr == SR_MAXPLUS || R.sr == SR_MINPLUS) {
      auto it = R.facts.find(k);
      if (it == R.facts.end()) R.facts.emplace_hint(R.facts.end(), k, t);
      else if (Engine::better(R.sr, t, it->second)) it->second = t;
    } else multi[k].push_back((double)t);
  }
  for (auto& m : multi) { Acc a; a.terms = m.second; R.facts[m.first] = Engine::finish(R.sr, a); }
  R.rows = R.facts;
  return ST_OK;
}

// atom_args: per atom, per column, 4 values (kind, var, mul, add-or-constant), MAXA columns reserved per atom.
// head_exprs: per head column, 1 + MAXV values (c0, coef[0..MAXV-1]).
int orc_rule(void* e, int head, int n_head_cols, const int64_t* head_exprs, int n_atoms,
             const int32_t* atom_rel, const int64_t* atom_args, int emit_count, const int32_t* atom_neg) {
  Engine* E = (Engine*)e; Rule r; r.head = head; r.emit_count = emit_count != 0;
  if (n_atoms < 1 || n_atoms > 4) return -1;
  for (int c = 0; c < n_head_cols; ++c) {
    Expr x; x.c0 = head_exprs[c * (1 + MAXV)];
    for (int v = 0; v < MAXV; ++v) x.coef[v] = head_exprs[c * (1 + MAXV) + 1 + v];
    r.head_cols.push_back(x);
  }
  if ((int)r.head_cols.size() + (r.emit_count ? 1 : 0) != E->rels[head].arity) return -1;
  for (int j = 0; j < n_atoms; ++j) {
    Atom a; a.rel = atom_rel[j]; a.neg = atom_neg && atom_neg[j];
    if (a.neg && j == 0) return -1;                        // the first atom binds the variables
    for (int c = 0; c < E->rels[a.rel].arity; ++c) {
      const int64_t* p = atom_args + (j * MAXA + c) * 4;
      Arg g; g.kind = (int)p[0]; g.var = (int)p[1]; g.mul = p[2]; g.add = p[3]; g.c = p[3];
      if (g.kind == 1 && (g.var < 0 || g.var >= MAXV || g.mul <= 0)) return -1;
      a.args.push_back(g);
    }
    r.atoms.push_back(a);
  }
  E->rules.push_back(r);
  return (int)E->rules.size() - 1;
}

void orc_reset(void* e) { Engine* E = (Engine*)e; for (Rel& r : E->rels) r.rows = r.facts; }

// stats: [iterations, contributions, delta_total, derived_tuples]
int orc_run(void* e, int mode, int64_t max_iter, int64_t* stats) {
  Engine* E = (Engine*)e;
  int st = E->run(mode, max_iter);
  if (stats) {
    stats[0] = E->iterations; stats[1] = E->contributions; stats[2] = E->delta_total;
    int64_t derived = 0;
    std::set<int> heads; for (const Rule& r : E->rules) heads.insert(r.head);
    for (int p : heads) derived += (int64_t)E->rels[p].rows.size() - (int64_t)E->rels[p].facts.size();
    stats[3] = derived;
  }
  return st;
}

int64_t orc_delta_trace(void* e, int64_t* out, int64_t cap) {
  Engine* E = (Engine*)e;
  for (int64_t i = 0; i < (int64_t)E->delta_trace.size() && i < cap; ++i) out[i] = E->delta_trace[i];
  return (int64_t)E->delta_trace.size();
}

int64_t orc_size(void* e, int rel) { return (int64_t)((Engine*)e)->rels[rel].rows.size(); }

// rows out: row-major [n, arity], ascending lexicographic order.
void orc_read(void* e, int rel, int32_t* rows, float* tags) {
  Rel& R = ((Engine*)e)->rels[rel]; int64_t i = 0;
  for (const auto& r : R.rows) { for (int c = 0; c < R.arity; ++c) rows[i * R.arity + c] = r.first[c]; tags[i] = r.second; ++i; }
}

int orc_backward(void* e, int rule, const float* g, float* const* grads) { return ((Engine*)e)->backward(rule, g, grads); }

}  // extern "C"
