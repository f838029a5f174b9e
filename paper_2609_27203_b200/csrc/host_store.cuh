// Relation store on the host side: load (validate, pack, sort, combine duplicates), column views, key re-layout, join indices.
// Host-side driver code of the engine; included by xlog_api.cu only (one translation unit).
#pragma once
#include "engine.cuh"

namespace xlog {
namespace {

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

}  // namespace
}  // namespace xlog
