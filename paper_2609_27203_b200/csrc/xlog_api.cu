// C ABI of the engine (see include/xlog.h): entry points only; the host-side driver lives in the host_*.cuh headers.
#include "engine.cuh"
#include "host_strata.cuh"

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
