// Gradient of a non-recursive logsumexp / sum rule.
// Host-side driver code of the engine; included by xlog_api.cu only (one translation unit).
#pragma once
#include "host_eval.cuh"

namespace xlog {
namespace {

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

}  // namespace
}  // namespace xlog
