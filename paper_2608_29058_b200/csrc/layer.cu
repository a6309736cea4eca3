// One call for the whole hot path of a layer (the procedure table of Section 3.4): probe, candidate evaluation,
// routing, materialisation of the routed block-sparse rows, one sparse attention launch, certificate.  Host code only:
// it enqueues the library's own entry points on the caller's stream in the order below; no host decision sits between
// the steps (the routes stay on the device), so the call returns before any kernel has run and can be captured into a
// CUDA graph.
#include "common.cuh"

extern "C" int rs_routed_prefill_layer(const rs_problem* p, const void* Q, const void* K, const void* V,
                                       const rs_candidate* lib, int n_cand, const rs_route_params* params,
                                       const int64_t* cost, const rs_layer_buffers* b, void* ws, size_t ws_bytes,
                                       int32_t* status, void* stream) {
  int rc = rs_check_problem(p);
  if (rc != RS_OK) return rc;
  if (!Q || !K || !V || !lib || n_cand <= 0 || n_cand > RS_MAX_CANDIDATES || !params || !b || !ws) return RS_ERR_INVALID_ARG;
  if (!b->vert || !b->slash || !b->lse_probe || !b->qpool || !b->kpool || !b->vmax || !b->stats || !b->choice ||
      !b->O || !b->lse_sel)
    return RS_ERR_INVALID_ARG;
  const int n_items = p->n_segments * p->n_q_heads;
  const bool online = params->fixed_choice == nullptr;
  if (online && b->idx_eval.n_vs_slots < n_items * n_cand) {
    bool any_vs = false;
    for (int c = 0; c < n_cand; ++c) any_vs |= lib[c].pattern == RS_VERTICAL_SLASH;
    if (any_vs) return RS_ERR_INVALID_ARG;             // online routing needs the evaluation layout
  }

  // 1. shared probe; all of Q is pooled only later, for the heads that are routed to block-sparse
  rc = rs_probe(p, Q, K, V, b->vert, b->slash, b->lse_probe, b->qpool, b->kpool, b->vmax, b->descr,
                RS_PROBE_QPOOL_LAST_ONLY, ws, ws_bytes, status, stream);
  if (rc != RS_OK) return rc;

  // 2. every candidate's index lists, coverage and pair count;  3. Eq. 4, Eq. 6-8, fallback
  if (online) {
    rc = rs_build_indices(p, lib, n_cand, b->vert, b->slash, b->qpool, b->kpool, nullptr, nullptr, &b->idx_eval,
                          b->stats, ws, ws_bytes, status, stream);
    if (rc != RS_OK) return rc;
  }
  rc = rs_route(p, lib, n_cand, online ? b->stats : nullptr, cost, b->vmax, params, b->choice, b->report, status, stream);
  if (rc != RS_OK) return rc;

  // 4. pooled queries of the block-sparse heads, then the routed index lists.  Online, the vertical-slash lists of the
  // evaluation are reused (n_vs_slots = 0 builds block-sparse rows only) and the attention call reads them in place.
  rc = rs_pool_queries(p, Q, lib, n_cand, b->choice, b->qpool, status, stream);
  if (rc != RS_OK) return rc;
  const bool reuse = online && n_cand > 1;
  rs_index_set mat = b->idx;
  if (reuse) mat.n_vs_slots = 0;
  rc = rs_build_indices(p, lib, n_cand, b->vert, b->slash, b->qpool, b->kpool, nullptr, b->choice, &mat, nullptr, ws,
                        ws_bytes, status, stream);
  if (rc != RS_OK) return rc;
  rs_index_set att = b->idx;
  if (reuse) {
    att.n_vs_slots = b->idx_eval.n_vs_slots; att.kv_cap = b->idx_eval.kv_cap; att.ks_cap = b->idx_eval.ks_cap;
    att.nd_cap = b->idx_eval.nd_cap;
    att.vs_cols = b->idx_eval.vs_cols; att.vs_offs = b->idx_eval.vs_offs; att.vs_diag = b->idx_eval.vs_diag;
    att.vs_count = b->idx_eval.vs_count;
  }

  // 5. one launch for all heads and segments
  rc = rs_sparse_prefill_attn(p, Q, K, V, lib, n_cand, &att, b->choice, b->O, b->o_dtype, b->lse_sel, b->onorm,
                              b->counters, ws, ws_bytes, status, stream);
  if (rc != RS_OK) return rc;

  // 6. Eq. 5 on the probe rows (skipped when the caller passes no rows)
  if (b->probe_rows != nullptr && b->n_probe_rows > 0 && b->onorm != nullptr) {
    rc = rs_certificate(p->n_q_heads, p->n_kv_heads, p->n_keys, b->lse_sel, b->lse_probe, b->probe_rows, b->n_probe_rows,
                        b->vmax + (size_t)(p->n_segments - 1) * p->n_kv_heads, b->onorm, (float)params->delta_q,
                        b->m_row, b->cert_row, nullptr, b->m_head, b->cert_head, status, stream);
  }
  return rc;
}
