// Snapshot and restore of one unit's cache state [Migration-Stable Quantization: the write-once ledger is a
// persistent low-bit store -- codes produced at a window's first demotion stay valid for its whole life, so a
// cache can be put away and brought back without requantizing anything].
//
// A snapshot is everything the routing and attention kernels read for one (layer, sequence) pair: the window
// tables, the page-owner tables, the decode work list, the unit's pages of both pools (in the library's own
// page layout -- opaque to the caller, valid for a cache of the same configuration) and the host's mirror of
// the layer.  Scratch (split partials) and the device status word are not part of it.
#include <stdlib.h>
#include <string.h>

#include <string>

#include "ctx.h"

using namespace qevict;

namespace {

qevict_status fail(qevict_handle h, qevict_status s, const char* msg) {
  h->last_error = msg;
  return s;
}

bool unit_of(qevict_handle h, int layer, int seq, size_t* u) {
  if (layer < 0 || layer >= h->geo.n_layers || seq < 0 || seq >= h->geo.batch) return false;
  *u = (size_t)layer * h->geo.batch + seq;
  return true;
}

const char* missing_array(const qevict_state_view* v) {
  if (!v->tier || !v->ledger || !v->fp_page || !v->q_page || !v->importance || !v->event_mass) return "a window table pointer of the view is NULL";
  if (!v->fp_owner || !v->q_owner || !v->entries || !v->last_mass) return "an owner / work-list pointer of the view is NULL";
  if (!v->fp_pool || !v->q_pool) return "a pool pointer of the view is NULL";
  return nullptr;
}

#define ST_CUDA(h, expr)                                                                 \
  do {                                                                                   \
    cudaError_t e__ = (expr);                                                            \
    if (e__ != cudaSuccess) {                                                            \
      (h)->last_error = std::string(#expr) + ": " + cudaGetErrorString(e__);             \
      return QEVICT_ERR_CUDA;                                                            \
    }                                                                                    \
  } while (0)

}  // namespace

extern "C" {

QEVICT_API qevict_status qevict_state_layout_of(qevict_handle h, qevict_state_layout* out) {
  if (!h || !out) return QEVICT_ERR_INVALID_ARG;
  const Geometry& g = h->geo;
  out->n_window_slots = g.NW;
  out->n_fp_pages = g.PF;
  out->n_q_pages = g.PQ;
  out->n_entries = g.EMAX;
  out->fp_pool_bytes = (uint64_t)g.PF * g.fp_page_bytes;
  out->q_pool_bytes = (uint64_t)g.PQ * g.q_page_bytes;
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_export_state(qevict_handle h, int32_t layer, int32_t seq, qevict_state_view* v) {
  if (!h || !v) return QEVICT_ERR_INVALID_ARG;
  if (v->struct_size != sizeof(qevict_state_view)) return fail(h, QEVICT_ERR_INVALID_ARG, "struct_size does not match this library's qevict_state_view");
  size_t u;
  if (!unit_of(h, layer, seq, &u)) return fail(h, QEVICT_ERR_INVALID_ARG, "layer or seq out of range");
  if (const char* m = missing_array(v)) return fail(h, QEVICT_ERR_INVALID_ARG, m);
  const Geometry& g = h->geo;
  const State& st = h->st;
  DeviceGuard guard(h->cfg.device);
  ST_CUDA(h, guard.err);
  ST_CUDA(h, cudaDeviceSynchronize());
  const size_t NW = g.NW;
  auto d2h = [](void* dst, const void* src, size_t n) { return cudaMemcpy(dst, src, n, cudaMemcpyDeviceToHost); };
  ST_CUDA(h, d2h(&v->n_windows, st.n_windows + u, 4));
  ST_CUDA(h, d2h(&v->open_window, st.open_window + u, 4));
  ST_CUDA(h, d2h(&v->open_fill, st.open_fill + u, 4));
  ST_CUDA(h, d2h(&v->n_live, st.n_live + u, 4));
  ST_CUDA(h, d2h(&v->knorm_acc, st.knorm_acc + u, 4));
  ST_CUDA(h, d2h(v->counters, st.counters + u * 4, 32));
  ST_CUDA(h, d2h(v->tier, st.tier + u * NW, NW));
  ST_CUDA(h, d2h(v->ledger, st.ledger + u * NW, NW));
  ST_CUDA(h, d2h(v->fp_page, st.fp_page + u * NW, NW * 4));
  ST_CUDA(h, d2h(v->q_page, st.q_page + u * NW, NW * 4));
  ST_CUDA(h, d2h(v->importance, st.importance + u * NW, NW * 4));
  ST_CUDA(h, d2h(v->event_mass, st.event_mass + u * NW, NW * 4));
  ST_CUDA(h, d2h(v->fp_owner, st.fp_owner + u * g.PF, (size_t)g.PF * 4));
  ST_CUDA(h, d2h(v->q_owner, st.q_owner + u * g.PQ, (size_t)g.PQ * 4));
  ST_CUDA(h, d2h(v->entries, st.entries + u * g.EMAX, (size_t)g.EMAX * 8));
  ST_CUDA(h, d2h(v->last_mass, st.mass_e + u * g.EMAX, (size_t)g.EMAX * 4));
  ST_CUDA(h, d2h(v->fp_pool, st.fp_pool + u * g.PF * (size_t)g.fp_page_bytes, (size_t)g.PF * g.fp_page_bytes));
  ST_CUDA(h, d2h(v->q_pool, st.q_pool + u * g.PQ * (size_t)g.q_page_bytes, (size_t)g.PQ * g.q_page_bytes));
  const LayerMirror& m = h->layers[layer];
  v->layer_prefilled = m.prefilled ? 1 : 0;
  v->layer_has_open = m.has_open ? 1 : 0;
  v->layer_open_fill = m.open_fill;
  v->layer_n_windows = m.n_windows;
  v->layer_aged = m.aged;
  v->decode_steps = h->decode_steps;
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_import_state(qevict_handle h, int32_t layer, int32_t seq, const qevict_state_view* v) {
  if (!h || !v) return QEVICT_ERR_INVALID_ARG;
  if (v->struct_size != sizeof(qevict_state_view)) return fail(h, QEVICT_ERR_INVALID_ARG, "struct_size does not match this library's qevict_state_view");
  size_t u;
  if (!unit_of(h, layer, seq, &u)) return fail(h, QEVICT_ERR_INVALID_ARG, "layer or seq out of range");
  if (const char* m = missing_array(v)) return fail(h, QEVICT_ERR_INVALID_ARG, m);
  if (h->broken) return fail(h, QEVICT_ERR_BAD_STATE, "an earlier call failed after it had started to enqueue work: destroy this cache");
  const Geometry& g = h->geo;
  // ---- everything a kernel would use as an index is checked before anything is written -----------------------
  if (!v->layer_prefilled) return fail(h, QEVICT_ERR_INVALID_ARG, "the snapshot was taken before prefill_assign");
  if (v->n_windows < 0 || v->n_windows > g.NW || v->open_window < -1 || v->open_window >= v->n_windows ||
      v->open_fill < 0 || v->open_fill >= g.W || v->n_live < 0 || v->n_live > g.EMAX)
    return fail(h, QEVICT_ERR_INVALID_ARG, "a scalar of the snapshot is out of range for this configuration");
  if (v->layer_n_windows != v->n_windows || (v->layer_has_open != 0) != (v->open_window >= 0) ||
      v->layer_open_fill != v->open_fill || v->layer_aged < 0 || v->layer_aged > g.aged_cap + 1)
    return fail(h, QEVICT_ERR_INVALID_ARG, "the layer mirror of the snapshot disagrees with its tables");
#ifdef QEVICT_DEBUG_BOUNDS
  // checking build only: with QEVICT_IMPORT_UNCHECKED set in the environment the index checks below are left
  // out, so that a test can hand the kernels a table entry that is out of range and see their own checks refuse it
  const bool unchecked = getenv("QEVICT_IMPORT_UNCHECKED") != nullptr;
#else
  const bool unchecked = false;
#endif
  for (int w = 0; w < g.NW && !unchecked; ++w) {
    if (v->tier[w] > QEVICT_TIER_SINK || v->ledger[w] > QEVICT_LEDGER_DORMANT || v->fp_page[w] < -1 || v->fp_page[w] >= g.PF ||
        v->q_page[w] < -1 || v->q_page[w] >= g.PQ)
      return fail(h, QEVICT_ERR_INVALID_ARG, "a window table entry of the snapshot is out of range");
  }
  for (int p = 0; p < g.PF && !unchecked; ++p)
    if (v->fp_owner[p] < -1 || v->fp_owner[p] >= g.NW) return fail(h, QEVICT_ERR_INVALID_ARG, "a full-precision page owner of the snapshot is out of range");
  for (int p = 0; p < g.PQ && !unchecked; ++p)
    if (v->q_owner[p] < -1 || v->q_owner[p] >= g.NW) return fail(h, QEVICT_ERR_INVALID_ARG, "a quantized page owner of the snapshot is out of range");
  for (int e = 0; e < v->n_live && !unchecked; ++e) {
    const uint32_t x = v->entries[2 * e], page = v->entries[2 * e + 1], kind = x >> ENTRY_KIND_SHIFT;
    if (kind > KIND_OPEN || (int)(x & ENTRY_WINDOW_MASK) >= g.NW || (int)page >= (kind == KIND_Q ? g.PQ : g.PF))
      return fail(h, QEVICT_ERR_INVALID_ARG, "a work-list entry of the snapshot is out of range");
  }
  // the sequences of a layer step together: the mirror is per layer, so a snapshot must agree with what the layer
  // already holds (from prefill_assign or from the import of another sequence)
  LayerMirror& m = h->layers[layer];
  if (m.prefilled && (m.has_open != (v->layer_has_open != 0) || m.open_fill != v->layer_open_fill ||
                      m.n_windows != v->layer_n_windows || m.aged != v->layer_aged))
    return fail(h, QEVICT_ERR_BAD_STATE, "the snapshot's position (windows, open fill, aged windows) differs from the layer's other sequences");
  const State& st = h->st;
  DeviceGuard guard(h->cfg.device);
  ST_CUDA(h, guard.err);
  ST_CUDA(h, cudaDeviceSynchronize());
  const size_t NW = g.NW;
  auto h2d = [](void* dst, const void* src, size_t n) { return cudaMemcpy(dst, src, n, cudaMemcpyHostToDevice); };
  ST_CUDA(h, h2d(st.n_windows + u, &v->n_windows, 4));
  ST_CUDA(h, h2d(st.open_window + u, &v->open_window, 4));
  ST_CUDA(h, h2d(st.open_fill + u, &v->open_fill, 4));
  ST_CUDA(h, h2d(st.n_live + u, &v->n_live, 4));
  ST_CUDA(h, h2d(st.knorm_acc + u, &v->knorm_acc, 4));
  ST_CUDA(h, h2d(st.counters + u * 4, v->counters, 32));
  ST_CUDA(h, h2d(st.tier + u * NW, v->tier, NW));
  ST_CUDA(h, h2d(st.ledger + u * NW, v->ledger, NW));
  ST_CUDA(h, h2d(st.fp_page + u * NW, v->fp_page, NW * 4));
  ST_CUDA(h, h2d(st.q_page + u * NW, v->q_page, NW * 4));
  ST_CUDA(h, h2d(st.importance + u * NW, v->importance, NW * 4));
  ST_CUDA(h, h2d(st.event_mass + u * NW, v->event_mass, NW * 4));
  ST_CUDA(h, h2d(st.fp_owner + u * g.PF, v->fp_owner, (size_t)g.PF * 4));
  ST_CUDA(h, h2d(st.q_owner + u * g.PQ, v->q_owner, (size_t)g.PQ * 4));
  ST_CUDA(h, h2d(st.entries + u * g.EMAX, v->entries, (size_t)g.EMAX * 8));
  ST_CUDA(h, h2d(st.mass_e + u * g.EMAX, v->last_mass, (size_t)g.EMAX * 4));
  ST_CUDA(h, h2d(st.fp_pool + u * g.PF * (size_t)g.fp_page_bytes, v->fp_pool, (size_t)g.PF * g.fp_page_bytes));
  ST_CUDA(h, h2d(st.q_pool + u * g.PQ * (size_t)g.q_page_bytes, v->q_pool, (size_t)g.PQ * g.q_page_bytes));
  m.prefilled = true;
  m.has_open = v->layer_has_open != 0;
  m.open_fill = v->layer_open_fill;
  m.n_windows = v->layer_n_windows;
  m.aged = v->layer_aged;
  if (v->decode_steps > h->decode_steps) h->decode_steps = v->decode_steps;
  return QEVICT_OK;
}

}  // extern "C"
