// Decode step for callers that must not allocate device memory.
//
// qevict_decode_attn_noalloc computes exactly what qevict_decode_attn computes, with the same kernels,
// but the attention kernel's scratch -- the per-split partial outputs, their (max, sum) pairs and the
// per-(head, window) softmax numerators that the combine kernel reads back -- lives in a fixed array
// inside this library's device image instead of in memory that somebody had to allocate.
#include <stdio.h>

#include "ctx.h"

using namespace qevict;

namespace {

// The scratch array.  Every GPU that loads the library carries these bytes until the process exits.
constexpr size_t NOALLOC_SCRATCH_BYTES = (size_t)QEVICT_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

// In host code `g_noalloc_scratch` is only a stand-in for the symbol, not a device address; the address is
// asked for once per device, with that device current, and remembered here.
constexpr int MAX_DEVICES = 64;
void* g_scratch_addr[MAX_DEVICES] = {};

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" QEVICT_API qevict_status qevict_decode_attn_noalloc(qevict_handle h, int32_t layer, const void* q,
                                                               const void* k_new, const void* v_new, void* out,
                                                               void* stream_) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  const Geometry& g = h->geo;
  int l0, l1;
  if (layer == -1) { l0 = 0; l1 = g.n_layers; }
  else if (layer >= 0 && layer < g.n_layers) { l0 = layer; l1 = layer + 1; }
  else { h->last_error = "layer out of range"; return QEVICT_ERR_INVALID_ARG; }
  if (!q || !out) { h->last_error = "q and out must not be NULL"; return QEVICT_ERR_INVALID_ARG; }
  if ((k_new == nullptr) != (v_new == nullptr)) {
    h->last_error = "k_new and v_new must both be given or both be NULL";
    return QEVICT_ERR_INVALID_ARG;
  }
  const int dev = h->cfg.device;
  if (dev < 0 || dev >= MAX_DEVICES) { h->last_error = "device ordinal not supported by the no-allocation entry point"; return QEVICT_ERR_UNSUPPORTED; }

  // The scratch is indexed by unit exactly like the handle's own scratch, so it has to span the units up
  // to the last one of the call.
  const size_t units_spanned = (size_t)l1 * g.batch;
  const size_t o_bytes = align256(units_spanned * g.Hq * (size_t)MAX_SPLITS * g.D * sizeof(float));
  const size_t ml_bytes = align256(units_spanned * g.Hq * (size_t)MAX_SPLITS * 2 * sizeof(float));
  const size_t w_bytes = align256(units_spanned * g.Hq * (size_t)g.EMAX * sizeof(float2));
  if (o_bytes + ml_bytes + w_bytes > NOALLOC_SCRATCH_BYTES) {
    char buf[192];
    snprintf(buf, sizeof(buf), "this call needs %zu bytes of attention scratch; the built-in array holds %zu (use qevict_decode_attn)",
             o_bytes + ml_bytes + w_bytes, NOALLOC_SCRATCH_BYTES);
    h->last_error = buf;
    return QEVICT_ERR_NO_MEMORY;
  }
  for (int l = l0; l < l1; ++l) {
    const LayerMirror& m = h->layers[l];
    if (!m.prefilled) { h->last_error = "decode before prefill_assign"; return QEVICT_ERR_BAD_STATE; }
    if (k_new && !m.has_open) {
      if (m.aged > g.aged_cap) { h->last_error = "too many filled windows are waiting: call qevict_rebalance"; return QEVICT_ERR_BAD_STATE; }
      if (m.n_windows + 1 > g.NW) { h->last_error = "context would exceed max_context"; return QEVICT_ERR_BAD_STATE; }
    }
  }
  cudaError_t e = cudaSetDevice(dev);
  if (e == cudaSuccess && !g_scratch_addr[dev]) {
    // set-up, once per device: ask the runtime where the array lives on this device
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e == cudaSuccess) g_scratch_addr[dev] = p;
  }
  if (e != cudaSuccess) { h->last_error = std::string("no-allocation set-up: ") + cudaGetErrorString(e); return QEVICT_ERR_CUDA; }
  unsigned char* scratch = static_cast<unsigned char*>(g_scratch_addr[dev]);

  KernelArgs a;
  a.geo = g;
  a.st = h->st;
  a.mig_parity = 0;  // no routing event on this path
#ifdef QEVICT_TRACE
  a.trace = h->st.trace + (size_t)TRACE_CALLS * TRACE_CALL_WORDS;  // not traced: the sink block
#endif
  a.st.o_part = reinterpret_cast<float*>(scratch);
  a.st.ml = reinterpret_cast<float*>(scratch + o_bytes);
  a.st.wrec = reinterpret_cast<float2*>(scratch + o_bytes + ml_bytes);
  a.unit0 = l0 * g.batch;
  a.n_units = (l1 - l0) * g.batch;

  if (k_new) {
    e = launch_append(a, k_new, v_new, stream);
    if (e != cudaSuccess) { h->last_error = std::string("append: ") + cudaGetErrorString(e); return QEVICT_ERR_CUDA; }
    h->launches++;
    for (int l = l0; l < l1; ++l) {
      LayerMirror& m = h->layers[l];
      if (!m.has_open) { m.has_open = true; m.open_fill = 0; m.n_windows++; }
      if (++m.open_fill == g.W) { m.has_open = false; m.open_fill = 0; m.aged++; }
    }
  }
  int e_bound = 1;
  for (int l = l0; l < l1; ++l) {
    const LayerMirror& m = h->layers[l];
    const int eb = g.Kfp + g.Kq + m.aged + (m.has_open ? 1 : 0);
    if (eb > e_bound) e_bound = eb;
  }
  DecodeParams p;
  p.e_bound = e_bound < g.EMAX ? e_bound : g.EMAX;
  p.q = q; p.entries = a.st.entries; p.n_live = a.st.n_live; p.open_fill = a.st.open_fill;
  p.fp_pool = a.st.fp_pool; p.q_pool = a.st.q_pool; p.o_part = a.st.o_part; p.ml = a.st.ml; p.wrec = a.st.wrec;
  p.status = a.st.status;
  p.rope = reinterpret_cast<const char*>(a.st.rope_table);
#ifdef QEVICT_TRACE
  p.trace = a.trace;
#endif
  p.unit0 = a.unit0; p.S = choose_splits(h, a.n_units); p.Hq = g.Hq; p.Hkv = g.Hkv; p.G = g.G; p.EMAX = g.EMAX;
  p.PF = g.PF; p.PQ = g.PQ; p.fp_page_bytes = g.fp_page_bytes; p.q_page_bytes = g.q_page_bytes; p.scale_log2 = g.scale_log2;
  e = h->decode_fn(p, a.n_units, stream);
  if (e != cudaSuccess) { h->last_error = std::string("attention: ") + cudaGetErrorString(e); return QEVICT_ERR_CUDA; }
  h->launches++;
  e = launch_combine(a, p.S, e_bound, out, stream);
  if (e != cudaSuccess) { h->last_error = std::string("combine: ") + cudaGetErrorString(e); return QEVICT_ERR_CUDA; }
  h->launches++;
  h->decode_steps++;
  return QEVICT_OK;
}
