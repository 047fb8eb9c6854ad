// Decode step for callers that must not allocate device memory.
//
// qevict_decode_attn_noalloc computes exactly what qevict_decode_attn computes, with the same kernels,
// but the attention kernel's scratch -- the per-split partial outputs, their (max, sum) pairs and the
// per-(head, window) softmax numerators that the combine kernel reads back -- lives in a fixed array
// inside this library's device image instead of in memory that somebody had to allocate.
#include <stdio.h>

#include <atomic>

#include "ctx.h"

using namespace qevict;

namespace {

// The scratch array.  Every GPU that loads the library carries these bytes until the process exits.
constexpr size_t NOALLOC_SCRATCH_BYTES = (size_t)QEVICT_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

// In host code `g_noalloc_scratch` is only a stand-in for the symbol, not a device address; the address is
// asked for once per device, with that device current, and remembered here (atomically: two handles on two
// threads may make their first call at the same time; both would store the same address).
constexpr int MAX_DEVICES = 64;
std::atomic<void*> g_scratch_addr[MAX_DEVICES];

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" QEVICT_API qevict_status qevict_decode_attn_noalloc(qevict_handle h, int32_t layer, const void* q,
                                                               const void* k_new, const void* v_new, void* out,
                                                               void* stream_) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  const Geometry& g = h->geo;
  int l0, l1;
  qevict_status pst;
  if (const char* msg = decode_precheck(h, layer, q, k_new, v_new, out, &l0, &l1, &pst)) { h->last_error = msg; return pst; }
  const int dev = h->cfg.device;
  if (dev < 0 || dev >= MAX_DEVICES) { h->last_error = "device ordinal not supported by the no-allocation entry point"; return QEVICT_ERR_UNSUPPORTED; }

  // The array holds the partial results of this call's units only: unit u of the call uses slot u - unit0.
  const size_t unit0 = (size_t)l0 * g.batch, n_units = (size_t)(l1 - l0) * g.batch;
  const size_t o_unit = g.Hq * (size_t)MAX_SPLITS * g.D * sizeof(float);
  const size_t ml_unit = g.Hq * (size_t)MAX_SPLITS * 2 * sizeof(float);
  const size_t w_unit = g.Hq * (size_t)g.EMAX * sizeof(float2);
  const size_t o_bytes = align256(n_units * o_unit), ml_bytes = align256(n_units * ml_unit), w_bytes = align256(n_units * w_unit);
  if (o_bytes + ml_bytes + w_bytes > NOALLOC_SCRATCH_BYTES) {
    char buf[192];
    snprintf(buf, sizeof(buf), "this call needs %zu bytes of attention scratch; the built-in array holds %zu (use qevict_decode_attn)",
             o_bytes + ml_bytes + w_bytes, NOALLOC_SCRATCH_BYTES);
    h->last_error = buf;
    return QEVICT_ERR_NO_MEMORY;
  }
  DeviceGuard guard(dev);
  cudaError_t e = guard.err;
  void* addr = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (e == cudaSuccess && !addr) {
    // set-up, once per device: ask the runtime where the array lives on this device (with lazy module loading
    // this is also what makes the runtime place the library's device image, array included, on the device)
    e = cudaGetSymbolAddress(&addr, g_noalloc_scratch);
    if (e == cudaSuccess) g_scratch_addr[dev].store(addr, std::memory_order_release);
  }
  if (e != cudaSuccess) { h->last_error = std::string("no-allocation set-up: ") + cudaGetErrorString(e); return QEVICT_ERR_CUDA; }
  // the kernels index their scratch by absolute unit: hand them the array's address moved back by unit0 slots
  const uintptr_t base = reinterpret_cast<uintptr_t>(addr);

  KernelArgs a;
  a.geo = g;
  a.st = h->st;
  a.mig_parity = 0;  // no routing event on this path
#ifdef QEVICT_TRACE
  a.trace = h->st.trace + (size_t)TRACE_CALLS * TRACE_CALL_WORDS;  // not traced: the sink block
#endif
  a.st.o_part = reinterpret_cast<float*>(base - unit0 * o_unit);
  a.st.ml = reinterpret_cast<float*>(base + o_bytes - unit0 * ml_unit);
  a.st.wrec = reinterpret_cast<float2*>(base + o_bytes + ml_bytes - unit0 * w_unit);
  a.unit0 = (int)unit0;
  a.n_units = (int)n_units;

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
  p.PF = g.PF; p.PQ = g.PQ; p.NW = g.NW; p.fp_page_bytes = g.fp_page_bytes; p.q_page_bytes = g.q_page_bytes; p.scale_log2 = g.scale_log2;
  e = h->decode_fn(p, a.n_units, stream);
  if (e != cudaSuccess) { h->broken = k_new != nullptr; h->last_error = std::string("attention: ") + cudaGetErrorString(e); return QEVICT_ERR_CUDA; }
  h->launches++;
  e = launch_combine(a, p.S, e_bound, out, stream);
  if (e != cudaSuccess) { h->broken = true; h->last_error = std::string("combine: ") + cudaGetErrorString(e); return QEVICT_ERR_CUDA; }
  h->launches++;
  h->decode_steps++;
  return QEVICT_OK;
}
