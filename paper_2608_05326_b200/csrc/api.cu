// Host side of the C ABI: validation, workspace carving, call-order bookkeeping, kernel launches.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "ctx.h"

using namespace qevict;

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int next_pow2(int x) {
  int p = 2;
  while (p < x) p <<= 1;
  return p;
}

}  // namespace

namespace {

// Text of the last failure of a call that has no handle to keep it in (qevict_create, qevict_workspace_bytes),
// per calling thread; qevict_last_error(NULL) returns it.
thread_local std::string t_create_error;

qevict_status fail(qevict_handle h, qevict_status s, const std::string& msg) {
  if (h) h->last_error = msg;
  else t_create_error = msg;
  return s;
}

// Brackets one kernel launch with events when instrumentation is on.
template <class F>
cudaError_t timed_launch(qevict_ctx* h, int kind, cudaStream_t stream, F launch) {
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (h->timing) {
    if (h->ev_used + 2 > h->ev_pool.size()) {
      cudaError_t e = cudaEventCreate(&e0);
      if (e != cudaSuccess) return e;
      e = cudaEventCreate(&e1);
      if (e != cudaSuccess) return e;
      h->ev_pool.push_back(e0);
      h->ev_pool.push_back(e1);
      h->ev_kind.push_back(kind);
    }
    e0 = h->ev_pool[h->ev_used];
    e1 = h->ev_pool[h->ev_used + 1];
    h->ev_kind[h->ev_used / 2] = kind;
    h->ev_used += 2;
    cudaError_t e = cudaEventRecord(e0, stream);
    if (e != cudaSuccess) return e;
  }
  cudaError_t e = launch();
  if (e != cudaSuccess) return e;
  if (e1) e = cudaEventRecord(e1, stream);
  h->launches++;
  return e;
}

const char* validate(const qevict_config* c) {
  if (!c) return "config is NULL";
  if (c->struct_size != sizeof(qevict_config)) return "struct_size does not match this library's qevict_config";
  if (c->batch < 1 || c->n_layers < 1) return "batch and n_layers must be >= 1";
  if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads) return "n_q_heads must be a multiple of n_kv_heads";
  if (c->n_q_heads > 128) return "n_q_heads > 128";
  if (c->dtype != QEVICT_DTYPE_FP16 && c->dtype != QEVICT_DTYPE_BF16) return "dtype must be fp16 or bf16";
  if (c->fp_budget_windows < 0 || c->q_budget_windows < 0 || c->fp_budget_windows + c->q_budget_windows < 1)
    return "tier budgets must be >= 0 and not both zero";
  if (c->window < 1 || c->max_context < c->window || c->max_context % c->window) return "max_context must be a positive multiple of window";
  if (c->group_size < 1 || c->window % c->group_size || c->head_dim % c->group_size) return "group_size must divide window and head_dim";
  if (c->rebalance_interval_hint < 0) return "rebalance_interval_hint < 0";
  if (c->rank_mode < QEVICT_RANK_CUMULATIVE || c->rank_mode > QEVICT_RANK_KEYNORM) return "rank_mode must be a QEVICT_RANK_* value";
  if (c->rank_mode == QEVICT_RANK_DECAYED && !(c->rank_param > 0.f && c->rank_param <= 1.f)) return "decayed ranking needs 0 < rank_param <= 1";
  if (c->rank_mode == QEVICT_RANK_PNORM && !(c->rank_param >= 2.f && c->rank_param <= 8.f && c->rank_param == floorf(c->rank_param)))
    return "p-norm ranking needs an integer rank_param in 2..8";
  if (c->one_way != 0 && c->one_way != 1) return "one_way must be 0 or 1";
  if (c->sink_windows < 0 || c->recent_windows < 0) return "sink_windows and recent_windows must be >= 0";
  if (c->sink_windows + c->recent_windows > c->max_context / c->window) return "protected windows exceed max_context";
  if (!(c->softmax_scale >= 0.f) || isinf(c->softmax_scale)) return "softmax_scale must be finite and >= 0";
  if (!(c->rope_base >= 0.f) || isinf(c->rope_base) || (c->rope_base > 0.f && c->rope_base < 1.f)) return "rope_base must be 0 or >= 1";
  return nullptr;
}

const char* unsupported(const qevict_config* c) {
  if (c->n_q_heads / c->n_kv_heads > 8) return "more than 8 query heads per KV head";
  if (c->head_dim != 64 && c->head_dim != 128) return "head_dim must be 64 or 128";
  if (c->window != 32 && c->window != 64) return "window must be 32 or 64";
  if (c->quant_bits != 2 && c->quant_bits != 4) return "quant_bits must be 2 or 4";
  if (c->group_size != 32 && c->group_size != 64) return "group_size must be 32 or 64";
  if (c->max_context / c->window > 8192) return "more than 8192 windows per sequence";
  {
    // the attention kernel keeps a warp's work-list entries one per lane and runs at most MAX_SPLITS splits of
    // DECODE_WARPS warps per (unit, KV head): longer work lists cannot be walked
    const int r = c->rebalance_interval_hint > 0 ? c->rebalance_interval_hint : c->window;
    const long long emax = (long long)c->fp_budget_windows + c->q_budget_windows + c->sink_windows + c->recent_windows +
                           (r + c->window - 1) / c->window + 2;
    if (emax > 32LL * DECODE_WARPS * MAX_SPLITS)
      return "fp_budget_windows + q_budget_windows + protected windows exceed the 8192 work-list entries per sequence the attention kernel walks";
  }
  if (c->rank_mode == QEVICT_RANK_KEYNORM && (long long)c->n_kv_heads * c->head_dim > 4096)
    return "key-norm ranking supports n_kv_heads * head_dim <= 4096";
  return nullptr;
}

void make_geometry(const qevict_config& c, Geometry& g) {
  memset(&g, 0, sizeof(g));
  g.batch = c.batch; g.n_layers = c.n_layers; g.n_units = c.batch * c.n_layers;
  g.Hq = c.n_q_heads; g.Hkv = c.n_kv_heads; g.G = g.Hq / g.Hkv; g.D = c.head_dim; g.dtype = c.dtype;
  g.W = c.window; g.bits = c.quant_bits; g.group = c.group_size; g.Kf = c.fp_budget_windows; g.Kq = c.q_budget_windows;
  g.NW = c.max_context / c.window;
  const int r = c.rebalance_interval_hint > 0 ? c.rebalance_interval_hint : c.window;
  g.aged_cap = (r + g.W - 1) / g.W + 1;
  g.n_sink = c.sink_windows; g.n_recent = c.recent_windows;
  g.rank_mode = c.rank_mode; g.rank_param = c.rank_param; g.one_way = c.one_way != 0;
  g.rope_base = c.rope_base;
  g.Kfp = g.Kf + g.n_sink + g.n_recent;
  g.PF = g.Kfp + g.aged_cap + 1;
  g.PQ = g.Kq + g.Kf;
  g.EMAX = g.Kfp + g.Kq + g.aged_cap + 1;
  g.tiles = g.W / 32;
  g.fp_tile_bytes = 32u * g.D * 2u;
  g.fp_head_bytes = g.tiles * 2u * g.fp_tile_bytes;
  g.fp_page_bytes = g.Hkv * g.fp_head_bytes;
  g.q_kc_bytes = 32u * g.D * g.bits / 8u;
  g.q_vc_bytes = g.q_kc_bytes;
  g.q_vp_bytes = 32u * (g.D / g.group) * 4u;
  g.q_tile_stride = g.q_kc_bytes + g.q_vc_bytes + g.q_vp_bytes;
  g.q_kp_bytes = g.D * 4u;
  g.q_kp_off = g.tiles * g.q_tile_stride;
  g.q_head_bytes = g.q_kp_off + (g.W / g.group) * g.q_kp_bytes;
  g.q_page_bytes = g.Hkv * g.q_head_bytes;
  const double scale = c.softmax_scale > 0.f ? (double)c.softmax_scale : 1.0 / sqrt((double)c.head_dim);
  g.scale_log2 = (float)(scale * 1.4426950408889634074);
}

// Lays the cache out inside one buffer; with base == nullptr only the size is computed.
size_t carve(const Geometry& g, char* base, State* st, qevict_ctx* ctx) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    char* p = base ? base + off : nullptr;
    off = align_up(off + bytes, 256);
    return p;
  };
  const size_t U = g.n_units;
  State s;
  s.fp_pool = take(U * g.PF * (size_t)g.fp_page_bytes);
  s.q_pool = take(U * g.PQ * (size_t)g.q_page_bytes);
  s.tier = (uint8_t*)take(U * g.NW);
  s.ledger = (uint8_t*)take(U * g.NW);
  s.fp_page = (int32_t*)take(U * g.NW * 4);
  s.q_page = (int32_t*)take(U * g.NW * 4);
  s.importance = (float*)take(U * g.NW * 4);
  s.event_mass = (float*)take(U * g.NW * 4);
  s.knorm_acc = (float*)take(U * 4);
  s.fp_owner = (int32_t*)take(U * g.PF * 4);
  s.q_owner = (int32_t*)take(U * g.PQ * 4);
  s.n_windows = (int32_t*)take(U * 4);
  s.open_window = (int32_t*)take(U * 4);
  s.open_fill = (int32_t*)take(U * 4);
  s.n_live = (int32_t*)take(U * 4);
  s.entries = (uint2*)take(U * g.EMAX * 8);
  s.copy_list = (int4*)take(U * (size_t)(g.Kfp > 0 ? g.Kfp : 1) * 16);
  s.n_copy = (int32_t*)take(U * 4);
  s.mig_queue = (int4*)take(U * (size_t)(g.PF + g.Kq + g.Kf) * 32);
  s.mig_count = (int32_t*)take((size_t)g.n_layers * 2 * 4);
  s.counters = (unsigned long long*)take(U * 4 * 8);
  s.o_part = (float*)take(U * g.Hq * (size_t)MAX_SPLITS * g.D * 4);
  s.ml = (float*)take(U * g.Hq * (size_t)MAX_SPLITS * 2 * 4);
  s.wrec = (float2*)take(U * g.Hq * (size_t)g.EMAX * 8);
  s.mass_e = (float*)take(U * (size_t)g.EMAX * 4);
  s.status = (int32_t*)take(STATUS_BYTES);
  s.rope_table = (uint4*)take(g.rope_base > 0.f ? (size_t)g.NW * g.tiles * 32u * (g.D / 2) * 4u : 0);
#ifdef QEVICT_TRACE
  s.trace = (unsigned long long*)take(TRACE_BYTES);
#endif
  char* sq = take(U * g.Hq * (size_t)g.D * 2);
  char* sk = take(U * g.Hkv * (size_t)g.D * 2);
  char* sv = take(U * g.Hkv * (size_t)g.D * 2);
  char* so = take(U * g.Hq * (size_t)g.D * 2);
  if (st) *st = s;
  if (ctx) { ctx->stage_q = sq; ctx->stage_k = sk; ctx->stage_v = sv; ctx->stage_out = so; }
  return off;
}

bool layer_range(qevict_handle h, int layer, int* l0, int* l1) {
  if (layer == -1) { *l0 = 0; *l1 = h->geo.n_layers; return true; }
  if (layer < 0 || layer >= h->geo.n_layers) return false;
  *l0 = layer; *l1 = layer + 1;
  return true;
}

#ifdef QEVICT_TRACE
// {start = all ones, end = 0} in the first `calls` call blocks of the timeline.
cudaError_t trace_clear(qevict_handle h, uint32_t calls) {
  if (!calls) return cudaSuccess;
  std::vector<unsigned long long> init(calls * TRACE_CALL_WORDS);
  for (size_t i = 0; i < init.size(); i += 2) { init[i] = ~0ull; init[i + 1] = 0ull; }
  return cudaMemcpy(h->st.trace, init.data(), init.size() * 8, cudaMemcpyHostToDevice);
}
#endif

KernelArgs make_args(qevict_handle h, int l0, int l1) {
  KernelArgs a;
  a.geo = h->geo;
  a.st = h->st;
  a.unit0 = l0 * h->geo.batch;
  a.n_units = (l1 - l0) * h->geo.batch;
  a.mig_parity = (int)(h->mig_epoch[l0] & 1u);
#ifdef QEVICT_TRACE
  const uint32_t call = h->trace_calls < (uint32_t)TRACE_CALLS ? h->trace_calls++ : (uint32_t)TRACE_CALLS;
  a.trace = h->st.trace + call * TRACE_CALL_WORDS;
#endif
  return a;
}

}  // namespace

const char* qevict::decode_precheck(const qevict_ctx* h, int layer, const void* q, const void* k_new, const void* v_new,
                                    const void* out, int* l0, int* l1, qevict_status* st) {
  const Geometry& g = h->geo;
  *st = QEVICT_ERR_INVALID_ARG;
  if (layer == -1) { *l0 = 0; *l1 = g.n_layers; }
  else if (layer >= 0 && layer < g.n_layers) { *l0 = layer; *l1 = layer + 1; }
  else return "layer out of range";
  if (!q || !out) return "q and out must not be NULL";
  if ((k_new == nullptr) != (v_new == nullptr)) return "k_new and v_new must both be given or both be NULL";
  *st = QEVICT_ERR_BAD_STATE;
  if (h->broken) return "an earlier call failed after it had started to enqueue work: destroy this cache";
  for (int l = *l0; l < *l1; ++l) {
    const LayerMirror& m = h->layers[l];
    if (!m.prefilled) return "decode before prefill_assign";
    if (k_new && !m.has_open) {
      if (m.aged > g.aged_cap) return "too many filled windows are waiting: call qevict_rebalance";
      if (m.n_windows + 1 > g.NW) return "context would exceed max_context";
    }
  }
  *st = QEVICT_OK;
  return nullptr;
}

// Splits per (unit, KV head): enough CTAs to fill the GPU in whole waves while every warp still walks
// several windows.
int qevict::choose_splits(const qevict_ctx* h, int n_units) {
  const Geometry& g = h->geo;
  // a warp holds its work-list entries one per lane: at most 32 entries per warp
  int smin = (g.EMAX + 32 * DECODE_WARPS - 1) / (32 * DECODE_WARPS);
  if (smin > MAX_SPLITS) smin = MAX_SPLITS;  // (configurations that would need more are refused at create)
  if (h->forced_splits > 0) {
    const int f = h->forced_splits < smin ? smin : h->forced_splits;
    return f < MAX_SPLITS ? f : MAX_SPLITS;
  }
  const int entries = g.Kfp + g.Kq + 1;
  const long pairs = (long)n_units * g.Hkv;
  // resident CTAs: three per SM; two where the third ring slot of the pre-RoPE variant makes the ring 96 KB
  const long slots = (long)h->sm_count * (g.rope_base > 0.f && g.D == 128 ? 2 : 3);
  int best = smin;
  double best_cost = 1e30;
  const int smax = entries / DECODE_WARPS < 1 ? 1 : (entries / DECODE_WARPS > MAX_SPLITS ? MAX_SPLITS : entries / DECODE_WARPS);
  for (int s = smin; s <= (smax < smin ? smin : smax); ++s) {
    const long ctas = pairs * s;
    const long waves = (ctas + slots - 1) / slots;
    const double per_warp = ceil((double)entries / (s * DECODE_WARPS)) * g.tiles;
    const double cost = (double)waves * (per_warp + 2.0);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
  }
  return best;
}

namespace {

#define QE_DEVICE(h)                        \
  DeviceGuard qe_device_guard((h)->cfg.device); \
  QE_CUDA(h, qe_device_guard.err)

// the same for a launch that follows one that has already been enqueued in this call: a failure here leaves the
// device tables ahead of (or behind) the host's mirror, so the cache refuses every later call
#define QE_CUDA_MID(h, expr)                                                              \
  do {                                                                                    \
    cudaError_t e__ = (expr);                                                             \
    if (e__ != cudaSuccess) {                                                             \
      (h)->broken = true;                                                                 \
      return fail(h, QEVICT_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__)); \
    }                                                                                     \
  } while (0)

#define QE_CUDA(h, expr)                                                                  \
  do {                                                                                    \
    cudaError_t e__ = (expr);                                                             \
    if (e__ != cudaSuccess) return fail(h, QEVICT_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__)); \
  } while (0)

// q_host_alias != nullptr (only with k_new): `q` is the handle's staging buffer and the append kernel fills it from
// that page-locked host buffer, so the caller needs no copy operation of its own for the queries.
qevict_status decode_impl(qevict_handle h, int layer, const void* q, const void* k_new, const void* v_new, void* out,
                          cudaStream_t stream, const void* q_host_alias = nullptr) {
  int l0, l1;
  qevict_status pst;
  if (const char* msg = decode_precheck(h, layer, q, k_new, v_new, out, &l0, &l1, &pst)) return fail(h, pst, msg);
  const Geometry& g = h->geo;
  QE_DEVICE(h);
  const KernelArgs a = make_args(h, l0, l1);
  if (k_new) {
    QE_CUDA(h, timed_launch(h, 0, stream, [&] { return launch_append(a, k_new, v_new, stream, q_host_alias, q_host_alias ? const_cast<void*>(q) : nullptr); }));
    for (int l = l0; l < l1; ++l) {
      LayerMirror& m = h->layers[l];
      if (!m.has_open) { m.has_open = true; m.open_fill = 0; m.n_windows++; }
      if (++m.open_fill == g.W) { m.has_open = false; m.open_fill = 0; m.aged++; }
    }
  }
  int e_bound = 1;  // upper bound of every unit's work-list length, from the host's mirror of the window counts
  for (int l = l0; l < l1; ++l) {
    const LayerMirror& m = h->layers[l];
    const int e = g.Kfp + g.Kq + m.aged + (m.has_open ? 1 : 0);
    if (e > e_bound) e_bound = e;
  }
  DecodeParams p;
  p.e_bound = e_bound < g.EMAX ? e_bound : g.EMAX;
  p.q = q; p.entries = h->st.entries; p.n_live = h->st.n_live; p.open_fill = h->st.open_fill;
  p.fp_pool = h->st.fp_pool; p.q_pool = h->st.q_pool; p.o_part = h->st.o_part; p.ml = h->st.ml; p.wrec = h->st.wrec;
  p.unit0 = a.unit0; p.S = choose_splits(h, a.n_units); p.Hq = g.Hq; p.Hkv = g.Hkv; p.G = g.G; p.EMAX = g.EMAX;
  p.PF = g.PF; p.PQ = g.PQ; p.NW = g.NW; p.fp_page_bytes = g.fp_page_bytes; p.q_page_bytes = g.q_page_bytes; p.scale_log2 = g.scale_log2; p.status = h->st.status;
  p.rope = reinterpret_cast<const char*>(h->st.rope_table);
#ifdef QEVICT_TRACE
  p.trace = a.trace;
#endif
  if (k_new) QE_CUDA_MID(h, timed_launch(h, 1, stream, [&] { return h->decode_fn(p, a.n_units, stream); }));
  else QE_CUDA(h, timed_launch(h, 1, stream, [&] { return h->decode_fn(p, a.n_units, stream); }));
  QE_CUDA_MID(h, timed_launch(h, 2, stream, [&] { return launch_combine(a, p.S, e_bound, out, stream); }));
  h->decode_steps++;
  return QEVICT_OK;
}

}  // namespace

extern "C" {

QEVICT_API const char* qevict_version(void) { return "0.2"; }

QEVICT_API int32_t qevict_build_flavour(void) {
#if defined(QEVICT_DEBUG_BOUNDS)
  return 2;
#elif defined(QEVICT_TRACE)
  return 1;
#else
  return 0;
#endif
}

QEVICT_API const char* qevict_status_string(qevict_status s) {
  switch (s) {
    case QEVICT_OK: return "ok";
    case QEVICT_ERR_INVALID_ARG: return "invalid argument";
    case QEVICT_ERR_BAD_STATE: return "bad state";
    case QEVICT_ERR_NO_MEMORY: return "not enough memory";
    case QEVICT_ERR_UNSUPPORTED: return "unsupported configuration";
    case QEVICT_ERR_CUDA: return "CUDA error";
    case QEVICT_ERR_DEVICE_CHECK: return "device-side check failed";
  }
  return "unknown status";
}

QEVICT_API const char* qevict_last_error(qevict_handle h) { return h ? h->last_error.c_str() : t_create_error.c_str(); }

QEVICT_API uint64_t qevict_launch_count(qevict_handle h) { return h ? h->launches : 0; }

QEVICT_API qevict_status qevict_budget_from_bytes(const qevict_config* cfg, uint64_t hist_bytes, double q_frac, int32_t* k_f,
                                       int32_t* k_q, uint64_t* m_f, uint64_t* m_q) {
  if (!cfg || !(q_frac >= 0.0 && q_frac <= 1.0)) return QEVICT_ERR_INVALID_ARG;
  if (cfg->n_kv_heads < 1 || cfg->head_dim < 1 || cfg->window < 1 || cfg->group_size < 1 || cfg->quant_bits < 1 ||
      cfg->window % cfg->group_size || cfg->head_dim % cfg->group_size)
    return QEVICT_ERR_INVALID_ARG;
  const uint64_t h = cfg->n_kv_heads, w = cfg->window, d = cfg->head_dim, g = cfg->group_size, b = cfg->quant_bits;
  const uint64_t mf = 2 * h * w * d * 2;
  const uint64_t mq = h * (2 * w * d * b / 8 + (w / g) * d * 4 + w * (d / g) * 4);
  if (m_f) *m_f = mf;
  if (m_q) *m_q = mq;
  if (k_f) *k_f = (int32_t)floor((1.0 - q_frac) * (double)hist_bytes / (double)mf);
  if (k_q) *k_q = (int32_t)floor(q_frac * (double)hist_bytes / (double)mq);
  return QEVICT_OK;
}

// Shapes the kernels cannot run with although every single field is in range; nullptr if fine.
static const char* unsupported_geometry(const Geometry& g) {
  // the routing kernel keeps one unit's candidate tables in shared memory (227 KB per CTA on this architecture)
  if (route_smem_bytes(g, next_pow2(g.NW)) > 227u * 1024u)
    return "the routing tables of one sequence (max_context / window windows, the budgets' pages) exceed the shared memory of an SM";
  return nullptr;
}

QEVICT_API qevict_status qevict_workspace_bytes(const qevict_config* cfg, uint64_t* bytes) {
  if (!bytes) return fail(nullptr, QEVICT_ERR_INVALID_ARG, "bytes is NULL");
  if (const char* m = validate(cfg)) return fail(nullptr, QEVICT_ERR_INVALID_ARG, m);
  if (const char* m = unsupported(cfg)) return fail(nullptr, QEVICT_ERR_UNSUPPORTED, m);
  Geometry g;
  make_geometry(*cfg, g);
  if (const char* m = unsupported_geometry(g)) return fail(nullptr, QEVICT_ERR_UNSUPPORTED, m);
  *bytes = carve(g, nullptr, nullptr, nullptr);
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_create(const qevict_config* cfg, void* device_mem, uint64_t bytes, qevict_handle* out) {
  if (!out) return fail(nullptr, QEVICT_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (const char* m = validate(cfg)) return fail(nullptr, QEVICT_ERR_INVALID_ARG, m);
  if (const char* m = unsupported(cfg)) return fail(nullptr, QEVICT_ERR_UNSUPPORTED, m);
  {
    Geometry g0;
    make_geometry(*cfg, g0);
    if (const char* m = unsupported_geometry(g0)) return fail(nullptr, QEVICT_ERR_UNSUPPORTED, m);
  }
  if (!device_mem || ((uintptr_t)device_mem & 255)) return fail(nullptr, QEVICT_ERR_INVALID_ARG, "device_mem must be a 256-byte aligned device pointer");
  qevict_ctx* h = new (std::nothrow) qevict_ctx();
  if (!h) return fail(nullptr, QEVICT_ERR_NO_MEMORY, "host allocation failed");
  h->cfg = *cfg;
  make_geometry(*cfg, h->geo);
  const Geometry& g = h->geo;
  const size_t need = carve(g, (char*)device_mem, &h->st, h);
  if (need > bytes) {
    delete h;
    return fail(nullptr, QEVICT_ERR_NO_MEMORY, "device_mem is smaller than qevict_workspace_bytes");
  }
  switch ((g.dtype == QEVICT_DTYPE_BF16 ? 2 : 0) + (g.D == 128 ? 1 : 0)) {
    case 0: h->decode_fn = decode_dispatch_h64(g.bits, g.group, g.tiles, g.G, g.rope_base > 0.f); break;
    case 1: h->decode_fn = decode_dispatch_h128(g.bits, g.group, g.tiles, g.G, g.rope_base > 0.f); break;
    case 2: h->decode_fn = decode_dispatch_b64(g.bits, g.group, g.tiles, g.G, g.rope_base > 0.f); break;
    default: h->decode_fn = decode_dispatch_b128(g.bits, g.group, g.tiles, g.G, g.rope_base > 0.f); break;
  }
  if (!h->decode_fn) {
    delete h;
    return fail(nullptr, QEVICT_ERR_UNSUPPORTED, "no attention kernel is built for this combination of quant_bits, group_size and window");
  }
  h->layers.resize(g.n_layers);
  h->mig_epoch.assign(g.n_layers, 0u);
  DeviceGuard guard(cfg->device);
  cudaError_t e = guard.err;
  if (e == cudaSuccess) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) == cudaSuccess && sms > 0) h->sm_count = sms;
    const size_t U = g.n_units;
    // tables: everything between the pools and the scratch starts cleared
    e = cudaMemset(h->st.tier, 0, U * g.NW);
#ifdef QEVICT_DEBUG_BOUNDS
    // checking build: both pools start as a NaN pattern (all ones is a NaN in fp16 and in bf16), so that a read
    // of a page nobody wrote shows in the results
    if (e == cudaSuccess) e = cudaMemset(h->st.fp_pool, 0xFF, U * g.PF * (size_t)g.fp_page_bytes);
    if (e == cudaSuccess) e = cudaMemset(h->st.q_pool, 0xFF, U * g.PQ * (size_t)g.q_page_bytes);
#endif
    if (e == cudaSuccess) e = cudaMemset(h->st.ledger, 0, U * g.NW);
    if (e == cudaSuccess) e = cudaMemset(h->st.fp_page, 0xFF, U * g.NW * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.q_page, 0xFF, U * g.NW * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.importance, 0, U * g.NW * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.event_mass, 0, U * g.NW * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.knorm_acc, 0, U * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.fp_owner, 0xFF, U * g.PF * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.q_owner, 0xFF, U * g.PQ * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.n_windows, 0, U * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.open_window, 0xFF, U * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.open_fill, 0, U * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.n_live, 0, U * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.n_copy, 0, U * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.mig_count, 0, (size_t)g.n_layers * 2 * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.counters, 0, U * 32);
    if (e == cudaSuccess) e = cudaMemset(h->st.mass_e, 0, U * (size_t)g.EMAX * 4);
    if (e == cudaSuccess) e = cudaMemset(h->st.status, 0, STATUS_BYTES);
#ifdef QEVICT_TRACE
    if (e == cudaSuccess) e = trace_clear(h, TRACE_CALLS + 1);
#endif
    if (e == cudaSuccess) e = launch_rope_table(g, h->st, 0);
    if (e == cudaSuccess) e = route_prepare(route_smem_bytes(g, next_pow2(g.NW)));
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
  }
  if (e != cudaSuccess) {
    delete h;
    return fail(nullptr, QEVICT_ERR_CUDA, std::string("set-up on the device failed: ") + cudaGetErrorString(e));
  }
  *out = h;
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_destroy(qevict_handle h) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  for (cudaEvent_t e : h->ev_pool) cudaEventDestroy(e);
  if (h->out_ready) cudaEventDestroy(h->out_ready);
  delete h;
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_set_kernel_timing(qevict_handle h, int32_t enable) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  h->timing = enable != 0;
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_kernel_timeline(qevict_handle h, int32_t max_records, int32_t* kernel, double* start_us,
                                                double* end_us, int32_t* n_records) {
  if (!h || !kernel || !start_us || !end_us || !n_records || max_records < 0) return QEVICT_ERR_INVALID_ARG;
  *n_records = 0;
#ifdef QEVICT_TRACE
  QE_DEVICE(h);
  QE_CUDA(h, cudaDeviceSynchronize());
  const uint32_t calls = h->trace_calls;
  std::vector<unsigned long long> buf(calls * TRACE_CALL_WORDS);
  if (calls) QE_CUDA(h, cudaMemcpy(buf.data(), h->st.trace, buf.size() * 8, cudaMemcpyDeviceToHost));
  struct Rec { int k; unsigned long long t0, t1; };
  std::vector<Rec> recs;
  for (uint32_t c = 0; c < calls; ++c)
    for (int k = 0; k < TRACE_KERNELS; ++k) {
      const unsigned long long* b = buf.data() + c * TRACE_CALL_WORDS + (size_t)k * TRACE_SMS * 2;
      Rec r{k, ~0ull, 0ull};
      for (int sm = 0; sm < TRACE_SMS; ++sm) {
        if (b[2 * sm] < r.t0) r.t0 = b[2 * sm];
        if (b[2 * sm + 1] > r.t1) r.t1 = b[2 * sm + 1];
      }
      if (r.t0 != ~0ull) recs.push_back(r);
    }
  const size_t n = recs.size() < (size_t)max_records ? recs.size() : (size_t)max_records;
  const size_t first = recs.size() - n;
  for (size_t i = 0; i < n; ++i) {
    kernel[i] = recs[first + i].k;
    start_us[i] = (double)(long long)(recs[first + i].t0 - recs[first].t0) * 1e-3;
    end_us[i] = (double)(long long)(recs[first + i].t1 - recs[first].t0) * 1e-3;
  }
  *n_records = (int32_t)n;
  QE_CUDA(h, trace_clear(h, calls));
  h->trace_calls = 0;
  return QEVICT_OK;
#else
  return fail(h, QEVICT_ERR_UNSUPPORTED, "this library was built without -DQEVICT_TRACE");
#endif
}

QEVICT_API qevict_status qevict_kernel_times(qevict_handle h, double* total_ms, uint64_t* n_launches) {
  if (!h || !total_ms || !n_launches) return QEVICT_ERR_INVALID_ARG;
  for (int k = 0; k < QEVICT_N_KERNELS; ++k) { total_ms[k] = 0.0; n_launches[k] = 0; }
  for (size_t i = 0; i + 1 < h->ev_used; i += 2) {
    QE_CUDA(h, cudaEventSynchronize(h->ev_pool[i + 1]));
    float ms = 0.f;
    QE_CUDA(h, cudaEventElapsedTime(&ms, h->ev_pool[i], h->ev_pool[i + 1]));
    const int k = h->ev_kind[i / 2];
    total_ms[k] += ms;
    n_launches[k] += 1;
  }
  h->ev_used = 0;
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_kernel_time(qevict_handle h, double* total_ms, uint64_t* n_launches) {
  if (!h || !total_ms || !n_launches) return QEVICT_ERR_INVALID_ARG;
  double ms[QEVICT_N_KERNELS];
  uint64_t n[QEVICT_N_KERNELS];
  const qevict_status st = qevict_kernel_times(h, ms, n);
  if (st != QEVICT_OK) return st;
  *total_ms = ms[1];
  *n_launches = n[1];
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_set_splits(qevict_handle h, int32_t splits) {
  if (!h || splits < 0 || splits > MAX_SPLITS) return QEVICT_ERR_INVALID_ARG;
  h->forced_splits = splits;
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_prefill_assign(qevict_handle h, int32_t layer, const void* k, const void* v, int32_t ctx_tokens,
                                    const float* window_scores, void* stream) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  int l0, l1;
  if (!layer_range(h, layer, &l0, &l1)) return fail(h, QEVICT_ERR_INVALID_ARG, "layer out of range");
  if (!k || !v || (!window_scores && h->cfg.rank_mode != QEVICT_RANK_KEYNORM))
    return fail(h, QEVICT_ERR_INVALID_ARG, "k, v and window_scores must not be NULL");
  const Geometry& g = h->geo;
  if (ctx_tokens < g.W || ctx_tokens % g.W) return fail(h, QEVICT_ERR_UNSUPPORTED, "ctx_tokens must be a positive multiple of window");
  if (ctx_tokens > h->cfg.max_context) return fail(h, QEVICT_ERR_INVALID_ARG, "ctx_tokens exceeds max_context");
  for (int l = l0; l < l1; ++l)
    if (h->layers[l].prefilled) return fail(h, QEVICT_ERR_BAD_STATE, "prefill_assign called twice for a layer");
  QE_DEVICE(h);
  cudaStream_t s = (cudaStream_t)stream;
  const KernelArgs a = make_args(h, l0, l1);
  const int n_prompt = ctx_tokens / g.W;
  QE_CUDA(h, launch_prefill_init(a, n_prompt, window_scores, s));
  if (g.rank_mode == QEVICT_RANK_KEYNORM) {
    QE_CUDA(h, launch_key_norm_scores(a, k, ctx_tokens, n_prompt, s));
    h->launches++;
  }
  QE_CUDA_MID(h, launch_route(a, 1, next_pow2(n_prompt), s));
  QE_CUDA_MID(h, launch_copy_prompt(a, k, v, ctx_tokens, g.Kfp, s));
  QE_CUDA_MID(h, launch_migrate(a, k, v, ctx_tokens, g.Kq, s));
  ++h->mig_epoch[l0];  // the next event of these units counts its queue in the other counter
  h->launches += 2 + (g.Kfp > 0) + (g.Kq > 0);
  for (int l = l0; l < l1; ++l) {
    h->layers[l].prefilled = true;
    h->layers[l].n_windows = n_prompt;
  }
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_decode_attn(qevict_handle h, int32_t layer, const void* q, const void* k_new, const void* v_new,
                                 void* out, void* stream) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  return decode_impl(h, layer, q, k_new, v_new, out, (cudaStream_t)stream);
}

static qevict_status decode_host_impl(qevict_handle h, int32_t layer, const void* q_host, const void* k_new_host,
                                      const void* v_new_host, void* out_host, void* stream, bool sync) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  int l0, l1;
  qevict_status pst;
  // every argument and call-order check comes before the first copy: a refused call enqueues nothing
  if (const char* msg = decode_precheck(h, layer, q_host, k_new_host, v_new_host, out_host, &l0, &l1, &pst)) return fail(h, pst, msg);
  const Geometry& g = h->geo;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t nu = (size_t)(l1 - l0) * g.batch;
  const size_t qb = nu * g.Hq * g.D * 2, kb = nu * g.Hkv * g.D * 2;
  QE_DEVICE(h);
  // Page-locked host buffers that the device can address are used in place where each byte is touched once:
  // the append kernel reads the new token from them and the merge kernel writes `out` into them, which saves
  // three copy operations (and their hand-overs between the copy engines and the SMs) per step.  The queries
  // are read by every CTA of the attention kernel, so they always go through device memory.  Pageable buffers
  // take staged copies throughout.
  auto device_alias = [](const void* p) -> void* {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
  };
  const void* k_dev = nullptr;
  const void* v_dev = nullptr;
  if (k_new_host) {
    k_dev = device_alias(k_new_host);
    v_dev = device_alias(v_new_host);
    if (!k_dev || !v_dev) {
      QE_CUDA(h, cudaMemcpyAsync(h->stage_k, k_new_host, kb, cudaMemcpyHostToDevice, s));
      QE_CUDA(h, cudaMemcpyAsync(h->stage_v, v_new_host, kb, cudaMemcpyHostToDevice, s));
      k_dev = h->stage_k;
      v_dev = h->stage_v;
    }
  }
  // the queries: every CTA of the attention kernel reads them, so they go to device memory first -- through the
  // append kernel when there is one and the buffer is page-locked (no copy operation at all), else by a copy
  const void* q_alias = k_new_host ? device_alias(q_host) : nullptr;
  if (!q_alias) QE_CUDA(h, cudaMemcpyAsync(h->stage_q, q_host, qb, cudaMemcpyHostToDevice, s));
  void* out_dev = device_alias(out_host);
  const qevict_status st = decode_impl(h, layer, h->stage_q, k_dev, v_dev, out_dev ? out_dev : h->stage_out, s, q_alias);
  if (st != QEVICT_OK) return st;
  if (!out_dev) QE_CUDA(h, cudaMemcpyAsync(out_host, h->stage_out, qb, cudaMemcpyDeviceToHost, s));
  if (sync) {
    QE_CUDA(h, cudaStreamSynchronize(s));
  } else {
    // qevict_wait_result waits for exactly this point of the stream, whatever the caller enqueues behind it
    if (!h->out_ready) QE_CUDA(h, cudaEventCreateWithFlags(&h->out_ready, cudaEventDisableTiming));
    QE_CUDA(h, cudaEventRecord(h->out_ready, s));
  }
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_decode_attn_host(qevict_handle h, int32_t layer, const void* q_host, const void* k_new_host,
                                      const void* v_new_host, void* out_host, void* stream) {
  return decode_host_impl(h, layer, q_host, k_new_host, v_new_host, out_host, stream, true);
}

QEVICT_API qevict_status qevict_decode_attn_host_async(qevict_handle h, int32_t layer, const void* q_host,
                                                       const void* k_new_host, const void* v_new_host, void* out_host,
                                                       void* stream) {
  return decode_host_impl(h, layer, q_host, k_new_host, v_new_host, out_host, stream, false);
}

QEVICT_API qevict_status qevict_wait_result(qevict_handle h) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  if (!h->out_ready) return fail(h, QEVICT_ERR_BAD_STATE, "no qevict_decode_attn_host_async call has been made on this cache");
  QE_CUDA(h, cudaEventSynchronize(h->out_ready));
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_rebalance(qevict_handle h, int32_t layer, void* stream) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  int l0, l1;
  if (!layer_range(h, layer, &l0, &l1)) return fail(h, QEVICT_ERR_INVALID_ARG, "layer out of range");
  if (h->broken) return fail(h, QEVICT_ERR_BAD_STATE, "an earlier call failed after it had started to enqueue work: destroy this cache");
  for (int l = l0; l < l1; ++l)
    if (!h->layers[l].prefilled) return fail(h, QEVICT_ERR_BAD_STATE, "rebalance before prefill_assign");
  const Geometry& g = h->geo;
  QE_DEVICE(h);
  cudaStream_t s = (cudaStream_t)stream;
  const KernelArgs a = make_args(h, l0, l1);
  QE_CUDA(h, timed_launch(h, 3, s, [&] { return launch_route(a, 0, next_pow2(g.Kfp + g.Kq + g.aged_cap + 1), s); }));
  // quantizations and promotions of the event in one launch (linked where they share a page)
  const int max_promote = g.Kf < g.Kq ? g.Kf : g.Kq;
  const int max_items = (g.Kq > 0 ? g.PF : 0) + max_promote;
  if (max_items > 0) {
    QE_CUDA_MID(h, timed_launch(h, 4, s, [&] { return launch_migrate(a, nullptr, nullptr, 0, max_items, s); }));
    ++h->mig_epoch[l0];  // the next event of these units counts its queue in the other counter
  }
  for (int l = l0; l < l1; ++l) h->layers[l].aged = 0;
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_get_stats(qevict_handle h, int32_t layer, qevict_stats* out) {
  if (!h || !out) return QEVICT_ERR_INVALID_ARG;
  int l0, l1;
  if (!layer_range(h, layer, &l0, &l1)) return fail(h, QEVICT_ERR_INVALID_ARG, "layer out of range");
  const Geometry& g = h->geo;
  QE_DEVICE(h);
  QE_CUDA(h, cudaDeviceSynchronize());
  memset(out, 0, sizeof(*out));
  const size_t u0 = (size_t)l0 * g.batch, nu = (size_t)(l1 - l0) * g.batch;
  std::vector<unsigned long long> c(nu * 4);
  std::vector<uint8_t> tiers(nu * g.NW);
  int32_t status = 0;
  QE_CUDA(h, cudaMemcpy(c.data(), h->st.counters + u0 * 4, nu * 32, cudaMemcpyDeviceToHost));
  QE_CUDA(h, cudaMemcpy(tiers.data(), h->st.tier + u0 * g.NW, nu * g.NW, cudaMemcpyDeviceToHost));
  QE_CUDA(h, cudaMemcpy(&status, h->st.status, 4, cudaMemcpyDeviceToHost));
  for (size_t u = 0; u < nu; ++u) {
    out->promotions += c[u * 4]; out->quantizations += c[u * 4 + 1];
    out->reactivations += c[u * 4 + 2]; out->deletions += c[u * 4 + 3];
  }
  for (uint8_t t : tiers) {
    switch (t) {
      case QEVICT_TIER_FULL: out->n_full++; break;
      case QEVICT_TIER_QUANT: out->n_quant++; break;
      case QEVICT_TIER_AGED: out->n_aged++; break;
      case QEVICT_TIER_OPEN: out->n_open++; break;
      case QEVICT_TIER_EVICTED: out->n_evicted++; break;
      case QEVICT_TIER_SINK: out->n_sink++; break;
      default: break;
    }
  }
  out->decode_steps = h->decode_steps;
  if (status != 0) {
    char buf[96];
    snprintf(buf, sizeof(buf), "device check %d failed", status);
    return fail(h, QEVICT_ERR_DEVICE_CHECK, buf);
  }
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_check_device(qevict_handle h, int32_t* code) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  QE_DEVICE(h);
  QE_CUDA(h, cudaDeviceSynchronize());
  int32_t status = 0;
  QE_CUDA(h, cudaMemcpy(&status, h->st.status, 4, cudaMemcpyDeviceToHost));
  if (code) *code = status;
  if (status != 0) {
    char buf[96];
    snprintf(buf, sizeof(buf), "device check %d failed", status);
    return fail(h, QEVICT_ERR_DEVICE_CHECK, buf);
  }
  return QEVICT_OK;
}

static bool unit_of(qevict_handle h, int layer, int seq, int* u) {
  if (layer < 0 || layer >= h->geo.n_layers || seq < 0 || seq >= h->geo.batch) return false;
  *u = layer * h->geo.batch + seq;
  return true;
}

QEVICT_API qevict_status qevict_export_tables(qevict_handle h, int32_t layer, int32_t seq, int32_t* n_windows, uint8_t* tier,
                                   uint8_t* ledger, int32_t* fp_page, int32_t* q_page, float* importance, void* stream) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  int u;
  if (!unit_of(h, layer, seq, &u)) return fail(h, QEVICT_ERR_INVALID_ARG, "layer or seq out of range");
  const Geometry& g = h->geo;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t o = (size_t)u * g.NW;
  QE_DEVICE(h);
  if (n_windows) QE_CUDA(h, cudaMemcpyAsync(n_windows, h->st.n_windows + u, 4, cudaMemcpyDeviceToDevice, s));
  if (tier) QE_CUDA(h, cudaMemcpyAsync(tier, h->st.tier + o, g.NW, cudaMemcpyDeviceToDevice, s));
  if (ledger) QE_CUDA(h, cudaMemcpyAsync(ledger, h->st.ledger + o, g.NW, cudaMemcpyDeviceToDevice, s));
  if (fp_page) QE_CUDA(h, cudaMemcpyAsync(fp_page, h->st.fp_page + o, (size_t)g.NW * 4, cudaMemcpyDeviceToDevice, s));
  if (q_page) QE_CUDA(h, cudaMemcpyAsync(q_page, h->st.q_page + o, (size_t)g.NW * 4, cudaMemcpyDeviceToDevice, s));
  if (importance) QE_CUDA(h, cudaMemcpyAsync(importance, h->st.importance + o, (size_t)g.NW * 4, cudaMemcpyDeviceToDevice, s));
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_export_event_mass(qevict_handle h, int32_t layer, int32_t seq, float* event_mass, void* stream) {
  if (!h || !event_mass) return QEVICT_ERR_INVALID_ARG;
  int u;
  if (!unit_of(h, layer, seq, &u)) return fail(h, QEVICT_ERR_INVALID_ARG, "layer or seq out of range");
  QE_DEVICE(h);
  QE_CUDA(h, cudaMemcpyAsync(event_mass, h->st.event_mass + (size_t)u * h->geo.NW, (size_t)h->geo.NW * 4,
                             cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_export_last_mass(qevict_handle h, int32_t layer, int32_t seq, float* mass, void* stream) {
  if (!h || !mass) return QEVICT_ERR_INVALID_ARG;
  int u;
  if (!unit_of(h, layer, seq, &u)) return fail(h, QEVICT_ERR_INVALID_ARG, "layer or seq out of range");
  QE_DEVICE(h);
  const KernelArgs a = make_args(h, 0, h->geo.n_layers);
  QE_CUDA(h, launch_export_mass(a, u, mass, (cudaStream_t)stream));
  h->launches++;
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_export_fp_page(qevict_handle h, int32_t layer, int32_t seq, int32_t fp_page, void* k_out,
                                    void* v_out, void* stream) {
  if (!h || !k_out || !v_out) return QEVICT_ERR_INVALID_ARG;
  int u;
  if (!unit_of(h, layer, seq, &u)) return fail(h, QEVICT_ERR_INVALID_ARG, "layer or seq out of range");
  if (fp_page < 0 || fp_page >= h->geo.PF) return fail(h, QEVICT_ERR_INVALID_ARG, "fp_page out of range");
  QE_DEVICE(h);
  const KernelArgs a = make_args(h, 0, h->geo.n_layers);
  QE_CUDA(h, launch_export_fp_page(a, u, fp_page, k_out, v_out, (cudaStream_t)stream));
  h->launches++;
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_export_q_page(qevict_handle h, int32_t layer, int32_t seq, int32_t q_page, uint8_t* k_codes,
                                   void* k_params, uint8_t* v_codes, void* v_params, void* stream) {
  if (!h || !k_codes || !k_params || !v_codes || !v_params) return QEVICT_ERR_INVALID_ARG;
  int u;
  if (!unit_of(h, layer, seq, &u)) return fail(h, QEVICT_ERR_INVALID_ARG, "layer or seq out of range");
  if (q_page < 0 || q_page >= h->geo.PQ) return fail(h, QEVICT_ERR_INVALID_ARG, "q_page out of range");
  QE_DEVICE(h);
  const KernelArgs a = make_args(h, 0, h->geo.n_layers);
  QE_CUDA(h, launch_export_q_page(a, u, q_page, k_codes, k_params, v_codes, v_params, (cudaStream_t)stream));
  h->launches++;
  return QEVICT_OK;
}

}  // extern "C"
