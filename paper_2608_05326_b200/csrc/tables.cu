// Window tables: append to the recent region, prefill initialisation, and the routing event
// (rank -> tiers -> page release / allocation -> migration lists -> decode work list).
#include <mutex>
#include <type_traits>

#include "kernels.cuh"
#include "layout.cuh"

namespace qevict {

namespace {

constexpr int ROUTE_MAX_THREADS = 512;

// order-preserving map float -> uint32 (ascending); -0 and +0 collapse
__device__ __forceinline__ uint32_t mono_bits(float f) {
  if (f == 0.f) f = 0.f;
  const uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Block-wide exclusive prefix sum of one int per thread; *total receives the sum.  scratch: 33 ints of
// shared memory.  Ends with a barrier, so scratch may be reused right away.
__device__ __forceinline__ int block_exclusive_scan(int cnt, int* scratch, int* total) {
  const int tid = threadIdx.x, nt = blockDim.x;
  const int lane = tid & 31, wid = tid >> 5;
  int inc = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  if (lane == 31) scratch[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    const int v = (lane < (nt >> 5)) ? scratch[lane] : 0;
    int iv = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, iv, o);
      if (lane >= o) iv += x;
    }
    scratch[lane] = iv - v;
    if (lane == 31) scratch[32] = iv;
  }
  __syncthreads();
  const int rank = scratch[wid] + inc - cnt;
  *total = scratch[32];
  __syncthreads();
  return rank;
}

// The same for three packed counters at once.  scratch: 99 ints.
__device__ __forceinline__ int3 block_exclusive_scan3(int3 cnt, int* scratch, int3* total) {
  const int tid = threadIdx.x, nt = blockDim.x;
  const int lane = tid & 31, wid = tid >> 5;
  int3 inc = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, inc.x, o), y = __shfl_up_sync(0xffffffffu, inc.y, o),
              z = __shfl_up_sync(0xffffffffu, inc.z, o);
    if (lane >= o) { inc.x += x; inc.y += y; inc.z += z; }
  }
  if (lane == 31) { scratch[wid] = inc.x; scratch[33 + wid] = inc.y; scratch[66 + wid] = inc.z; }
  __syncthreads();
  if (wid < 3) {
    int* sc = scratch + 33 * wid;
    const int v = (lane < (nt >> 5)) ? sc[lane] : 0;
    int iv = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, iv, o);
      if (lane >= o) iv += x;
    }
    sc[lane] = iv - v;
    if (lane == 31) sc[32] = iv;
  }
  __syncthreads();
  const int3 rank = make_int3(scratch[wid] + inc.x - cnt.x, scratch[33 + wid] + inc.y - cnt.y, scratch[66 + wid] + inc.z - cnt.z);
  *total = make_int3(scratch[32], scratch[65], scratch[98]);
  __syncthreads();
  return rank;
}

// Stable, deterministic block-wide stream compaction: calls emit(i, rank) for every i in [0, n)
// with pred(i), rank = number of smaller i with pred.  Returns the total.  pred must be pure until
// emit(i) has run.  scratch: 33 ints of shared memory.
template <class Pred, class Emit>
__device__ int block_compact(int n, int* scratch, Pred pred, Emit emit) {
  const int tid = threadIdx.x, nt = blockDim.x;
  const int chunk = (n + nt - 1) / nt;
  const int b = min(n, tid * chunk), e = min(n, b + chunk);
  int cnt = 0;
  for (int i = b; i < e; ++i) cnt += pred(i) ? 1 : 0;
  int total;
  int rank = block_exclusive_scan(cnt, scratch, &total);
  for (int i = b; i < e; ++i) {
    if (pred(i)) emit(i, rank++);
  }
  __syncthreads();
  return total;
}

// ------------------------------------------------------------------------------------------ append
// One CTA per unit.  Global memory is waited on twice: the unit's scalars together with the new token,
// then the open window's page id; everything else is stores.
// q_src != nullptr: the step's queries are also brought from `q_src` (page-locked host memory the device can
// address) into `q_dst` (device memory), [units of the call][q_vecs] 16-byte pieces: the host entry point then
// needs no separate copy operation for them, and the attention kernel finds them in device memory.
template <class T>
__global__ void __launch_bounds__(128) append_kernel(const KernelArgs a, const T* __restrict__ k_new,
                                                     const T* __restrict__ v_new, const uint4* __restrict__ q_src,
                                                     uint4* __restrict__ q_dst, int q_vecs) {
  const Geometry& g = a.geo;
  const int ul = blockIdx.x, u = a.unit0 + ul, tid = threadIdx.x;
  __shared__ int s_page;
  pdl_prologue();
  QE_TRACE_SCOPE(a.trace, 0);
  // every thread reads the scalars itself (same addresses: one broadcast transaction each)
  const int ow0 = a.st.open_window[u];
  const int fill0 = a.st.open_fill[u];
  const int n_live0 = a.st.n_live[u];
  const int n_win0 = a.st.n_windows[u];
  // the token: 16-byte pieces of the [H_kv][d] rows, in flight while the tables are being looked at
  constexpr int MAXV = 4;  // pieces per thread kept in registers (H_kv * d <= 4096 elements)
  const int nvec = g.Hkv * g.D / 8;
  uint4 kx[MAXV], vx[MAXV];
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    const int v = tid + i * 128;
    if (v < nvec) {
      kx[i] = __ldg(reinterpret_cast<const uint4*>(k_new + (size_t)ul * g.Hkv * g.D) + v);
      vx[i] = __ldg(reinterpret_cast<const uint4*>(v_new + (size_t)ul * g.Hkv * g.D) + v);
    }
  }
  if (q_src) {  // all loads of a round are issued before the first store waits for one
#pragma unroll 1
    for (int base = 0; base < q_vecs; base += 4 * 128) {
      uint4 qx[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int v = base + tid + i * 128;
        if (v < q_vecs) qx[i] = __ldg(q_src + (size_t)ul * q_vecs + v);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int v = base + tid + i * 128;
        if (v < q_vecs) q_dst[(size_t)ul * q_vecs + v] = qx[i];
      }
    }
  }
  int page, slot, window;
  const bool is_new = ow0 < 0;
  if (is_new) {
    // open a window: it takes the lowest free full-precision page
    window = n_win0;
    slot = 0;
    if (tid < 32) {
      int found = -1;
      const int32_t* owner = a.st.fp_owner + (size_t)u * g.PF;
#pragma unroll 1
      for (int base = 0; base < g.PF && found < 0; base += 32) {
        const int pg = base + tid;
        const bool free_pg = pg < g.PF && owner[pg] < 0;
        const unsigned m = __ballot_sync(0xffffffffu, free_pg);
        if (m) found = base + __ffs(m) - 1;
      }
      if (tid == 0) s_page = found;
    }
    __syncthreads();
    page = s_page;
    if (window >= g.NW || page < 0 || n_live0 >= g.EMAX) {
      if (tid == 0)
        record_check(a.st.status, window >= g.NW ? CHECK_WINDOW_OVERFLOW : (page < 0 ? CHECK_FP_POOL_EXHAUSTED : CHECK_ENTRY_OVERFLOW));
      return;
    }
  } else {
    window = ow0;
    slot = fill0;
    if (!QE_IN_RANGE(ow0 < g.NW && fill0 >= 0 && fill0 < g.W, a.st.status, CHECK_BOUNDS_WINDOW)) return;
    page = a.st.fp_page[(size_t)u * g.NW + ow0];
    if (!QE_IN_RANGE(page >= 0 && page < g.PF, a.st.status, CHECK_BOUNDS_PAGE)) return;
  }
  char* pbase = a.st.fp_pool + ((size_t)u * g.PF + page) * g.fp_page_bytes;
  if (is_new) {
    // unfilled token slots of the open window must hold finite values (they are multiplied by a zero
    // probability in the PV product)
    uint4* z = reinterpret_cast<uint4*>(pbase);
#pragma unroll 4
    for (uint32_t i = tid; i < g.fp_page_bytes / 16; i += 128) z[i] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
  }
  const int tile = slot >> 5, tk = slot & 31;
  // The token goes through shared memory so that the scatter into the fragment-major page is two short loops
  // (keys as channel pairs, values element by element) rather than a long unrolled sequence: this code runs
  // once per launch with cold instruction caches, so its size is its cost.
  __shared__ __align__(16) T s_k[128 * MAXV * 8];
  __shared__ __align__(16) T s_v[128 * MAXV * 8];
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    const int v = tid + i * 128;
    if (v < nvec) {
      reinterpret_cast<uint4*>(s_k)[v] = kx[i];
      reinterpret_cast<uint4*>(s_v)[v] = vx[i];
    }
  }
  __syncthreads();
  {
    const int n_stage = (nvec < MAXV * 128 ? nvec : MAXV * 128) * 8;  // elements held in shared memory
    const int dsh = 31 - __clz(g.D);                                  // the head dimension is a power of two
    char* tbase = pbase + (size_t)tile * 2 * g.fp_tile_bytes;
#pragma unroll 1
    for (int el = 2 * tid; el < n_stage; el += 256) {
      const int h = el >> dsh, ch = el & (g.D - 1);
      T* kt = reinterpret_cast<T*>(tbase + (size_t)h * g.fp_head_bytes);
      *reinterpret_cast<uint32_t*>(kt + fpk_off(tk, ch, g.D)) = *reinterpret_cast<const uint32_t*>(s_k + el);
    }
#pragma unroll 1
    for (int el = tid; el < n_stage; el += 128) {
      const int h = el >> dsh, ch = el & (g.D - 1);
      T* vt = reinterpret_cast<T*>(tbase + (size_t)h * g.fp_head_bytes + g.fp_tile_bytes);
      vt[fpv_off(tk, ch)] = s_v[el];
    }
  }
  for (int v = tid + MAXV * 128; v < nvec; v += 128) {  // wider rows than the register buffer holds
    const uint4 kk = __ldg(reinterpret_cast<const uint4*>(k_new + (size_t)ul * g.Hkv * g.D) + v);
    const uint4 vv = __ldg(reinterpret_cast<const uint4*>(v_new + (size_t)ul * g.Hkv * g.D) + v);
    const int h = (v * 8) / g.D, ch0 = v * 8 - h * g.D;
    T* kt = reinterpret_cast<T*>(pbase + (size_t)h * g.fp_head_bytes + (size_t)tile * 2 * g.fp_tile_bytes);
    T* vt = reinterpret_cast<T*>(reinterpret_cast<char*>(kt) + g.fp_tile_bytes);
    const T* ke = reinterpret_cast<const T*>(&kk);
    const T* ve = reinterpret_cast<const T*>(&vv);
    for (int e = 0; e < 8; ++e) {
      kt[fpk_off(tk, ch0 + e, g.D)] = ke[e];
      vt[fpv_off(tk, ch0 + e)] = ve[e];
    }
  }
  // key-norm ranking: the token's key norms (one per KV head) join the open window's sum; a window that is
  // complete gets its score, minus the mean norm.  Fixed summation order.
  float knorm_new = 0.f;
  if (g.rank_mode == QEVICT_RANK_KEYNORM) {
    __shared__ float s_sq[128 * MAXV];
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      const int v = tid + i * 128;
      float ss = 0.f;
      if (v < nvec) {
        const T* ke = reinterpret_cast<const T*>(&kx[i]);
#pragma unroll
        for (int e = 0; e < 8; ++e) { const float x = Tr<T>::to_float(ke[e]); ss = fmaf(x, x, ss); }
      }
      s_sq[v] = ss;
    }
    __syncthreads();
    if (tid == 0) {
      const int per_head = g.D / 8;
      float tok = 0.f;
      for (int h = 0; h < g.Hkv && h * per_head < 128 * MAXV; ++h) {
        float ss = 0.f;
        for (int j = 0; j < per_head; ++j) ss += s_sq[h * per_head + j];
        tok += sqrtf(ss);
      }
      knorm_new = (is_new ? 0.f : a.st.knorm_acc[u]) + tok;
    }
  }
  if (tid == 0) {
    const size_t wi = (size_t)u * g.NW + window;
    const int e_idx = is_new ? n_live0 : n_live0 - 1;  // the open window is always the last entry
    const bool full = slot + 1 == g.W;
    if (is_new) {
      a.st.fp_owner[(size_t)u * g.PF + page] = window;
      a.st.fp_page[wi] = page;
      a.st.q_page[wi] = -1;
      a.st.ledger[wi] = QEVICT_LEDGER_NONE;
      a.st.importance[wi] = 0.f;
      a.st.event_mass[wi] = 0.f;
      a.st.n_windows[u] = window + 1;
      a.st.n_live[u] = n_live0 + 1;
    }
    a.st.tier[wi] = full ? QEVICT_TIER_AGED : QEVICT_TIER_OPEN;
    a.st.entries[(size_t)u * g.EMAX + e_idx] =
        make_uint2((uint32_t)window | ((full ? KIND_FP : KIND_OPEN) << ENTRY_KIND_SHIFT), (uint32_t)page);
    a.st.open_window[u] = full ? -1 : window;
    a.st.open_fill[u] = full ? 0 : slot + 1;
    if (g.rank_mode == QEVICT_RANK_KEYNORM) {
      a.st.knorm_acc[u] = knorm_new;
      if (full) a.st.importance[wi] = -knorm_new / (float)(g.W * g.Hkv);
    }
  }
}

// ------------------------------------------------------------------------------------ prefill init
__global__ void prefill_init_kernel(const KernelArgs a, int n_prompt, const float* __restrict__ scores) {
  const Geometry& g = a.geo;
  const int ul = blockIdx.y, u = a.unit0 + ul;
  const int w = blockIdx.x * blockDim.x + threadIdx.x;
  if (w < n_prompt) {
    const size_t wi = (size_t)u * g.NW + w;
    a.st.tier[wi] = w < g.n_sink ? QEVICT_TIER_SINK : QEVICT_TIER_AGED;
    a.st.importance[wi] = scores ? scores[(size_t)ul * n_prompt + w] : 0.f;
  }
  if (w == 0) a.st.n_windows[u] = n_prompt;
}

// ------------------------------------------------------------------------------- key-norm scores (prefill)
// One CTA per (prompt window, unit): score = minus the mean over tokens and KV heads of the L2 norm of the keys.
template <class T>
__global__ void __launch_bounds__(128) key_norm_kernel(const KernelArgs a, const T* __restrict__ k_prompt, int ctx) {
  const Geometry& g = a.geo;
  const int w = blockIdx.x, ul = blockIdx.y, u = a.unit0 + ul, tid = threadIdx.x;
  __shared__ float s_part[128];
  float acc = 0.f;
  for (int pair = tid; pair < g.W * g.Hkv; pair += 128) {  // (head, token of the window)
    const int h = pair / g.W, tk = pair - h * g.W;
    const uint4* row = reinterpret_cast<const uint4*>(k_prompt + (((size_t)ul * g.Hkv + h) * ctx + (size_t)w * g.W + tk) * g.D);
    float ss = 0.f;
    for (int v = 0; v < g.D / 8; ++v) {
      const uint4 x = __ldg(row + v);
      const T* e = reinterpret_cast<const T*>(&x);
#pragma unroll
      for (int j = 0; j < 8; ++j) { const float f = Tr<T>::to_float(e[j]); ss = fmaf(f, f, ss); }
    }
    acc += sqrtf(ss);
  }
  s_part[tid] = acc;
  __syncthreads();
  if (tid == 0) {
    float sum = 0.f;
    for (int i = 0; i < 128; ++i) sum += s_part[i];
    a.st.importance[(size_t)u * g.NW + w] = -sum / (float)(g.W * g.Hkv);
  }
}

// ------------------------------------------------------------------------------------------- route
// One CTA per unit.  The candidates (Full, Quantized and aged windows) are gathered in ascending window
// order into shared memory together with the two page-owner tables; ranking, tier assignment, page
// release and allocation, migration lists and the decode work list all run on those shared copies, and
// the tables go back to global memory once at the end.  Global memory is waited on three times.
// A window is gathered by a routing event if it is a candidate (Full, Quantized, or filled and out of the
// protected recent region) or pinned (sink prefix, or filled and still inside the recent region: windows
// recent_lo and above).  Pinned windows keep their state; they are gathered because they are part of the
// decode work list and, at prefill, need a full-precision page like the Full windows.
constexpr uint8_t PINNED = 0x80;  // flag in the new-state byte of a gathered window
__device__ __forceinline__ bool is_candidate(uint8_t t, int w, int recent_lo) {
  return t == QEVICT_TIER_FULL || t == QEVICT_TIER_QUANT || (t == QEVICT_TIER_AGED && w < recent_lo);
}
__device__ __forceinline__ bool is_pinned(uint8_t t, int w, int recent_lo) {
  return t == QEVICT_TIER_SINK || (t == QEVICT_TIER_AGED && w >= recent_lo);
}

template <int NT>  // threads per CTA
__global__ void __launch_bounds__(NT) route_kernel(const KernelArgs a, int prefill, int sort_cap) {
  const Geometry& g = a.geo;
  const int u = a.unit0 + blockIdx.x, tid = threadIdx.x;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);  // [sort_cap]
  int4* qrec = reinterpret_cast<int4*>(keys + sort_cap);                      // [PF + Kq] first demotions of this event
  int4* prec = qrec + (g.PF + g.Kq);                                         // [Kf] promotions of this event
  int32_t* cw = reinterpret_cast<int32_t*>(prec + (g.Kf > 0 ? g.Kf : 1));     // [sort_cap] window of candidate c
  int32_t* cfp = cw + sort_cap;                                              // [sort_cap] its full-precision page
  int32_t* cq = cfp + sort_cap;                                              // [sort_cap] its quantized page
  int32_t* ofp = cq + sort_cap;                                              // [PF] owner of each page
  int32_t* oq = ofp + g.PF;                                                  // [PQ]
  int32_t* free_fp = oq + g.PQ;                                              // [PF] free page ids, ascending
  int32_t* free_q = free_fp + g.PF;                                          // [PQ]
  int32_t* reader = free_q + g.PQ;                                           // [PF] quantization that reads a page
  int32_t* flist = reader + g.PF;                                            // [EMAX] Full, then Quantized candidates
  int32_t* scratch = flist + g.EMAX;                                         // [128]
  int32_t* rhist = scratch + 128;                                            // [512] radix-selection histograms
  uint8_t* ctier = reinterpret_cast<uint8_t*>(rhist + 512);                 // [sort_cap] state before
  uint8_t* cled = ctier + sort_cap;                                          // [sort_cap] ledger flag
  uint8_t* cnew = cled + sort_cap;                                           // [sort_cap] state after
  pdl_prologue();
  QE_TRACE_SCOPE(a.trace, 3);

  uint8_t* tier = a.st.tier + (size_t)u * g.NW;
  uint8_t* ledger = a.st.ledger + (size_t)u * g.NW;
  int32_t* fp_page = a.st.fp_page + (size_t)u * g.NW;
  int32_t* q_page = a.st.q_page + (size_t)u * g.NW;
  const float* imp = a.st.importance + (size_t)u * g.NW;
  int32_t* fp_owner = a.st.fp_owner + (size_t)u * g.PF;
  int32_t* q_owner = a.st.q_owner + (size_t)u * g.PQ;
  const int nw = a.st.n_windows[u];
  const int ow = a.st.open_window[u];
  // The page owner tables: requested here, parked in shared memory only once the gather's loads are in flight
  // too (a store that waits for its load would hold up every request behind it).  The open window is no
  // candidate and keeps its page; the page is the one it owns.
  const int o_f0 = tid < g.PF ? fp_owner[tid] : -1;
  const int o_q0 = tid < g.PQ ? q_owner[tid] : -1;
  int* s_react = scratch + 100;
  int* s_del = scratch + 101;
  int* s_ow_page = scratch + 102;  // written by the one thread that sees the open window's page (read only if ow >= 0)
  if (tid == 0) { *s_react = 0; *s_del = 0; }
  auto park_owners = [&] {
    if (tid < g.PF) { ofp[tid] = o_f0; if (ow >= 0 && o_f0 == ow) *s_ow_page = tid; }
    if (tid < g.PQ) oq[tid] = o_q0;
#pragma unroll 1
    for (int i = tid + NT; i < g.PF; i += NT) {
      const int o = fp_owner[i];
      ofp[i] = o;
      if (ow >= 0 && o == ow) *s_ow_page = i;
    }
#pragma unroll 1
    for (int i = tid + NT; i < g.PQ; i += NT) oq[i] = q_owner[i];
  };

  // ---- ranking functions other than Eq. 1: fold the event accumulator into the score of every stored
  // window (each operation rounded on its own, so that the ranking is taken on reproducible numbers) ----
  if ((g.rank_mode == QEVICT_RANK_DECAYED || g.rank_mode == QEVICT_RANK_PNORM) && !prefill) {
    float* score = a.st.importance + (size_t)u * g.NW;
    float* ev = a.st.event_mass + (size_t)u * g.NW;
    const int p = (int)g.rank_param;
#pragma unroll 1
    for (int w = tid; w < nw; w += NT) {
      const uint8_t t = tier[w];
      if (t == QEVICT_TIER_NONE || t == QEVICT_TIER_EVICTED) continue;
      const float uw = ev[w], s0 = score[w];
      float s1;
      if (g.rank_mode == QEVICT_RANK_DECAYED) {
        s1 = __fadd_rn(__fmul_rn(g.rank_param, s0), uw);
      } else {
        float v = uw;
#pragma unroll 1
        for (int i = 1; i < p; ++i) v = __fmul_rn(v, uw);
        s1 = __fadd_rn(s0, v);
      }
      score[w] = s1;
      ev[w] = 0.f;
    }
    __syncthreads();
  }

  // ---- gather the candidates and the pinned windows in ascending window order -------------------------
  const int recent_lo = nw - (ow >= 0 ? 1 : 0) - g.n_recent;
  auto emit_gathered = [&](int w, int k, uint8_t t) {
    if (k >= sort_cap) return;
    const bool pin = is_pinned(t, w, recent_lo);
    cw[k] = w;
    ctier[k] = t;
    cled[k] = ledger[w];
    cfp[k] = fp_page[w];
    cq[k] = q_page[w];
    if (pin) cnew[k] = PINNED | t;
    // pinned windows get the largest keys: they are never counted among the smaller keys of a candidate
    keys[k] = pin ? (0xFFFFFFFF00000000ull | (uint32_t)k) : (((unsigned long long)(~mono_bits(imp[w])) << 32) | (uint32_t)k);
  };
  int n_all, n_real;
  const int chunk = (nw + NT - 1) / NT;
  constexpr int PRE_MAX = 10;
  const int cs = (g.NW + NT - 1) / NT;  // rows of the table per thread (not of the windows in use)
  // Small tables: every thread requests all five columns of its rows at once, before it knows how many
  // windows exist or which of them are candidates (rows past the last window hold state NONE), so the
  // whole gather costs one global round trip.  Unrolled for 5 or 10 rows per thread: this is run-once code,
  // and the shorter variant is half the instructions to fetch.
  auto gather_small = [&](auto pre_tag) {
    constexpr int PRE = decltype(pre_tag)::value;
    const int b = tid * cs;
    uint8_t tc[PRE], lc[PRE];
    int32_t fc[PRE], qc[PRE];
    float ic[PRE];
#pragma unroll
    for (int k = 0; k < PRE; ++k) {
      const bool ok = k < cs && b + k < g.NW;
      tc[k] = ok ? tier[b + k] : (uint8_t)QEVICT_TIER_NONE;
      lc[k] = ok ? ledger[b + k] : (uint8_t)0;
      fc[k] = ok ? fp_page[b + k] : -1;
      qc[k] = ok ? q_page[b + k] : -1;
      ic[k] = ok ? imp[b + k] : 0.f;
    }
    park_owners();
    int cnt = 0;  // gathered | candidates << 16
#pragma unroll
    for (int k = 0; k < PRE; ++k) {
      const bool c = is_candidate(tc[k], b + k, recent_lo);
      cnt += (c || is_pinned(tc[k], b + k, recent_lo) ? 1 : 0) + (c ? 0x10000 : 0);
    }
    int tot;
    int rank = block_exclusive_scan(cnt, scratch, &tot) & 0xFFFF;
    n_all = tot & 0xFFFF; n_real = tot >> 16;
    if (cnt) {
#pragma unroll
      for (int k = 0; k < PRE; ++k) {
        const int w = b + k;
        const bool pin = is_pinned(tc[k], w, recent_lo);
        if ((is_candidate(tc[k], w, recent_lo) || pin) && rank < sort_cap) {
          cw[rank] = w;
          ctier[rank] = tc[k];
          cled[rank] = lc[k];
          cfp[rank] = fc[k];
          cq[rank] = qc[k];
          if (pin) cnew[rank] = PINNED | tc[k];
          keys[rank] = pin ? (0xFFFFFFFF00000000ull | (uint32_t)rank)
                           : (((unsigned long long)(~mono_bits(ic[k])) << 32) | (uint32_t)rank);
          ++rank;
        }
      }
    }
    __syncthreads();
  };
  if (cs <= PRE_MAX && (g.rank_mode == QEVICT_RANK_CUMULATIVE || g.rank_mode == QEVICT_RANK_KEYNORM || prefill)) {
    if (cs <= 5) gather_small(std::integral_constant<int, 5>{});
    else gather_small(std::integral_constant<int, PRE_MAX>{});
  } else if (chunk <= 16) {
    // every thread reads its (up to 16) window states in one go and keeps them in registers
    uint8_t tc[16];
    const int b = tid * chunk;
#pragma unroll
    for (int k = 0; k < 16; ++k) tc[k] = (k < chunk && b + k < nw) ? tier[b + k] : (uint8_t)QEVICT_TIER_NONE;
    park_owners();
    int cnt = 0;  // gathered | candidates << 16
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      const bool c = is_candidate(tc[k], b + k, recent_lo);
      cnt += (c || is_pinned(tc[k], b + k, recent_lo) ? 1 : 0) + (c ? 0x10000 : 0);
    }
    int tot;
    int rank = block_exclusive_scan(cnt, scratch, &tot) & 0xFFFF;
    n_all = tot & 0xFFFF; n_real = tot >> 16;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      if (is_candidate(tc[k], b + k, recent_lo) || is_pinned(tc[k], b + k, recent_lo)) emit_gathered(b + k, rank++, tc[k]);
    }
    __syncthreads();
  } else {
    int* s_real = scratch + 103;
    if (tid == 0) *s_real = 0;
    park_owners();
    __syncthreads();
    n_all = block_compact(nw, scratch,
                          [&](int w) { const uint8_t t = tier[w]; return is_candidate(t, w, recent_lo) || is_pinned(t, w, recent_lo); },
                          [&](int w, int k) {
                            const uint8_t t = tier[w];
                            if (is_candidate(t, w, recent_lo)) atomicAdd(s_real, 1);
                            emit_gathered(w, k, t);
                          });
    n_real = *s_real;
  }
  const int n_cand = min(n_all, sort_cap);
#ifdef QEVICT_DEBUG_BOUNDS
  // page ids of the gathered windows index the owner tables below: one out of range is recorded and dropped
#pragma unroll 1
  for (int c = tid; c < n_cand; c += NT) {
    if (!QE_IN_RANGE(cfp[c] >= -1 && cfp[c] < g.PF, a.st.status, CHECK_BOUNDS_PAGE)) cfp[c] = -1;
    if (!QE_IN_RANGE(cq[c] >= -1 && cq[c] < g.PQ, a.st.status, CHECK_BOUNDS_PAGE)) cq[c] = -1;
    if (!QE_IN_RANGE(cw[c] >= 0 && cw[c] < g.NW, a.st.status, CHECK_BOUNDS_WINDOW)) cw[c] = 0;
  }
  __syncthreads();
#endif

  // ---- rank: score higher first, window index lower first; TopK_{K_f} -> Full, next TopK_{K_q} ->
  // Quantized, remainder -> Evicted -----------------------------------------------------------------
  if (g.one_way) {
    // One-way policy (no promotion): the Full tier is drawn from the candidates that are not Quantized, the
    // Quantized tier from everything else.  Two counting ranks (this is a diagnostic policy: no selection path).
    constexpr uint8_t UNDECIDED = 0x7F;
#pragma unroll 1
    for (int c = tid; c < n_cand; c += NT) {
      const unsigned long long mine = keys[c];
      if ((uint32_t)(mine >> 32) == 0xFFFFFFFFu) continue;  // pinned: state already set
      uint8_t nt = UNDECIDED;
      if (ctier[c] != QEVICT_TIER_QUANT) {
        int pos = 0;
#pragma unroll 1
        for (int i = 0; i < n_cand; ++i) pos += (ctier[i] != QEVICT_TIER_QUANT && keys[i] < mine) ? 1 : 0;
        if (pos < g.Kf) nt = QEVICT_TIER_FULL;
      }
      cnew[c] = nt;
    }
    __syncthreads();
#pragma unroll 1
    for (int c = tid; c < n_cand; c += NT) {
      if (cnew[c] != UNDECIDED) continue;
      const unsigned long long mine = keys[c];
      int pos = 0;  // smaller keys among the candidates outside the new Full tier (pinned windows hold the largest keys)
#pragma unroll 1
      for (int i = 0; i < n_cand; ++i) pos += (cnew[i] != QEVICT_TIER_FULL && !(cnew[i] & PINNED) && keys[i] < mine) ? 1 : 0;
      // written only after the count: other threads test this entry for "not Full", which holds before and after
      cnew[c] = pos < g.Kq ? QEVICT_TIER_QUANT : QEVICT_TIER_EVICTED;
    }
  } else if (n_cand <= 256) {
    // rank of a key = number of smaller keys (all keys are distinct); two adjacent lanes share a key and
    // count over one half of the keys each
    const int half = tid & 1, i0 = half ? n_cand / 2 : 0, i1 = half ? n_cand : n_cand / 2;
#pragma unroll 1
    for (int cb = 0; cb < n_cand; cb += NT / 2) {  // same trip count for the whole block
      const int c = cb + (tid >> 1);
      const unsigned long long mine = c < n_cand ? keys[c] : ~0ull;
      int pos = 0;
      if (c < n_cand)
        for (int i = i0; i < i1; ++i) pos += keys[i] < mine ? 1 : 0;
      pos += __shfl_xor_sync(0xffffffffu, pos, 1);
      if (c < n_cand && !half && (uint32_t)(mine >> 32) != 0xFFFFFFFFu)  // pinned windows keep the state set above
        cnew[c] = pos < g.Kf ? QEVICT_TIER_FULL : (pos < g.Kf + g.Kq ? QEVICT_TIER_QUANT : QEVICT_TIER_EVICTED);
    }
  } else {
    // Only the two cuts are needed, not the order: most-significant-digit-first radix selection of the
    // K_f-th and the (K_f + K_q)-th smallest key, both in the same six passes (four 8-bit digits of the
    // score, two of the candidate index).  thr[j] = the selected key: a candidate belongs to the first
    // K_j exactly if its key is <= thr[j].
    const int n_rk = min(n_real, n_cand);  // candidates (the pinned windows hold the largest keys)
    const int kk[2] = {min(g.Kf, n_rk), min(g.Kf + g.Kq, n_rk)};
    int* hist = rhist;                                   // [2][256]
    uint32_t* sel = reinterpret_cast<uint32_t*>(scratch + 104);  // [2][2] selected prefixes {low, high word}
    int* need = scratch + 108;                           // [2] rank still to find inside the current bucket
    if (tid < 2) { sel[2 * tid] = 0u; sel[2 * tid + 1] = 0u; need[tid] = kk[tid]; }
    unsigned long long mask = 0ull;
#pragma unroll 1
    for (int pass = 0; pass < 6; ++pass) {
      const int shift = pass < 4 ? 56 - 8 * pass : (pass == 4 ? 8 : 0);
#pragma unroll 1
      for (int i = tid; i < 512; i += NT) hist[i] = 0;
      __syncthreads();
      const unsigned long long p0 = ((unsigned long long)sel[1] << 32) | sel[0], p1 = ((unsigned long long)sel[3] << 32) | sel[2];
#pragma unroll 1
      for (int c = tid; c < n_cand; c += NT) {
        const unsigned long long key = keys[c];
        const int d = (int)((key >> shift) & 255ull);
        if ((key & mask) == p0) atomicAdd(&hist[d], 1);
        if ((key & mask) == p1) atomicAdd(&hist[256 + d], 1);
      }
      __syncthreads();
      if (tid < 64) {
        // warp j finds the digit of cut j: the first digit whose running count reaches need[j]
        const int j = tid >> 5, lane = tid & 31;
        const int* hj = hist + 256 * j;
        int loc[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { loc[i] = hj[lane * 8 + i]; sum += loc[i]; }
        int inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += v;
        }
        const int want = need[j];
        const unsigned hit = __ballot_sync(0xffffffffu, inc >= want);
        const int owner = hit ? __ffs(hit) - 1 : 31;  // kk >= 1 and the bucket holds >= want keys, so hit != 0
        if (lane == owner) {
          int run = inc - sum, d = 0;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if (run + loc[i] < want && i < 7) { run += loc[i]; d = i + 1; }
            else break;
          }
          need[j] = want - run;
          sel[2 * j + (shift >= 32 ? 1 : 0)] |= (uint32_t)(lane * 8 + d) << (shift & 31);
        }
      }
      mask |= 255ull << shift;
      __syncthreads();
    }
    const unsigned long long t0 = ((unsigned long long)sel[1] << 32) | sel[0], t1 = ((unsigned long long)sel[3] << 32) | sel[2];
#pragma unroll 1
    for (int c = tid; c < n_cand; c += NT) {
      const unsigned long long key = keys[c];
      if ((uint32_t)(key >> 32) == 0xFFFFFFFFu) continue;  // pinned: state already set
      cnew[c] = (kk[0] > 0 && key <= t0) ? QEVICT_TIER_FULL : ((kk[1] > 0 && key <= t1) ? QEVICT_TIER_QUANT : QEVICT_TIER_EVICTED);
    }
  }
  __syncthreads();

  // ---- releases (owner tables only; the candidates' page ids stay readable until the lists are built) --
#pragma unroll 1
  for (int c = tid; c < n_cand; c += NT) {
    const uint8_t old = ctier[c], nt = cnew[c];
    if ((nt == QEVICT_TIER_QUANT && old != QEVICT_TIER_QUANT) || nt == QEVICT_TIER_EVICTED) {
      if (cfp[c] >= 0) ofp[cfp[c]] = -1;
    }
    if (nt == QEVICT_TIER_EVICTED && cq[c] >= 0) oq[cq[c]] = -1;
    if (nt == QEVICT_TIER_QUANT && old != QEVICT_TIER_QUANT && cled[c] == QEVICT_LEDGER_DORMANT) {
      cled[c] = QEVICT_LEDGER_ACTIVE;  // reactivation: the retained codes are reused, no data moves
      atomicAdd(s_react, 1);
    }
  }
#pragma unroll 1
  for (int i = tid; i < g.PF; i += NT) reader[i] = -1;
  __syncthreads();

  // ---- one packed scan yields six stable compactions at once (all ascending): free full-precision pages,
  // free quantized pages, first demotions (need a quantized page), windows entering the Full tier without
  // a page (promotions; prompt windows at prefill), and the Full / Quantized members of the work list ----
  auto q_needs = [&](int c) { return cnew[c] == QEVICT_TIER_QUANT && ctier[c] != QEVICT_TIER_QUANT && cled[c] == QEVICT_LEDGER_NONE; };
  auto fp_needs = [&](int c) {
    return ((cnew[c] == QEVICT_TIER_FULL && ctier[c] != QEVICT_TIER_FULL) || (cnew[c] & PINNED)) && cfp[c] < 0;
  };
  auto lists_as_full = [&](int c) { return cnew[c] == QEVICT_TIER_FULL || (cnew[c] & PINNED); };
  int32_t* need_q = reinterpret_cast<int32_t*>(keys);  // the sort keys are dead from here on
  int32_t* need_fp = need_q + sort_cap;
  const int ch_f = (g.PF + NT - 1) / NT, ch_q = (g.PQ + NT - 1) / NT;
  const int ch_c = (n_cand + NT - 1) / NT;
  const int bf = min(g.PF, tid * ch_f), ef = min(g.PF, bf + ch_f), bq = min(g.PQ, tid * ch_q), eq = min(g.PQ, bq + ch_q);
  const int bc = min(n_cand, tid * ch_c), ec = min(n_cand, bc + ch_c);
  int3 cnt = make_int3(0, 0, 0);  // {free fp | free q << 16, need q | need fp << 16, Full | Quantized << 16}
#pragma unroll 1
  for (int pg = bf; pg < ef; ++pg) cnt.x += ofp[pg] < 0 ? 1 : 0;
#pragma unroll 1
  for (int pg = bq; pg < eq; ++pg) cnt.x += oq[pg] < 0 ? 0x10000 : 0;
#pragma unroll 1
  for (int c = bc; c < ec; ++c) {
    cnt.y += (q_needs(c) ? 1 : 0) + (fp_needs(c) ? 0x10000 : 0);
    cnt.z += (lists_as_full(c) ? 1 : 0) + (cnew[c] == QEVICT_TIER_QUANT ? 0x10000 : 0);
  }
  int3 tot;
  int3 rk = block_exclusive_scan3(cnt, scratch, &tot);
  const int n_free_fp = tot.x & 0xFFFF, n_free_q = tot.x >> 16, n_q_need = tot.y & 0xFFFF, n_fp_need = tot.y >> 16;
  const int n_f = tot.z & 0xFFFF, n_q = tot.z >> 16;
  int32_t* qlist = flist + n_f;
  {
    int r = rk.x & 0xFFFF;
#pragma unroll 1
    for (int pg = bf; pg < ef; ++pg) if (ofp[pg] < 0) free_fp[r++] = pg;
    r = rk.x >> 16;
#pragma unroll 1
    for (int pg = bq; pg < eq; ++pg) if (oq[pg] < 0) free_q[r++] = pg;
    int r0 = rk.y & 0xFFFF, r1 = rk.y >> 16, r2 = rk.z & 0xFFFF, r3 = rk.z >> 16;
#pragma unroll 1
    for (int c = bc; c < ec; ++c) {
      if (q_needs(c)) need_q[r0++] = c;
      if (fp_needs(c)) need_fp[r1++] = c;
      if (lists_as_full(c)) { if (r2 < g.EMAX) flist[r2] = c; ++r2; }
      if (cnew[c] == QEVICT_TIER_QUANT) { if (n_f + r3 < g.EMAX) qlist[r3] = c; ++r3; }
    }
  }
  const int qcap = g.PF + g.Kq;
  const int nq = min(n_q_need, min(n_free_q, qcap)), nfp = min(n_fp_need, min(n_free_fp, prefill ? g.Kfp : g.Kf));
  const int n_items = nq + (prefill ? 0 : nfp);
  int qbase = 0;  // thread 0: where this unit's records start in the call's queue (waited for only at the end)
  if (tid == 0) {
    if (n_q_need > nq) record_check(a.st.status, CHECK_Q_POOL_EXHAUSTED);
    if (n_fp_need > nfp) record_check(a.st.status, CHECK_FP_POOL_EXHAUSTED);
    // this unit's migrations join the call's queue (the order of the units in it does not matter: the
    // items are independent of one another); the reply is needed only at the very end
    if (n_items > 0) qbase = atomicAdd(a.st.mig_count + 2 * (a.unit0 / g.batch) + a.mig_parity, n_items);
  }
  __syncthreads();

  // first demotions take the free quantized pages in ascending order.  reader[p] = index of the
  // quantization that reads full-precision page p
#pragma unroll 1
  for (int k = tid; k < nq; k += NT) {
    const int c = need_q[k], pg = free_q[k];
    oq[pg] = cw[c];
    qrec[k] = make_int4(cw[c], prefill ? -1 : cfp[c], pg, -1);  // {window, source page, destination page, linked promotion}
    if (!prefill && cfp[c] >= 0) reader[cfp[c]] = k;
    cq[c] = pg;
    cled[c] = QEVICT_LEDGER_ACTIVE;
  }
  __syncthreads();
  // windows entering the Full tier take the free full-precision pages in ascending order.  A promotion
  // that receives a page some quantization of this event still has to read is linked to that quantization
  // (the migration kernel runs it right after it, in the same warps).
  int4* copy_list = a.st.copy_list + (size_t)u * g.Kfp;
#pragma unroll 1
  for (int k = tid; k < nfp; k += NT) {
    const int c = need_fp[k], pg = free_fp[k];
    ofp[pg] = cw[c];
    cfp[c] = pg;
    if (prefill) {
      copy_list[k] = make_int4(cw[c], pg, 0, 0);
    } else {
      const int rd = reader[pg];
      prec[k] = make_int4(cw[c], cq[c], pg, rd >= 0 ? 1 : 0);  // {window, source quantized page, destination page, linked}
      if (rd >= 0) qrec[rd].w = k;
    }
  }
  __syncthreads();

  // ---- commit: the candidates' rows and the owner tables go back to global memory --------------------
#pragma unroll 1
  for (int c = tid; c < n_cand; c += NT) {
    const uint8_t old = ctier[c], nt = cnew[c];
    const int w = cw[c];
    if (nt & PINNED) {  // state unchanged; at prefill the window has just received its page
      fp_page[w] = cfp[c];
      continue;
    }
    if (nt == QEVICT_TIER_FULL) {
      if (old == QEVICT_TIER_QUANT) cled[c] = QEVICT_LEDGER_DORMANT;  // codes retained for a later demotion
    } else if (nt == QEVICT_TIER_QUANT) {
      if (old != QEVICT_TIER_QUANT) cfp[c] = -1;
    } else {  // evicted: everything released, ledger deleted
      cfp[c] = -1;
      cq[c] = -1;
      cled[c] = QEVICT_LEDGER_NONE;
      atomicAdd(s_del, 1);
    }
    tier[w] = nt;
    ledger[w] = cled[c];
    fp_page[w] = cfp[c];
    q_page[w] = cq[c];
  }
#pragma unroll 1
  for (int i = tid; i < g.PF; i += NT) fp_owner[i] = ofp[i];
#pragma unroll 1
  for (int i = tid; i < g.PQ; i += NT) q_owner[i] = oq[i];
  // the migration records (32 bytes each; format: see the migration kernel), written by the first warp: the
  // reply of the queue reservation reaches the other lanes by shuffle
  if (tid < 32) {
    const int base = __shfl_sync(0xffffffffu, qbase, 0);
    int4* queue = a.st.mig_queue + ((size_t)a.unit0 * (g.PF + g.Kq + g.Kf) + base) * 2;
#pragma unroll 1
    for (int i = tid; i < n_items; i += 32) {
      if (i < nq) {
        const int4 it = qrec[i];
        queue[2 * i] = make_int4(u, 0, it.x, it.y);
        queue[2 * i + 1] = make_int4(it.z, it.w >= 0 ? prec[it.w].y : -1, 0, 0);
      } else {
        const int4 it = prec[i - nq];
        queue[2 * i] = make_int4(u, it.w ? 2 : 1, it.x, it.y);
        queue[2 * i + 1] = make_int4(it.z, -1, 0, 0);
      }
    }
  }
  __syncthreads();  // cfp / cq / cled are final (the evictions above reset theirs)

  // ---- decode work list: Full and Quantized windows (each ascending) interleaved in proportion, so that
  // every stretch of the list -- and therefore every warp of the attention kernel at every moment --
  // sees the same mix of 16-bit and low-bit pages; open window last -------------------------------------
  uint2* entries = a.st.entries + (size_t)u * g.EMAX;
  {
    const int n = n_f + n_q;
#pragma unroll 1
    for (int k = tid; k < n && k < g.EMAX; k += NT) {
      const int cf = (int)(((long long)k * n_f) / n);                       // Full windows before position k
      const bool is_f = (int)(((long long)(k + 1) * n_f) / n) > cf;
      if (is_f) {
        const int c = flist[cf];
        entries[k] = make_uint2((uint32_t)cw[c] | (KIND_FP << ENTRY_KIND_SHIFT), (uint32_t)cfp[c]);
      } else {
        const int c = qlist[k - cf];
        entries[k] = make_uint2((uint32_t)cw[c] | (KIND_Q << ENTRY_KIND_SHIFT), (uint32_t)cq[c]);
      }
    }
  }
  if (tid == 0) {
    int n = n_f + n_q;
    if (ow >= 0) {
      if (n < g.EMAX) entries[n] = make_uint2((uint32_t)ow | (KIND_OPEN << ENTRY_KIND_SHIFT), (uint32_t)*s_ow_page);
      n += 1;
    }
    if (n > g.EMAX) { record_check(a.st.status, CHECK_ENTRY_OVERFLOW); n = g.EMAX; }
    a.st.n_live[u] = n;
    a.st.n_copy[u] = prefill ? nfp : 0;
    // reductions, not read-modify-write: nothing at the kernel's end waits for a load
    unsigned long long* c = a.st.counters + (size_t)u * 4;
    if (!prefill && nfp) atomicAdd(c + 0, (unsigned long long)nfp);
    if (nq) atomicAdd(c + 1, (unsigned long long)nq);
    if (*s_react) atomicAdd(c + 2, (unsigned long long)*s_react);
    if (*s_del) atomicAdd(c + 3, (unsigned long long)*s_del);
  }
}

__global__ void export_mass_kernel(const KernelArgs a, int u, float* __restrict__ mass) {
  const Geometry& g = a.geo;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  // caller zeroed `mass`; scatter the per-entry masses of the last step
  if (i < a.st.n_live[u]) {
    const uint32_t w = a.st.entries[(size_t)u * g.EMAX + i].x & ENTRY_WINDOW_MASK;
    mass[w] = a.st.mass_e[(size_t)u * g.EMAX + i];
  }
}

}  // namespace

size_t route_smem_bytes(const Geometry& g, int sort_cap) {
  return (size_t)sort_cap * (8 + 12 + 3) + (size_t)(g.PF + g.Kq + (g.Kf > 0 ? g.Kf : 1)) * 16 +
         (size_t)(3 * g.PF + 2 * g.PQ + g.EMAX + 128 + 512) * 4 + 16;
}

// The dynamic shared-memory limit of a kernel is a per-device attribute shared by every cache of the process:
// it is only ever raised, to the largest size any cache on that device has asked for.
cudaError_t route_prepare(size_t max_smem) {
  static std::mutex mu;
  static size_t granted[64] = {};
  if (max_smem <= 48 * 1024) return cudaSuccess;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  if (dev >= 0 && dev < 64 && granted[dev] >= max_smem) return cudaSuccess;
  e = cudaFuncSetAttribute(route_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(route_kernel<ROUTE_MAX_THREADS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem);
  if (e == cudaSuccess && dev >= 0 && dev < 64) granted[dev] = max_smem;
  return e;
}

cudaError_t launch_append(const KernelArgs& a, const void* k_new, const void* v_new, cudaStream_t s, const void* q_src,
                          void* q_dst) {
  const int q_vecs = a.geo.Hq * a.geo.D / 8;
  if (a.geo.dtype == QEVICT_DTYPE_FP16)
    return launch_pdl(append_kernel<__half>, dim3(a.n_units), dim3(128), 0, s, a, (const __half*)k_new, (const __half*)v_new,
                      (const uint4*)q_src, (uint4*)q_dst, q_vecs);
  return launch_pdl(append_kernel<__nv_bfloat16>, dim3(a.n_units), dim3(128), 0, s, a, (const __nv_bfloat16*)k_new,
                    (const __nv_bfloat16*)v_new, (const uint4*)q_src, (uint4*)q_dst, q_vecs);
}

cudaError_t launch_key_norm_scores(const KernelArgs& a, const void* k_prompt, int ctx, int n_prompt, cudaStream_t s) {
  dim3 grid(n_prompt, a.n_units);
  if (a.geo.dtype == QEVICT_DTYPE_FP16) key_norm_kernel<__half><<<grid, 128, 0, s>>>(a, (const __half*)k_prompt, ctx);
  else key_norm_kernel<__nv_bfloat16><<<grid, 128, 0, s>>>(a, (const __nv_bfloat16*)k_prompt, ctx);
  return cudaGetLastError();
}

cudaError_t launch_prefill_init(const KernelArgs& a, int n_prompt, const float* scores, cudaStream_t s) {
  dim3 grid((n_prompt + 255) / 256, a.n_units);
  prefill_init_kernel<<<grid, 256, 0, s>>>(a, n_prompt, scores);
  return cudaGetLastError();
}

cudaError_t launch_route(const KernelArgs& a, int prefill, int sort_cap, cudaStream_t s) {
  // more threads only pay when there are enough candidates (every phase is a loop over them): from 129 candidate
  // slots on, 512 threads rank them in one round (two lanes per candidate) instead of two: route 9.1 -> 7.7 us on
  // the 32k configuration (193 candidates), 12.7 -> 10.4 us on the 128k one
  // (only while the launch is a single wave of CTAs: with hundreds of units the kernel is bound by throughput, not
  // by one CTA's latency, and the narrower CTAs pack better: 512 units of config 2 took 38 instead of 27 us)
  if (sort_cap > 512 || (sort_cap > 128 && a.n_units <= 160))
    return launch_pdl(route_kernel<ROUTE_MAX_THREADS>, dim3(a.n_units), dim3(ROUTE_MAX_THREADS), route_smem_bytes(a.geo, sort_cap), s, a,
                      prefill, sort_cap);
  return launch_pdl(route_kernel<256>, dim3(a.n_units), dim3(256), route_smem_bytes(a.geo, sort_cap), s, a, prefill, sort_cap);
}

cudaError_t launch_export_mass(const KernelArgs& a, int unit, float* mass, cudaStream_t s) {
  cudaError_t e = cudaMemsetAsync(mass, 0, sizeof(float) * a.geo.NW, s);
  if (e != cudaSuccess) return e;
  export_mass_kernel<<<(a.geo.EMAX + 255) / 256, 256, 0, s>>>(a, unit, mass);
  return cudaGetLastError();
}

}  // namespace qevict
