// Page kernels: quantize on first demotion, dequantize on promotion, prompt copy, plain-layout export.
//
// Quantizer [Methodology, "Migration-Stable Quantization"]: asymmetric min/max per group; keys per
// channel across `group` tokens, values per token across `group` channels.  Reading of the unstated
// details: zero = group minimum, scale = RNE_T((max - min) / qmax) with IEEE float32 subtract and
// divide, code = clamp(rint((x - zero) / scale)) in IEEE float32 (round half to even); a group whose
// scale is not a positive finite number gets scale 1 and codes 0.  The dequantized value is the
// single correctly rounded fused multiply-add RNE_T(code * scale + zero).
#include "kernels.cuh"
#include "layout.cuh"

namespace qevict {

namespace {

constexpr int PAGE_THREADS = 128;
constexpr int MIGRATE_THREADS = 128;

template <class T>
__device__ __forceinline__ void group_params(float mn, float mx, int qmax, T& s_out, T& z_out, float& s_f, bool& bad) {
  const float r = __fsub_rn(mx, mn);
  const T st = Tr<T>::from_float(__fdiv_rn(r, (float)qmax));
  float s = Tr<T>::to_float(st);
  bad = !(s > 0.f) || isinf(s) || isnan(s);
  if (bad) s = 1.f;
  s_out = Tr<T>::from_float(s);
  z_out = Tr<T>::from_float(mn);  // exact: mn is a value of T
  s_f = s;
}

// code = clamp(rint((x - zero) / scale)) on the IEEE float32 quotient.  The quotient is first estimated with
// the group's reciprocal (error of a few 1e-6 at most for codes up to 15); only when an estimate of the
// vector lies within 1e-3 of a rounding boundary (or is not finite) is the exact division carried out, so
// the result is the exact-division result in every case.  x >= zero (the group minimum), so the estimate
// needs no lower clamp.  This is run-once code whose length is its cost: one test per vector, not per code.
__device__ __forceinline__ float code_estimate(float x, float z, float inv_s, bool& near) {
  const float q = __fmul_rn(__fsub_rn(x, z), inv_s);
  const float r = rintf(q);
  near = near || !(fabsf(fabsf(q - r) - 0.5f) >= 1e-3f);
  return r;
}
__device__ __forceinline__ float code_exact(float x, float z, float s) {
  return fmaxf(rintf(__fdiv_rn(__fsub_rn(x, z), s)), 0.f);
}

// ---- migration tasks ---------------------------------------------------------------------------------
// Everything works in the fragment coordinates of the pages.  The members of a quantization group sit in
// the registers of the 8 lanes that share lane % 4, so a group's minimum and maximum are a few local
// comparisons and three shuffles, and every lane holds exactly the elements whose codes make up its own
// 32-bit code words.  A task is one warp's share of one half (keys or values) of a window of one KV head:
//   keys:   (block of `group` tokens, ks)      -> 16-byte vectors (ks, mt = 0, 1) of the block's tiles
//   values: (tile, channel group gc, ks)       -> 16-byte vectors (i, ks), i over the group's channels
// and the promotion task with the same coordinates writes exactly the vectors the quantization task reads
// (same lanes, same addresses), so a linked pair needs no ordering beyond program order inside the warp.
template <class T>
__device__ __forceinline__ void unpack2(uint32_t u, float& lo, float& hi) {
  const typename Tr<T>::T2 h2 = *reinterpret_cast<const typename Tr<T>::T2*>(&u);
  lo = Tr<T>::to_float(h2.x);
  hi = Tr<T>::to_float(h2.y);
}

template <class T>
__device__ __forceinline__ uint32_t pack2(T lo, T hi) {
  typename Tr<T>::T2 h2;
  h2.x = lo; h2.y = hi;
  return *reinterpret_cast<const uint32_t*>(&h2);
}

// slot k = hi * 2 + e of a lane: folds the registers of one vector (register a = hi * 2 + x) into the
// running minimum / maximum of the slots
template <class T>
__device__ __forceinline__ void fold_minmax(const uint4& v, float (&mn)[4], float (&mx)[4]) {
  const uint32_t r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    float f[2];
    unpack2<T>(r[a], f[0], f[1]);
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int k = (a >> 1) * 2 + e;
      mn[k] = fminf(mn[k], f[e]);
      mx[k] = fmaxf(mx[k], f[e]);
    }
  }
}

// codes of one vector: returns sum over (a, e) of code << (bits * a + 16 * e); `keep` clears the codes of the
// slots whose group has no usable scale
template <class T>
__device__ __forceinline__ uint32_t vector_codes(const uint4& v, const float (&mn)[4], const float (&sc)[4],
                                                 const float (&inv)[4], uint32_t keep, int qmax, int bits) {
  const uint32_t r[4] = {v.x, v.y, v.z, v.w};
  float c[4][2];
  bool near = false;
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    float f[2];
    unpack2<T>(r[a], f[0], f[1]);
#pragma unroll
    for (int e = 0; e < 2; ++e) c[a][e] = code_estimate(f[e], mn[(a >> 1) * 2 + e], inv[(a >> 1) * 2 + e], near);
  }
  if (__builtin_expect(near, 0)) {
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      float f[2];
      unpack2<T>(r[a], f[0], f[1]);
#pragma unroll
      for (int e = 0; e < 2; ++e) c[a][e] = code_exact(f[e], mn[(a >> 1) * 2 + e], sc[(a >> 1) * 2 + e]);
    }
  }
  uint32_t w = 0u;
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int e = 0; e < 2; ++e) w |= (uint32_t)(int)fminf(c[a][e], (float)qmax) << (bits * a + 16 * e);
  return w & keep;
}

// Minimum / maximum of the four slots over the 8 lanes of equal lane % 4, then the group parameters of
// each slot: the lane with (lane >> 2) & 3 == k works out slot k (one division per lane instead of four) and
// the others fetch it by shuffle.  Lanes 0..3 store the 16-byte parameter record (layout
// (hi * 2 + is_zero) * 2 + e).  `keep` gets the code bits of the slots whose scale is usable.
template <class T>
__device__ __forceinline__ void slot_params(float (&mn)[4], float (&mx)[4], int qmax, int bits, float (&sc)[4],
                                            float (&inv)[4], uint32_t& keep, uint4* param_dst, int lane) {
#pragma unroll
  for (int o = 4; o <= 16; o <<= 1) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      mn[k] = fminf(mn[k], __shfl_xor_sync(0xffffffffu, mn[k], o));
      mx[k] = fmaxf(mx[k], __shfl_xor_sync(0xffffffffu, mx[k], o));
    }
  }
  const int km = (lane >> 2) & 3;
  const float mn_m = km & 2 ? (km & 1 ? mn[3] : mn[2]) : (km & 1 ? mn[1] : mn[0]);
  const float mx_m = km & 2 ? (km & 1 ? mx[3] : mx[2]) : (km & 1 ? mx[1] : mx[0]);
  T st_m, zt_m;
  float s_m;
  bool bad_m;
  group_params<T>(mn_m, mx_m, qmax, st_m, zt_m, s_m, bad_m);
  const float inv_m = bad_m ? 0.f : __frcp_rn(s_m);  // zero marks an unusable scale (its estimates are 0 or NaN)
  T st[4], zt[4];
  keep = 0u;
  const uint32_t pair = (uint32_t)qmax | ((uint32_t)qmax << bits);  // the two registers of one `hi`
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int src = (lane & 3) + 4 * k;
    sc[k] = __shfl_sync(0xffffffffu, s_m, src);
    inv[k] = __shfl_sync(0xffffffffu, inv_m, src);
    st[k] = Tr<T>::from_float(sc[k]);  // exact: the scale is a value of T
    zt[k] = Tr<T>::from_float(mn[k]);  // exact: the minimum is a value of T
    if (inv[k] != 0.f) keep |= pair << (2 * bits * (k >> 1) + 16 * (k & 1));
  }
  if (lane < 4) *param_dst = make_uint4(pack2<T>(st[0], st[1]), pack2<T>(zt[0], zt[1]), pack2<T>(st[2], st[3]), pack2<T>(zt[2], zt[3]));
}

// two codes of a pair -> two dequantized values (the registers the decode kernel forms in flight)
template <class T>
__device__ __forceinline__ uint4 dequant_vector(uint32_t w, int sh, int bits, const uint4& pr) {
  const uint32_t mask = bits == 4 ? 0x000F000Fu : 0x00030003u, MG = Tr<T>::MAGIC;
  uint4 r;
  r.x = dequant2<T>(and_or(w >> (sh + 0 * bits), mask, MG), pr.x, pr.y);
  r.y = dequant2<T>(and_or(w >> (sh + 1 * bits), mask, MG), pr.x, pr.y);
  r.z = dequant2<T>(and_or(w >> (sh + 2 * bits), mask, MG), pr.z, pr.w);
  r.w = dequant2<T>(and_or(w >> (sh + 3 * bits), mask, MG), pr.z, pr.w);
  return r;
}

// ---- keys: task (blk, ks) -----------------------------------------------------------------------------
template <class T>
__device__ __forceinline__ void quant_key_task(const Geometry& g, int blk, int ks, const T* __restrict__ rows,
                                               const char* __restrict__ fp_head, char* qb, int lane) {
  const int D = g.D, bits = g.bits, qmax = (1 << bits) - 1, tpg = g.group >> 5, gq = lane >> 2, t = lane & 3;
  uint4 x[2][2];  // [tile of the group][mt]; register a = hi * 2 + rh, halves e
#pragma unroll
  for (int tl = 0; tl < 2; ++tl) {
    if (tl >= tpg) continue;
    const int tile = blk * tpg + tl;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      if (fp_head) {
        x[tl][mt] = reinterpret_cast<const uint4*>(fp_head + (size_t)tile * 2 * g.fp_tile_bytes)[(ks * 2 + mt) * 32 + lane];
      } else {
        uint32_t r[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          const int tk = tile * 32 + 16 * mt + 8 * (a & 1) + gq, ch = 16 * ks + 8 * (a >> 1) + 2 * t;
          r[a] = *reinterpret_cast<const uint32_t*>(rows + (size_t)tk * D + ch);
        }
        x[tl][mt] = make_uint4(r[0], r[1], r[2], r[3]);
      }
    }
  }
  float mn[4] = {INFINITY, INFINITY, INFINITY, INFINITY}, mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
  for (int tl = 0; tl < 2; ++tl) {
    if (tl >= tpg) continue;
    fold_minmax<T>(x[tl][0], mn, mx);
    fold_minmax<T>(x[tl][1], mn, mx);
  }
  float sc[4], inv[4];
  uint32_t keep;
  slot_params<T>(mn, mx, qmax, bits, sc, inv, keep, reinterpret_cast<uint4*>(qb + g.q_kp_off + (size_t)blk * g.q_kp_bytes) + ks * 4 + t, lane);
#pragma unroll
  for (int tl = 0; tl < 2; ++tl) {
    if (tl >= tpg) continue;
    uint32_t* dstw = reinterpret_cast<uint32_t*>(qb + (size_t)(blk * tpg + tl) * g.q_tile_stride);
    const uint32_t w0 = vector_codes<T>(x[tl][0], mn, sc, inv, keep, qmax, bits);
    const uint32_t w1 = vector_codes<T>(x[tl][1], mn, sc, inv, keep, qmax, bits);
    if (bits == 4) {
      dstw[code_word_off(ks * 2 + 0, lane)] = w0;
      dstw[code_word_off(ks * 2 + 1, lane)] = w1;
    } else {
      dstw[code_word_off(ks, lane)] = w0 | (w1 << 8);
    }
  }
}

template <class T>
__device__ __forceinline__ void promote_key_task(const Geometry& g, int blk, int ks, const char* __restrict__ qb, char* fb,
                                                 int lane) {
  const int bits = g.bits, tpg = g.group >> 5, t = lane & 3;
  const uint4 pr = reinterpret_cast<const uint4*>(qb + g.q_kp_off + (size_t)blk * g.q_kp_bytes)[ks * 4 + t];
#pragma unroll
  for (int tl = 0; tl < 2; ++tl) {
    if (tl >= tpg) continue;
    const int tile = blk * tpg + tl;
    const uint32_t* kc = reinterpret_cast<const uint32_t*>(qb + (size_t)tile * g.q_tile_stride);
    uint4* kt = reinterpret_cast<uint4*>(fb + (size_t)tile * 2 * g.fp_tile_bytes);
    if (bits == 4) {
      const uint32_t w0 = kc[code_word_off(ks * 2 + 0, lane)], w1 = kc[code_word_off(ks * 2 + 1, lane)];
      kt[(ks * 2 + 0) * 32 + lane] = dequant_vector<T>(w0, 0, 4, pr);
      kt[(ks * 2 + 1) * 32 + lane] = dequant_vector<T>(w1, 0, 4, pr);
    } else {
      const uint32_t w = kc[code_word_off(ks, lane)];
      kt[(ks * 2 + 0) * 32 + lane] = dequant_vector<T>(w, 0, 2, pr);
      kt[(ks * 2 + 1) * 32 + lane] = dequant_vector<T>(w, 8, 2, pr);
    }
  }
}

// ---- values: task (tile, gc, ks) ------------------------------------------------------------------------
template <class T>
__device__ __forceinline__ void quant_value_task(const Geometry& g, int tile, int gc, int ks, const T* __restrict__ rows,
                                                 const char* __restrict__ fp_head, char* qb, int lane) {
  const int D = g.D, bits = g.bits, qmax = (1 << bits) - 1, ipg = g.group >> 4, gq = lane >> 2, t = lane & 3;
  uint4 x[4];  // [i inside the group]; register a = hi * 2 + ah, halves e
#pragma unroll
  for (int ii = 0; ii < 4; ++ii) {
    if (ii >= ipg) continue;
    const int i = gc * ipg + ii;
    if (fp_head) {
      x[ii] = reinterpret_cast<const uint4*>(fp_head + (size_t)tile * 2 * g.fp_tile_bytes + g.fp_tile_bytes)[(i * 2 + ks) * 32 + lane];
    } else {
      uint32_t r[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int tk = tile * 32 + 16 * ks + 8 * (a >> 1) + 2 * t, ch = 16 * i + 8 * (a & 1) + gq;
        r[a] = pack2<T>(rows[(size_t)tk * D + ch], rows[(size_t)(tk + 1) * D + ch]);
      }
      x[ii] = make_uint4(r[0], r[1], r[2], r[3]);
    }
  }
  float mn[4] = {INFINITY, INFINITY, INFINITY, INFINITY}, mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
  for (int ii = 0; ii < 4; ++ii) {
    if (ii >= ipg) continue;
    fold_minmax<T>(x[ii], mn, mx);
  }
  float sc[4], inv[4];
  uint32_t keep;
  char* tb = qb + (size_t)tile * g.q_tile_stride;
  slot_params<T>(mn, mx, qmax, bits, sc, inv, keep, reinterpret_cast<uint4*>(tb + g.q_kc_bytes + g.q_vc_bytes) + (gc * 2 + ks) * 4 + t, lane);
  uint32_t* dstw = reinterpret_cast<uint32_t*>(tb + g.q_kc_bytes);
#pragma unroll
  for (int ii = 0; ii < 4; ++ii) {
    if (ii >= ipg) continue;
    const int i = gc * ipg + ii;
    const uint32_t w = vector_codes<T>(x[ii], mn, sc, inv, keep, qmax, bits);
    if (bits == 4) {
      dstw[code_word_off(i * 2 + ks, lane)] = w;
    } else {
      // a 2-bit word holds both token halves (the ks = 0 byte of each 16-bit half below the ks = 1 byte);
      // the two tasks that share a word write disjoint bytes
      unsigned char* b = reinterpret_cast<unsigned char*>(dstw + code_word_off(i, lane));
      b[ks] = (unsigned char)(w & 0xFFu);
      b[2 + ks] = (unsigned char)((w >> 16) & 0xFFu);
    }
  }
}

template <class T>
__device__ __forceinline__ void promote_value_task(const Geometry& g, int tile, int gc, int ks, const char* __restrict__ qb,
                                                   char* fb, int lane) {
  const int bits = g.bits, ipg = g.group >> 4, t = lane & 3;
  const char* tb = qb + (size_t)tile * g.q_tile_stride;
  const uint32_t* vc = reinterpret_cast<const uint32_t*>(tb + g.q_kc_bytes);
  const uint4 pr = reinterpret_cast<const uint4*>(tb + g.q_kc_bytes + g.q_vc_bytes)[(gc * 2 + ks) * 4 + t];
  uint4* vt = reinterpret_cast<uint4*>(fb + (size_t)tile * 2 * g.fp_tile_bytes + g.fp_tile_bytes);
#pragma unroll
  for (int ii = 0; ii < 4; ++ii) {
    if (ii >= ipg) continue;
    const int i = gc * ipg + ii;
    const uint32_t w = vc[code_word_off(bits == 4 ? i * 2 + ks : i, lane)];
    vt[(i * 2 + ks) * 32 + lane] = dequant_vector<T>(w, bits == 4 ? 0 : ks * 8, bits, pr);
  }
}

// Migration kernel.  The routing event leaves one queue of 32-byte records for the whole call:
//   {unit, kind, window, src} {dst, link, -, -}
//   kind 0  first demotion: quantize full-precision page src (-1: the prompt rows of `window`) into
//           quantized page dst; link >= 0: afterwards dequantize quantized page `link` into page src
//           (a promotion of the same event that was handed the page being vacated)
//   kind 1  promotion: dequantize quantized page src into full-precision page dst
//   kind 2  nothing (a promotion that is linked to a demotion)
// Every warp of a fixed-size grid takes (record, KV head, keys | values, task) tuples round-robin, so the
// launch costs the same whether one unit or all of them migrate something, and the tasks are independent
// (see above), so nothing waits on another warp.
template <class T>
__global__ void __launch_bounds__(MIGRATE_THREADS, 6) migrate_kernel(const KernelArgs a, const T* __restrict__ k_prompt,
                                                                  const T* __restrict__ v_prompt, int ctx) {
  const Geometry& g = a.geo;
  pdl_prologue();
  QE_TRACE_SCOPE(a.trace, 4);
  int32_t* cnt = a.st.mig_count + 2 * (a.unit0 / g.batch);
  const int4* queue = a.st.mig_queue + (size_t)a.unit0 * (g.PF + g.Kq + g.Kf) * 2;
  int n_entries = *reinterpret_cast<volatile int32_t*>(cnt + a.mig_parity);
#ifdef QEVICT_DEBUG_BOUNDS
  if (!QE_IN_RANGE(n_entries >= 0 && (long long)n_entries <= (long long)a.n_units * (g.PF + g.Kq + g.Kf), a.st.status, CHECK_BOUNDS_RECORD))
    n_entries = 0;
#endif
  // the next routing event of these units counts in the other counter: nothing reads it before this kernel ends
  if (blockIdx.x == 0 && threadIdx.x == 0) cnt[a.mig_parity ^ 1] = 0;
  const int lane = threadIdx.x & 31;
  const int gw = blockIdx.x * (MIGRATE_THREADS / 32) + (threadIdx.x >> 5), n_warps = gridDim.x * (MIGRATE_THREADS / 32);
  const int ks_n = g.D >> 4, ng = g.D / g.group;
  const int n_kt = (g.W / g.group) * ks_n, n_vt = g.tiles * ng * 2, tpp = n_kt > n_vt ? n_kt : n_vt;
  const int per_rec = g.Hkv * 2 * tpp, total = n_entries * per_rec;
#pragma unroll 1
  for (int id = gw; id < total; id += n_warps) {
    const int rec = id / per_rec, rem = id - rec * per_rec, hp = rem / tpp, task = rem - hp * tpp;
    const int hk = hp >> 1, part = hp & 1;
    if (task >= (part ? n_vt : n_kt)) continue;
    const int4 r0 = queue[2 * rec], r1 = queue[2 * rec + 1];
    const int u = r0.x, kind = r0.y, ul = u - a.unit0;
    if (kind == 2) continue;
#ifdef QEVICT_DEBUG_BOUNDS
    {  // a record whose unit, kind, window or pages are out of range is recorded and skipped
      bool ok = ul >= 0 && ul < a.n_units && kind >= 0 && kind <= 1 && r0.z >= 0 && r0.z < g.NW;
      if (kind == 0) ok = ok && r0.w >= -1 && r0.w < g.PF && r1.x >= 0 && r1.x < g.PQ && r1.y >= -1 && r1.y < g.PQ &&
                          (r0.w >= 0 || (k_prompt && (long long)(r0.z + 1) * g.W <= ctx)) && (r1.y < 0 || r0.w >= 0);
      else ok = ok && r0.w >= 0 && r0.w < g.PQ && r1.x >= 0 && r1.x < g.PF;
      if (!ok) {
        if (lane == 0) record_check(a.st.status, CHECK_BOUNDS_RECORD);
        continue;
      }
    }
#endif
    char* fp_u = a.st.fp_pool + (size_t)u * g.PF * g.fp_page_bytes + (size_t)hk * g.fp_head_bytes;
    char* q_u = a.st.q_pool + (size_t)u * g.PQ * g.q_page_bytes + (size_t)hk * g.q_head_bytes;
    // task coordinates
    int c0, c1, c2 = 0;
    if (part == 0) { c0 = task / ks_n; c1 = task - c0 * ks_n; }                    // (blk, ks)
    else { c2 = task & 1; c1 = (task >> 1) % ng; c0 = (task >> 1) / ng; }           // (tile, gc, ks)
    // one promotion at most follows: the record's own (kind 1) or the one linked to its quantization
    const char* pq = nullptr;
    char* pf = nullptr;
    if (kind == 0) {
      const T* rows = nullptr;
      const char* fp_head = nullptr;
      if (r0.w < 0) rows = (part ? v_prompt : k_prompt) + (((size_t)ul * g.Hkv + hk) * ctx + (size_t)r0.z * g.W) * g.D;
      else fp_head = fp_u + (size_t)r0.w * g.fp_page_bytes;
      char* qb = q_u + (size_t)r1.x * g.q_page_bytes;
      if (part == 0) quant_key_task<T>(g, c0, c1, rows, fp_head, qb, lane);
      else quant_value_task<T>(g, c0, c1, c2, rows, fp_head, qb, lane);
      if (r1.y >= 0) {
        pq = q_u + (size_t)r1.y * g.q_page_bytes;
        pf = fp_u + (size_t)r0.w * g.fp_page_bytes;
      }
    } else {
      pq = q_u + (size_t)r0.w * g.q_page_bytes;
      pf = fp_u + (size_t)r1.x * g.fp_page_bytes;
    }
    if (pq) {
      if (part == 0) promote_key_task<T>(g, c0, c1, pq, pf, lane);
      else promote_value_task<T>(g, c0, c1, c2, pq, pf, lane);
    }
  }
}

// One CTA per (list item, KV head): prompt rows -> fragment-major full-precision page.
template <class T>
__global__ void __launch_bounds__(PAGE_THREADS) copy_prompt_kernel(const KernelArgs a, const T* __restrict__ k_prompt,
                                                                   const T* __restrict__ v_prompt, int ctx) {
  const Geometry& g = a.geo;
  const int ul = blockIdx.z, u = a.unit0 + ul, hk = blockIdx.y;
  const int n_items = a.st.n_copy[u];
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
  const int4 it = a.st.copy_list[(size_t)u * g.Kfp + item];
  const int w = it.x, dst = it.y, D = g.D;
  if (!QE_IN_RANGE(w >= 0 && (long long)(w + 1) * g.W <= ctx && dst >= 0 && dst < g.PF, a.st.status, CHECK_BOUNDS_RECORD)) continue;
  const T* kr = k_prompt + (((size_t)ul * g.Hkv + hk) * ctx + (size_t)w * g.W) * D;
  const T* vr = v_prompt + (((size_t)ul * g.Hkv + hk) * ctx + (size_t)w * g.W) * D;
  char* fb = a.st.fp_pool + ((size_t)u * g.PF + dst) * g.fp_page_bytes + (size_t)hk * g.fp_head_bytes;
  for (int tile = 0; tile < g.tiles; ++tile) {
    T* kt = reinterpret_cast<T*>(fb + (size_t)tile * 2 * g.fp_tile_bytes);
    T* vt = reinterpret_cast<T*>(fb + (size_t)tile * 2 * g.fp_tile_bytes + g.fp_tile_bytes);
    for (int i = threadIdx.x; i < 32 * D; i += PAGE_THREADS) {
      const int tk = i / D, ch = i - tk * D;
      kt[fpk_off(tk, ch, D)] = kr[(size_t)(tile * 32 + tk) * D + ch];
      vt[fpv_off(tk, ch)] = vr[(size_t)(tile * 32 + tk) * D + ch];
    }
  }
  }
}

template <class T>
__global__ void export_fp_page_kernel(const KernelArgs a, int u, int page, T* __restrict__ k_out, T* __restrict__ v_out) {
  const Geometry& g = a.geo;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;  // over [Hkv][W][D]
  if (i >= g.Hkv * g.W * g.D) return;
  const int ch = i % g.D, tk = (i / g.D) % g.W, h = i / (g.D * g.W);
  const char* hb = a.st.fp_pool + ((size_t)u * g.PF + page) * g.fp_page_bytes + (size_t)h * g.fp_head_bytes;
  const int tile = tk >> 5;
  const T* kt = reinterpret_cast<const T*>(hb + (size_t)tile * 2 * g.fp_tile_bytes);
  const T* vt = reinterpret_cast<const T*>(hb + (size_t)tile * 2 * g.fp_tile_bytes + g.fp_tile_bytes);
  k_out[i] = kt[fpk_off(tk & 31, ch, g.D)];
  v_out[i] = vt[fpv_off(tk & 31, ch)];
}

template <class T>
__global__ void export_q_page_kernel(const KernelArgs a, int u, int page, uint8_t* __restrict__ k_codes,
                                     T* __restrict__ k_params, uint8_t* __restrict__ v_codes, T* __restrict__ v_params) {
  const Geometry& g = a.geo;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;  // over [Hkv][W][D]
  if (i >= g.Hkv * g.W * g.D) return;
  const int D = g.D, W = g.W, G = g.group;
  const int ch = i % D, tk = (i / D) % W, h = i / (D * W);
  const char* qb = a.st.q_pool + ((size_t)u * g.PQ + page) * g.q_page_bytes + (size_t)h * g.q_head_bytes;
  const int tile = tk >> 5, tkk = tk & 31;
  const uint32_t cmask = (1u << g.bits) - 1u;
  const uint32_t* kc = reinterpret_cast<const uint32_t*>(qb + (size_t)tile * g.q_tile_stride);
  const uint32_t* vc = reinterpret_cast<const uint32_t*>(qb + (size_t)tile * g.q_tile_stride + g.q_kc_bytes);
  const CodePos pk = kcode_pos(tkk, ch, D, g.bits), pv = vcode_pos(tkk, ch, g.bits);
  k_codes[i] = (uint8_t)((kc[pk.word] >> pk.shift) & cmask);
  v_codes[i] = (uint8_t)((vc[pv.word] >> pv.shift) & cmask);
  if (tk % G == 0) {  // key params [Hkv][W/G][D][2]
    const T* kp = reinterpret_cast<const T*>(qb + g.q_kp_off + (size_t)(tk / G) * g.q_kp_bytes);
    const size_t o = (((size_t)h * (W / G) + tk / G) * D + ch) * 2;
    k_params[o] = kp[kparam_off(ch, 0)];
    k_params[o + 1] = kp[kparam_off(ch, 1)];
  }
  if (ch % G == 0) {  // value params [Hkv][W][D/G][2]
    const T* vp = reinterpret_cast<const T*>(qb + (size_t)tile * g.q_tile_stride + g.q_kc_bytes + g.q_vc_bytes);
    const size_t o = (((size_t)h * W + tk) * (D / G) + ch / G) * 2;
    v_params[o] = vp[vparam_off(tkk, ch / G, 0)];
    v_params[o + 1] = vp[vparam_off(tkk, ch / G, 1)];
  }
}

}  // namespace

// CTAs per (unit, KV head) that walk a migration list: as many as there can be items, but no more
// than keeps the whole launch near two thousand CTAs (lists are mostly short or empty at decode time).
static int items_grid(int max_items, const KernelArgs& a) {
  const int pairs = a.geo.Hkv * 2 * a.n_units;
  int per = 1024 / (pairs > 0 ? pairs : 1);
  if (per < 1) per = 1;
  return max_items < per ? max_items : per;
}

#define QE_BY_DTYPE(geo, CALL_H, CALL_B) \
  do { if ((geo).dtype == QEVICT_DTYPE_FP16) { CALL_H; } else { CALL_B; } } while (0)

cudaError_t launch_migrate(const KernelArgs& a, const void* k_prompt, const void* v_prompt, int ctx, int max_items,
                           cudaStream_t s) {
  if (max_items <= 0) return cudaSuccess;
  // warp tasks there can be at most, capped at the CTAs that are resident at once (6 per SM)
  const int ks_n = a.geo.D >> 4, n_kt = (a.geo.W / a.geo.group) * ks_n, n_vt = a.geo.tiles * (a.geo.D / a.geo.group) * 2;
  const long long bound = ((long long)max_items * a.n_units * a.geo.Hkv * 2 * (n_kt > n_vt ? n_kt : n_vt) + 3) / 4;
  dim3 grid((unsigned)(bound < 888 ? bound : 888));
  const size_t sm = 0;
  if (a.geo.dtype == QEVICT_DTYPE_FP16)
    return launch_pdl(migrate_kernel<__half>, grid, dim3(MIGRATE_THREADS), sm, s, a, (const __half*)k_prompt, (const __half*)v_prompt, ctx);
  return launch_pdl(migrate_kernel<__nv_bfloat16>, grid, dim3(MIGRATE_THREADS), sm, s, a, (const __nv_bfloat16*)k_prompt,
                    (const __nv_bfloat16*)v_prompt, ctx);
}

cudaError_t launch_copy_prompt(const KernelArgs& a, const void* k_prompt, const void* v_prompt, int ctx, int max_items,
                               cudaStream_t s) {
  if (max_items <= 0) return cudaSuccess;
  dim3 grid(items_grid(max_items, a), a.geo.Hkv, a.n_units);
  QE_BY_DTYPE(a.geo,
              (copy_prompt_kernel<__half><<<grid, PAGE_THREADS, 0, s>>>(a, (const __half*)k_prompt, (const __half*)v_prompt, ctx)),
              (copy_prompt_kernel<__nv_bfloat16><<<grid, PAGE_THREADS, 0, s>>>(a, (const __nv_bfloat16*)k_prompt,
                                                                           (const __nv_bfloat16*)v_prompt, ctx)));
  return cudaGetLastError();
}

cudaError_t launch_export_fp_page(const KernelArgs& a, int unit, int page, void* k_out, void* v_out, cudaStream_t s) {
  const int n = a.geo.Hkv * a.geo.W * a.geo.D;
  QE_BY_DTYPE(a.geo, (export_fp_page_kernel<__half><<<(n + 255) / 256, 256, 0, s>>>(a, unit, page, (__half*)k_out, (__half*)v_out)),
              (export_fp_page_kernel<__nv_bfloat16><<<(n + 255) / 256, 256, 0, s>>>(a, unit, page, (__nv_bfloat16*)k_out,
                                                                                (__nv_bfloat16*)v_out)));
  return cudaGetLastError();
}

cudaError_t launch_export_q_page(const KernelArgs& a, int unit, int page, uint8_t* k_codes, void* k_params,
                                 uint8_t* v_codes, void* v_params, cudaStream_t s) {
  const int n = a.geo.Hkv * a.geo.W * a.geo.D;
  QE_BY_DTYPE(a.geo,
              (export_q_page_kernel<__half><<<(n + 255) / 256, 256, 0, s>>>(a, unit, page, k_codes, (__half*)k_params, v_codes,
                                                                        (__half*)v_params)),
              (export_q_page_kernel<__nv_bfloat16><<<(n + 255) / 256, 256, 0, s>>>(a, unit, page, k_codes, (__nv_bfloat16*)k_params,
                                                                               v_codes, (__nv_bfloat16*)v_params)));
  return cudaGetLastError();
}

}  // namespace qevict
