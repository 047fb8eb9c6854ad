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
constexpr int MIGRATE_THREADS = 256;

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

__device__ __forceinline__ uint32_t quant_code(float x, float z, float s, int qmax, bool bad) {
  if (bad) return 0u;
  const float tq = rintf(__fdiv_rn(__fsub_rn(x, z), s));
  const int c = (int)fminf(fmaxf(tq, 0.f), (float)qmax);
  return (uint32_t)c;
}

// ---- quantize one half (keys or values) of one window of one KV head ------------------------------------
// Shared memory: the half in plain [W][D] order and its parameters as floats.  Every thread then builds
// whole 32-bit code words (no atomics) and stores them straight into the page.
template <class T>
__device__ void quantize_part(const Geometry& g, int part, const T* __restrict__ rows /* prompt rows or null */,
                              const char* __restrict__ fp_head /* source page head or null */, char* qb,
                              unsigned char* smem_raw) {
  const int tid = threadIdx.x, W = g.W, D = g.D, G = g.group, qmax = (1 << g.bits) - 1;
  T* sx = reinterpret_cast<T*>(smem_raw);                       // [W][D]
  float* sf = reinterpret_cast<float*>(sx + W * D);             // scale (or -1 if the group is degenerate)
  float* zf = sf + (part == 0 ? (W / G) * D : W * (D / G));     // zero
  const int KG = D / 32;

  // ---- stage the half in plain order ---------------------------------------------------------------
  if (rows) {
    const uint4* r4 = reinterpret_cast<const uint4*>(rows);
    for (int i = tid; i < W * D / 8; i += MIGRATE_THREADS) reinterpret_cast<uint4*>(sx)[i] = r4[i];
  } else {
    // the page is fragment-major: 16-byte loads (many in flight), each vector scattered to plain positions
    const int nvec = 32 * D / 8;
    for (int tile = 0; tile < g.tiles; ++tile) {
      const uint4* src = reinterpret_cast<const uint4*>(fp_head + (size_t)tile * 2 * g.fp_tile_bytes + (part ? g.fp_tile_bytes : 0));
#pragma unroll 4
      for (int v = tid; v < nvec; v += MIGRATE_THREADS) {
        const uint4 x = src[v];
        const int ln = v & 31, vec = v >> 5, gg = ln >> 2, tt = ln & 3;
        const T* xe = reinterpret_cast<const T*>(&x);
#pragma unroll
        for (int el = 0; el < 8; ++el) {
          const int a1 = el >> 2, a2 = (el >> 1) & 1, e = el & 1;
          int tk, ch;
          // element el of a vector = register (a1*2 + a2), half e
          if (part == 0) { const int kks = vec >> 1, kmt = vec & 1; tk = 16 * kmt + 8 * a2 + gg; ch = 16 * kks + 8 * a1 + 2 * tt + e; }
          else { const int vi = vec >> 1, vks = vec & 1; tk = 16 * vks + 8 * a1 + 2 * tt + e; ch = 16 * vi + 8 * a2 + gg; }
          sx[(tile * 32 + tk) * D + ch] = xe[el];
        }
      }
    }
  }
  __syncthreads();

  // ---- parameters ----------------------------------------------------------------------------------
  if (part == 0) {  // keys: one group per (block of G tokens, channel)
    for (int i = tid; i < (W / G) * D; i += MIGRATE_THREADS) {
      const int blk = i / D, ch = i - blk * D;
      float mn = INFINITY, mx = -INFINITY;
      for (int tk = blk * G; tk < (blk + 1) * G; ++tk) {
        const float x = Tr<T>::to_float(sx[tk * D + ch]);
        mn = fminf(mn, x); mx = fmaxf(mx, x);
      }
      T st, zt; float s; bool bad;
      group_params<T>(mn, mx, qmax, st, zt, s, bad);
      sf[i] = bad ? -1.f : s;
      zf[i] = mn;
      T* kp = reinterpret_cast<T*>(qb + g.q_kp_off + (size_t)blk * g.q_kp_bytes);
      kp[kparam_off(ch, 0)] = st;
      kp[kparam_off(ch, 1)] = zt;
    }
  } else {  // values: one group per (token, block of G channels)
    const int ng = D / G;
    for (int i = tid; i < W * ng; i += MIGRATE_THREADS) {
      const int gc = i / W, tk = i - gc * W;  // consecutive threads take consecutive tokens
      float mn = INFINITY, mx = -INFINITY;
      for (int k = 0; k < G; ++k) {
        const int ch = gc * G + ((k + tk) & (G - 1));  // rotated start: spreads the threads over the banks
        const float x = Tr<T>::to_float(sx[tk * D + ch]);
        mn = fminf(mn, x); mx = fmaxf(mx, x);
      }
      T st, zt; float s; bool bad;
      group_params<T>(mn, mx, qmax, st, zt, s, bad);
      sf[tk * ng + gc] = bad ? -1.f : s;
      zf[tk * ng + gc] = mn;
      T* vp = reinterpret_cast<T*>(qb + (size_t)(tk >> 5) * g.q_tile_stride + g.q_kc_bytes + g.q_vc_bytes);
      vp[vparam_off(tk & 31, gc, 0)] = st;
      vp[vparam_off(tk & 31, gc, 1)] = zt;
    }
  }
  __syncthreads();

  // ---- codes: one 32-bit word (8 or 16 codes) per thread and iteration ----------------------------------
  const int words_per_tile = g.q_kc_bytes / 4;
  const int cpw = 32 / g.bits;  // codes per word
  for (int tile = 0; tile < g.tiles; ++tile) {
    uint32_t* dstw = reinterpret_cast<uint32_t*>(qb + (size_t)tile * g.q_tile_stride + (part ? g.q_kc_bytes : 0));
    for (int wo = tid; wo < words_per_tile; wo += MIGRATE_THREADS) {
      // word offset -> (word index of the lane, lane)
      const int q4 = wo >> 2, ln = q4 & 31, widx = (q4 >> 5) * 4 + (wo & 3), gg = ln >> 2, tt = ln & 3;
      uint32_t word = 0u;
      for (int k = 0; k < cpw; ++k) {
        // slot k of the word: sub-word (2-bit only), register m / a, element e
        const int e = k & 1, m = (k >> 1) & 3, sub = k >> 3;
        int tk, ch;
        if (part == 0) {
          const int ks = g.bits == 4 ? (widx >> 1) : widx;
          const int mt = g.bits == 4 ? (widx & 1) : sub;
          tk = 16 * mt + 8 * (m & 1) + gg;
          ch = 16 * ks + 8 * (m >> 1) + 2 * tt + e;
        } else {
          const int i = g.bits == 4 ? (widx >> 1) : widx;
          const int ks = g.bits == 4 ? (widx & 1) : sub;
          tk = 16 * ks + 8 * (m >> 1) + 2 * tt + e;
          ch = 16 * i + 8 * (m & 1) + gg;
        }
        const int row = tile * 32 + tk;
        const int pi = part == 0 ? (row / G) * D + ch : row * (D / G) + ch / G;
        const float s = sf[pi];
        const uint32_t code = quant_code(Tr<T>::to_float(sx[row * D + ch]), zf[pi], s, qmax, s < 0.f);
        word |= code << (g.bits * (sub * 4 + m) + 16 * e);
      }
      dstw[wo] = word;
    }
  }
}

// ---- dequantize one half of one window of one KV head into a full-precision page -----------------------
// Produces exactly the operand registers the decode kernel forms in flight.
template <class T>
__device__ void promote_part(const Geometry& g, int part, const char* __restrict__ qb, char* fb) {
  const int D = g.D, KG = D / 32, MT = D / 16, bits = g.bits;
  const uint32_t mask = bits == 4 ? 0x000F000Fu : 0x00030003u, MG = Tr<T>::MAGIC;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, t = lane & 3, nwarps = MIGRATE_THREADS / 32;
  for (int tile = 0; tile < g.tiles; ++tile) {
    const char* tb = qb + (size_t)tile * g.q_tile_stride;
    if (part == 0) {
      const uint32_t* kc = reinterpret_cast<const uint32_t*>(tb);
      const uint4* kp = reinterpret_cast<const uint4*>(qb + g.q_kp_off + (size_t)((tile * 32) / g.group) * g.q_kp_bytes);
      uint4* kt = reinterpret_cast<uint4*>(fb + (size_t)tile * 2 * g.fp_tile_bytes);
      for (int v = wid; v < 2 * (D / 16); v += nwarps) {  // key vectors (ks, mt)
        const int ks = v >> 1, mt = v & 1;
        const int widx = bits == 4 ? ks * 2 + mt : ks;
        const int sh = bits == 4 ? 0 : mt * 8;
        const uint32_t w = kc[code_word_off(widx, lane)];
        const uint4 pr = kp[ks * 4 + t];
        uint4 r;
        r.x = dequant2<T>(and_or(w >> (sh + 0 * bits), mask, MG), pr.x, pr.y);
        r.y = dequant2<T>(and_or(w >> (sh + 1 * bits), mask, MG), pr.x, pr.y);
        r.z = dequant2<T>(and_or(w >> (sh + 2 * bits), mask, MG), pr.z, pr.w);
        r.w = dequant2<T>(and_or(w >> (sh + 3 * bits), mask, MG), pr.z, pr.w);
        kt[v * 32 + lane] = r;
      }
    } else {
      const uint32_t* vc = reinterpret_cast<const uint32_t*>(tb + g.q_kc_bytes);
      const uint4* vp = reinterpret_cast<const uint4*>(tb + g.q_kc_bytes + g.q_vc_bytes);
      uint4* vt = reinterpret_cast<uint4*>(fb + (size_t)tile * 2 * g.fp_tile_bytes + g.fp_tile_bytes);
      for (int v = wid; v < 2 * MT; v += nwarps) {  // value vectors (i, ks)
        const int i = v >> 1, ks = v & 1;
        const int widx = bits == 4 ? i * 2 + ks : i;
        const int sh = bits == 4 ? 0 : ks * 8;
        const uint32_t w = vc[code_word_off(widx, lane)];
        const int gc = (16 * i) / g.group;
        const uint4 pr = vp[(gc * 2 + ks) * 4 + t];
        uint4 r;
        r.x = dequant2<T>(and_or(w >> (sh + 0 * bits), mask, MG), pr.x, pr.y);
        r.y = dequant2<T>(and_or(w >> (sh + 1 * bits), mask, MG), pr.x, pr.y);
        r.z = dequant2<T>(and_or(w >> (sh + 2 * bits), mask, MG), pr.z, pr.w);
        r.w = dequant2<T>(and_or(w >> (sh + 3 * bits), mask, MG), pr.z, pr.w);
        vt[v * 32 + lane] = r;
      }
    }
  }
}

// Migration kernel.  CTA = (list slot, KV head x {keys, values}, unit); it walks the unit's quantization
// list and then the promotions nobody else handles.  A promotion whose new full-precision page is the
// page a quantization of the same event reads from is linked to that quantization and runs in the same
// CTA right after it, so no page is overwritten before it has been read.
template <class T>
__global__ void __launch_bounds__(MIGRATE_THREADS) migrate_kernel(const KernelArgs a, const T* __restrict__ k_prompt,
                                                                  const T* __restrict__ v_prompt, int ctx) {
  const Geometry& g = a.geo;
  const int ul = blockIdx.z, u = a.unit0 + ul, hk = blockIdx.y >> 1, part = blockIdx.y & 1;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_prologue();
  const int n_quant = a.st.n_quant[u], n_promote = a.st.n_promote[u];
  const int4* quant_list = a.st.quant_list + (size_t)u * (g.PF + g.Kq);
  const int4* promote_list = a.st.promote_list + (size_t)u * g.Kf;
  auto promote = [&](int k) {
    const int4 it = promote_list[k];
    promote_part<T>(g, part, a.st.q_pool + ((size_t)u * g.PQ + it.y) * g.q_page_bytes + (size_t)hk * g.q_head_bytes,
                    a.st.fp_pool + ((size_t)u * g.PF + it.z) * g.fp_page_bytes + (size_t)hk * g.fp_head_bytes);
  };
  for (int item = blockIdx.x; item < n_quant + n_promote; item += gridDim.x) {
    if (item < n_quant) {
      const int4 it = quant_list[item];  // {window, source page (-1: prompt), destination page, linked promotion}
      const T* rows = nullptr;
      const char* fp_head = nullptr;
      if (it.y < 0) rows = (part ? v_prompt : k_prompt) + (((size_t)ul * g.Hkv + hk) * ctx + (size_t)it.x * g.W) * g.D;
      else fp_head = a.st.fp_pool + ((size_t)u * g.PF + it.y) * g.fp_page_bytes + (size_t)hk * g.fp_head_bytes;
      __syncthreads();  // the staging buffer is reused from item to item
      quantize_part<T>(g, part, rows, fp_head,
                       a.st.q_pool + ((size_t)u * g.PQ + it.z) * g.q_page_bytes + (size_t)hk * g.q_head_bytes, smem_raw);
      if (it.w >= 0) {
        __syncthreads();  // every thread has finished reading the source page
        promote(it.w);
      }
    } else {
      const int k = item - n_quant;
      if (promote_list[k].w == 0) promote(k);  // not linked to a quantization
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
  const int4 it = a.st.copy_list[(size_t)u * g.Kf + item];
  const int w = it.x, dst = it.y, D = g.D;
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

size_t migrate_smem_bytes(const Geometry& g) {
  const size_t params = (size_t)((g.W / g.group) * g.D > g.W * (g.D / g.group) ? (g.W / g.group) * g.D : g.W * (g.D / g.group));
  return (size_t)g.W * g.D * 2 + 2 * params * 4;
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
  dim3 grid(items_grid(max_items, a), a.geo.Hkv * 2, a.n_units);
  const size_t sm = migrate_smem_bytes(a.geo);
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
