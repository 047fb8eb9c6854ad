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

// One CTA per (list item, KV head).  Shared memory: K and V of the window in plain [W][D] order,
// the packed code words, and the parameters as floats.
template <class T>
__global__ void __launch_bounds__(PAGE_THREADS) quantize_kernel(const KernelArgs a, const T* __restrict__ k_prompt,
                                                                const T* __restrict__ v_prompt, int ctx) {
  const Geometry& g = a.geo;
  const int ul = blockIdx.z, u = a.unit0 + ul, hk = blockIdx.y, item = blockIdx.x, tid = threadIdx.x;
  if (item >= a.st.n_quant[u]) return;
  const int4 it = a.st.quant_list[(size_t)u * (g.PF + g.Kq) + item];
  const int w = it.x, src = it.y, dst = it.z;
  const int W = g.W, D = g.D, G = g.group, qmax = (1 << g.bits) - 1;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* sk = reinterpret_cast<T*>(smem_raw);                   // [W][D]
  T* sv = sk + W * D;                                       // [W][D]
  uint32_t* kw = reinterpret_cast<uint32_t*>(sv + W * D);   // [tiles][kc words]
  const int words_per_tile = g.q_kc_bytes / 4;
  uint32_t* vw = kw + g.tiles * words_per_tile;             // [tiles][vc words]
  float* ksf = reinterpret_cast<float*>(vw + g.tiles * words_per_tile);  // [W/G][D] scale (or -1 if bad)
  float* kzf = ksf + (W / G) * D;
  float* vsf = kzf + (W / G) * D;                           // [W][D/G]
  float* vzf = vsf + W * (D / G);

  // ---- stage the window in plain order -----------------------------------------------------------
  if (src < 0) {
    const T* kr = k_prompt + (((size_t)ul * g.Hkv + hk) * ctx + (size_t)w * W) * D;
    const T* vr = v_prompt + (((size_t)ul * g.Hkv + hk) * ctx + (size_t)w * W) * D;
    const uint4* k4 = reinterpret_cast<const uint4*>(kr);
    const uint4* v4 = reinterpret_cast<const uint4*>(vr);
    for (int i = tid; i < W * D / 8; i += PAGE_THREADS) {
      reinterpret_cast<uint4*>(sk)[i] = k4[i];
      reinterpret_cast<uint4*>(sv)[i] = v4[i];
    }
  } else {
    const char* hb = a.st.fp_pool + ((size_t)u * g.PF + src) * g.fp_page_bytes + (size_t)hk * g.fp_head_bytes;
    for (int tile = 0; tile < g.tiles; ++tile) {
      const T* kt = reinterpret_cast<const T*>(hb + (size_t)tile * 2 * g.fp_tile_bytes);
      const T* vt = reinterpret_cast<const T*>(hb + (size_t)tile * 2 * g.fp_tile_bytes + g.fp_tile_bytes);
      for (int i = tid; i < 32 * D; i += PAGE_THREADS) {
        const int tk = i / D, ch = i - tk * D;
        sk[(tile * 32 + tk) * D + ch] = kt[fpk_off(tk, ch, D)];
        sv[(tile * 32 + tk) * D + ch] = vt[fpv_off(tk, ch)];
      }
    }
  }
  for (int i = tid; i < 2 * g.tiles * words_per_tile; i += PAGE_THREADS) kw[i] = 0u;
  __syncthreads();

  char* qb = a.st.q_pool + ((size_t)u * g.PQ + dst) * g.q_page_bytes + (size_t)hk * g.q_head_bytes;

  // ---- parameters --------------------------------------------------------------------------------
  for (int i = tid; i < (W / G) * D; i += PAGE_THREADS) {  // keys: (token block, channel)
    const int blk = i / D, ch = i - blk * D;
    float mn = INFINITY, mx = -INFINITY;
    for (int tk = blk * G; tk < (blk + 1) * G; ++tk) {
      const float x = Tr<T>::to_float(sk[tk * D + ch]);
      mn = fminf(mn, x); mx = fmaxf(mx, x);
    }
    T st, zt; float sf; bool bad;
    group_params<T>(mn, mx, qmax, st, zt, sf, bad);
    ksf[i] = bad ? -1.f : sf;
    kzf[i] = mn;
    T* kp = reinterpret_cast<T*>(qb + g.q_kp_off + (size_t)blk * g.q_kp_bytes);
    kp[kparam_off(ch, 0)] = st;
    kp[kparam_off(ch, 1)] = zt;
  }
  for (int i = tid; i < W * (D / G); i += PAGE_THREADS) {  // values: (token, channel block)
    const int tk = i / (D / G), gc = i - tk * (D / G);
    float mn = INFINITY, mx = -INFINITY;
    for (int ch = gc * G; ch < (gc + 1) * G; ++ch) {
      const float x = Tr<T>::to_float(sv[tk * D + ch]);
      mn = fminf(mn, x); mx = fmaxf(mx, x);
    }
    T st, zt; float sf; bool bad;
    group_params<T>(mn, mx, qmax, st, zt, sf, bad);
    vsf[i] = bad ? -1.f : sf;
    vzf[i] = mn;
    const int tile = tk >> 5;
    T* vp = reinterpret_cast<T*>(qb + (size_t)tile * g.q_tile_stride + g.q_kc_bytes + g.q_vc_bytes);
    vp[vparam_off(tk & 31, gc, 0)] = st;
    vp[vparam_off(tk & 31, gc, 1)] = zt;
  }
  __syncthreads();

  // ---- codes -------------------------------------------------------------------------------------
  for (int i = tid; i < W * D; i += PAGE_THREADS) {
    const int tk = i / D, ch = i - tk * D;
    const int tile = tk >> 5, tkk = tk & 31;
    {
      const int pi = (tk / G) * D + ch;
      const float s = ksf[pi];
      const uint32_t c = quant_code(Tr<T>::to_float(sk[i]), kzf[pi], s, qmax, s < 0.f);
      const CodePos p = kcode_pos(tkk, ch, D, g.bits);
      atomicOr(&kw[tile * words_per_tile + p.word], c << p.shift);
    }
    {
      const int pi = tk * (D / G) + ch / G;
      const float s = vsf[pi];
      const uint32_t c = quant_code(Tr<T>::to_float(sv[i]), vzf[pi], s, qmax, s < 0.f);
      const CodePos p = vcode_pos(tkk, ch, g.bits);
      atomicOr(&vw[tile * words_per_tile + p.word], c << p.shift);
    }
  }
  __syncthreads();
  for (int tile = 0; tile < g.tiles; ++tile) {
    uint4* kc = reinterpret_cast<uint4*>(qb + (size_t)tile * g.q_tile_stride);
    uint4* vc = reinterpret_cast<uint4*>(qb + (size_t)tile * g.q_tile_stride + g.q_kc_bytes);
    for (int i = tid; i < words_per_tile / 4; i += PAGE_THREADS) {
      kc[i] = reinterpret_cast<const uint4*>(kw + tile * words_per_tile)[i];
      vc[i] = reinterpret_cast<const uint4*>(vw + tile * words_per_tile)[i];
    }
  }
}

// One CTA per (list item, KV head): rebuild the window from its codes into a full-precision page,
// producing exactly the operand registers the decode kernel forms in flight.
template <class T>
__global__ void __launch_bounds__(PAGE_THREADS) promote_kernel(const KernelArgs a) {
  const Geometry& g = a.geo;
  const int u = a.unit0 + blockIdx.z, hk = blockIdx.y, item = blockIdx.x;
  if (item >= a.st.n_promote[u]) return;
  const int4 it = a.st.promote_list[(size_t)u * g.Kf + item];
  const int srcq = it.y, dst = it.z;
  const int D = g.D, KG = D / 32, MT = D / 16, bits = g.bits;
  const uint32_t mask = bits == 4 ? 0x000F000Fu : 0x00030003u, MG = Tr<T>::MAGIC;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, t = lane & 3, nwarps = PAGE_THREADS / 32;
  const char* qb = a.st.q_pool + ((size_t)u * g.PQ + srcq) * g.q_page_bytes + (size_t)hk * g.q_head_bytes;
  char* fb = a.st.fp_pool + ((size_t)u * g.PF + dst) * g.fp_page_bytes + (size_t)hk * g.fp_head_bytes;
  for (int tile = 0; tile < g.tiles; ++tile) {
    const uint32_t* kc = reinterpret_cast<const uint32_t*>(qb + (size_t)tile * g.q_tile_stride);
    const uint32_t* vc = reinterpret_cast<const uint32_t*>(qb + (size_t)tile * g.q_tile_stride + g.q_kc_bytes);
    const uint4* vp = reinterpret_cast<const uint4*>(qb + (size_t)tile * g.q_tile_stride + g.q_kc_bytes + g.q_vc_bytes);
    const uint4* kp = reinterpret_cast<const uint4*>(qb + g.q_kp_off + (size_t)((tile * 32) / g.group) * g.q_kp_bytes);
    uint4* kt = reinterpret_cast<uint4*>(fb + (size_t)tile * 2 * g.fp_tile_bytes);
    uint4* vt = reinterpret_cast<uint4*>(fb + (size_t)tile * 2 * g.fp_tile_bytes + g.fp_tile_bytes);
    for (int v = wid; v < 4 * KG; v += nwarps) {  // key vectors (j, c)
      const int j = v / KG, c = v - j * KG;
      const int widx = bits == 4 ? j * KG + c : j * (KG / 2) + (c >> 1);
      const int sh = bits == 4 ? 0 : (c & 1) * 8;
      const uint32_t w = kc[code_word_off(widx, lane)];
      const uint4 p0 = kp[(c * 2 + 0) * 4 + t], p1 = kp[(c * 2 + 1) * 4 + t];
      uint4 r;
      r.x = dequant2<T>(((w >> (sh + 0 * bits)) & mask) | MG, p0.x, p0.y);
      r.y = dequant2<T>(((w >> (sh + 1 * bits)) & mask) | MG, p0.z, p0.w);
      r.z = dequant2<T>(((w >> (sh + 2 * bits)) & mask) | MG, p1.x, p1.y);
      r.w = dequant2<T>(((w >> (sh + 3 * bits)) & mask) | MG, p1.z, p1.w);
      kt[v * 32 + lane] = r;
    }
    for (int v = wid; v < 2 * MT; v += nwarps) {  // value vectors (i, ks)
      const int i = v >> 1, ks = v & 1;
      const int widx = bits == 4 ? i * 2 + ks : i;
      const int sh = bits == 4 ? 0 : ks * 8;
      const uint32_t w = vc[code_word_off(widx, lane)];
      const int gc = (16 * i) / g.group;
      const uint4 pr = vp[(gc * 2 + ks) * 4 + t];
      uint4 r;
      r.x = dequant2<T>(((w >> (sh + 0 * bits)) & mask) | MG, pr.x, pr.y);
      r.y = dequant2<T>(((w >> (sh + 1 * bits)) & mask) | MG, pr.x, pr.y);
      r.z = dequant2<T>(((w >> (sh + 2 * bits)) & mask) | MG, pr.z, pr.w);
      r.w = dequant2<T>(((w >> (sh + 3 * bits)) & mask) | MG, pr.z, pr.w);
      vt[v * 32 + lane] = r;
    }
  }
}

// One CTA per (list item, KV head): prompt rows -> fragment-major full-precision page.
template <class T>
__global__ void __launch_bounds__(PAGE_THREADS) copy_prompt_kernel(const KernelArgs a, const T* __restrict__ k_prompt,
                                                                   const T* __restrict__ v_prompt, int ctx) {
  const Geometry& g = a.geo;
  const int ul = blockIdx.z, u = a.unit0 + ul, hk = blockIdx.y, item = blockIdx.x;
  if (item >= a.st.n_copy[u]) return;
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

size_t quantize_smem_bytes(const Geometry& g) {
  return (size_t)2 * g.W * g.D * 2 + (size_t)2 * g.tiles * g.q_kc_bytes +
         (size_t)(2 * (g.W / g.group) * g.D + 2 * g.W * (g.D / g.group)) * 4;
}

}  // namespace

#define QE_BY_DTYPE(geo, CALL_H, CALL_B) \
  do { if ((geo).dtype == QEVICT_DTYPE_FP16) { CALL_H; } else { CALL_B; } } while (0)

cudaError_t launch_quantize(const KernelArgs& a, const void* k_prompt, const void* v_prompt, int ctx, int max_items,
                            cudaStream_t s) {
  if (max_items <= 0) return cudaSuccess;
  dim3 grid(max_items, a.geo.Hkv, a.n_units);
  const size_t sm = quantize_smem_bytes(a.geo);
  QE_BY_DTYPE(a.geo,
              (quantize_kernel<__half><<<grid, PAGE_THREADS, sm, s>>>(a, (const __half*)k_prompt, (const __half*)v_prompt, ctx)),
              (quantize_kernel<__nv_bfloat16><<<grid, PAGE_THREADS, sm, s>>>(a, (const __nv_bfloat16*)k_prompt,
                                                                          (const __nv_bfloat16*)v_prompt, ctx)));
  return cudaGetLastError();
}

cudaError_t launch_promote(const KernelArgs& a, int max_items, cudaStream_t s) {
  if (max_items <= 0) return cudaSuccess;
  dim3 grid(max_items, a.geo.Hkv, a.n_units);
  QE_BY_DTYPE(a.geo, (promote_kernel<__half><<<grid, PAGE_THREADS, 0, s>>>(a)),
              (promote_kernel<__nv_bfloat16><<<grid, PAGE_THREADS, 0, s>>>(a)));
  return cudaGetLastError();
}

cudaError_t launch_copy_prompt(const KernelArgs& a, const void* k_prompt, const void* v_prompt, int ctx, int max_items,
                               cudaStream_t s) {
  if (max_items <= 0) return cudaSuccess;
  dim3 grid(max_items, a.geo.Hkv, a.n_units);
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
