// Tiered split-KV flash-decode kernel.
//
// One decode step attends every query head over the accessible tokens of its unit [attention
// equation of the Methodology] and records, per (query head, window), the window's softmax
// numerator, from which the combine kernel forms the window mass of Eq. 1.
//
// Work decomposition: CTA = (split, KV head, unit), 4 warps.  Warp `wid` of split `s` owns the work
// list entries s*4+wid, s*4+wid + 4S, ...; the list is ordered Full.., Quantized.., recent.., so a
// strided walk gives every warp the same mix of 16-bit and low-bit windows (balanced bytes).  Each
// warp runs an independent online softmax over its windows; the four warps are merged in shared
// memory and the CTA writes one partial (m, l, O) per query head of its KV head.
//
// Per 32-token tile:  S = Q K^T with the (<= 8) grouped heads on the M side of mma.m16n8k16 and
// tokens on N, softmax in fp32 in the log2 domain, O^T += V^T P^T with channels on M, tokens on K and
// heads on N, so the probability fragments feed the second product without any shuffle; the
// probabilities enter it as a 16-bit value plus its rounding residual (two products per fragment).  Pages are
// stored fragment-major (layout.cuh): a full-precision tile is read with 16-byte loads that are
// already operands; a quantized tile is read as packed words, and codes become operands in
// registers with one exact subtract and one fused multiply-add per pair.
#pragma once

#include "common.cuh"

namespace qevict {

struct DecodeParams {
  const void* q;          // [units in call][Hq][D]
  const uint2* entries;   // [n_units][EMAX]
  const int32_t* n_live;  // [n_units]
  const int32_t* open_fill;
  const char* fp_pool;
  const char* q_pool;
  float* o_part;          // [n_units][Hq][MAX_SPLITS][D]
  float* ml;              // [n_units][Hq][MAX_SPLITS][2]
  float2* wrec;           // [n_units][Hq][EMAX]
  int unit0, S, Hq, Hkv, G, EMAX, PF, PQ;
  uint32_t fp_page_bytes, q_page_bytes;
  float scale_log2;
};

template <class T, int D, int BITS, int GROUP, int TILES>
struct DecodeTraits {
  static constexpr int KG = D / 32;   // 16-byte key vectors per 8-token row block
  static constexpr int KS = D / 16;   // k-steps of the QK product
  static constexpr int MT = D / 16;   // m-tiles (16 channels) of the PV product
  static constexpr int W = TILES * 32;
  static constexpr uint32_t FP_TILE_BYTES = 32 * D * 2;
  static constexpr uint32_t FP_HEAD_BYTES = TILES * 2 * FP_TILE_BYTES;
  static constexpr uint32_t KC_BYTES = 32 * D * BITS / 8;
  static constexpr uint32_t VC_BYTES = KC_BYTES;
  static constexpr uint32_t VP_BYTES = 32 * (D / GROUP) * 4;
  static constexpr uint32_t Q_TILE_STRIDE = KC_BYTES + VC_BYTES + VP_BYTES;
  static constexpr uint32_t KP_BYTES = D * 4;
  static constexpr uint32_t KP_OFF = TILES * Q_TILE_STRIDE;
  static constexpr uint32_t Q_HEAD_BYTES = KP_OFF + (W / GROUP) * KP_BYTES;
  static constexpr int WPL = KC_BYTES / 128;  // code words per lane per tile (keys; same for values)
  static constexpr int STEP = BITS;           // bit distance between consecutive pair slots
  static constexpr uint32_t MASK = (BITS == 4) ? 0x000F000Fu : 0x00030003u;
};

// ---- S = Q K^T for one tile -----------------------------------------------------------------------
template <class T, int D, class LD>
__device__ __forceinline__ void qk_fp_tile(float (&s)[4][4], const uint32_t (&qa)[D / 16][2], const uint4* kt,
                                           int lane, LD ld) {
  constexpr int KG = D / 32;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
#pragma unroll
    for (int c = 0; c < KG; ++c) {
      const uint4 kv = ld(kt + (j * KG + c) * 32 + lane);
      mma16816<T>(s[j], qa[2 * c][0], 0u, qa[2 * c][1], 0u, kv.x, kv.y);
      mma16816<T>(s[j], qa[2 * c + 1][0], 0u, qa[2 * c + 1][1], 0u, kv.z, kv.w);
    }
  }
}

template <class T, int D, int BITS, class LD>
__device__ __forceinline__ void qk_q_tile(float (&s)[4][4], const uint32_t (&qa)[D / 16][2], const uint4* kc,
                                          const uint4* kp, int lane, LD ld) {
  constexpr int KG = D / 32;
  constexpr int WPL = 32 * D * BITS / 8 / 128;
  constexpr uint32_t MASK = (BITS == 4) ? 0x000F000Fu : 0x00030003u;
  constexpr uint32_t MG = Tr<T>::MAGIC;
  const int t = lane & 3;
  uint32_t cw[WPL];
#pragma unroll
  for (int v = 0; v < WPL / 4; ++v) {
    const uint4 x = ld(kc + v * 32 + lane);
    cw[4 * v] = x.x; cw[4 * v + 1] = x.y; cw[4 * v + 2] = x.z; cw[4 * v + 3] = x.w;
  }
#pragma unroll
  for (int c = 0; c < KG; ++c) {
    const uint4 p0 = ld(kp + (c * 2 + 0) * 4 + t);  // k-step 2c:   {s,z} for the low / high channel octet
    const uint4 p1 = ld(kp + (c * 2 + 1) * 4 + t);  // k-step 2c+1
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t w;
      int sh;
      if (BITS == 4) { w = cw[j * KG + c]; sh = 0; } else { w = cw[j * (KG / 2) + (c >> 1)]; sh = (c & 1) * 8; }
      const uint32_t b0 = dequant2<T>(((w >> (sh + 0 * BITS)) & MASK) | MG, p0.x, p0.y);
      const uint32_t b1 = dequant2<T>(((w >> (sh + 1 * BITS)) & MASK) | MG, p0.z, p0.w);
      const uint32_t b2 = dequant2<T>(((w >> (sh + 2 * BITS)) & MASK) | MG, p1.x, p1.y);
      const uint32_t b3 = dequant2<T>(((w >> (sh + 3 * BITS)) & MASK) | MG, p1.z, p1.w);
      mma16816<T>(s[j], qa[2 * c][0], 0u, qa[2 * c][1], 0u, b0, b1);
      mma16816<T>(s[j], qa[2 * c + 1][0], 0u, qa[2 * c + 1][1], 0u, b2, b3);
    }
  }
}

// ---- O^T += V^T P^T for one tile --------------------------------------------------------------------
template <class T, int D, class LD>
__device__ __forceinline__ void pv_fp_tile(float (&o)[D / 16][4], const uint32_t (&pa)[2][2],
                                           const uint32_t (&pb)[2][2], const uint4* vt, int lane, LD ld) {
#pragma unroll
  for (int i = 0; i < D / 16; ++i) {
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
      const uint4 vv = ld(vt + (i * 2 + ks) * 32 + lane);
      mma16816<T>(o[i], vv.x, vv.y, vv.z, vv.w, pa[ks][0], pa[ks][1]);
      mma16816<T>(o[i], vv.x, vv.y, vv.z, vv.w, pb[ks][0], pb[ks][1]);
    }
  }
}

template <class T, int D, int BITS, int GROUP, class LD>
__device__ __forceinline__ void pv_q_tile(float (&o)[D / 16][4], const uint32_t (&pa)[2][2],
                                          const uint32_t (&pb)[2][2], const uint4* vc, const uint4* vp, int lane,
                                          LD ld) {
  constexpr int MT = D / 16;
  constexpr int WPL = 32 * D * BITS / 8 / 128;
  constexpr uint32_t MASK = (BITS == 4) ? 0x000F000Fu : 0x00030003u;
  constexpr uint32_t MG = Tr<T>::MAGIC;
  const int t = lane & 3;
  uint32_t vw[WPL];
#pragma unroll
  for (int v = 0; v < WPL / 4; ++v) {
    const uint4 x = ld(vc + v * 32 + lane);
    vw[4 * v] = x.x; vw[4 * v + 1] = x.y; vw[4 * v + 2] = x.z; vw[4 * v + 3] = x.w;
  }
#pragma unroll
  for (int gc = 0; gc < D / GROUP; ++gc) {
    const uint4 pr0 = ld(vp + (gc * 2 + 0) * 4 + t);  // tokens 0..15:  {s,z} low octet, {s,z} high octet
    const uint4 pr1 = ld(vp + (gc * 2 + 1) * 4 + t);  // tokens 16..31
#pragma unroll
    for (int ii = 0; ii < GROUP / 16; ++ii) {
      const int i = gc * (GROUP / 16) + ii;
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        const uint4 pr = ks ? pr1 : pr0;
        uint32_t w;
        int sh;
        if (BITS == 4) { w = vw[i * 2 + ks]; sh = 0; } else { w = vw[i]; sh = ks * 8; }
        const uint32_t a0 = dequant2<T>(((w >> (sh + 0 * BITS)) & MASK) | MG, pr.x, pr.y);
        const uint32_t a1 = dequant2<T>(((w >> (sh + 1 * BITS)) & MASK) | MG, pr.x, pr.y);
        const uint32_t a2 = dequant2<T>(((w >> (sh + 2 * BITS)) & MASK) | MG, pr.z, pr.w);
        const uint32_t a3 = dequant2<T>(((w >> (sh + 3 * BITS)) & MASK) | MG, pr.z, pr.w);
        mma16816<T>(o[i], a0, a1, a2, a3, pa[ks][0], pa[ks][1]);
        mma16816<T>(o[i], a0, a1, a2, a3, pb[ks][0], pb[ks][1]);
      }
    }
  }
  (void)MT;
}

// Two probabilities -> a 16-bit pair plus the pair of rounding residuals.  The PV product is taken with
// both (P = P_main + P_res), so the 8 (11) significand bits of the operand type do not limit the output.
template <class T> __device__ __forceinline__ void split_pair(float lo, float hi, uint32_t& main, uint32_t& res);
template <> __device__ __forceinline__ void split_pair<__half>(float lo, float hi, uint32_t& main, uint32_t& res) {
  const __half2 m = __floats2half2_rn(lo, hi);
  main = as_u32(m);
  res = as_u32(__floats2half2_rn(lo - __low2float(m), hi - __high2float(m)));
}
template <> __device__ __forceinline__ void split_pair<__nv_bfloat16>(float lo, float hi, uint32_t& main, uint32_t& res) {
  const __nv_bfloat162 m = __floats2bfloat162_rn(lo, hi);
  main = as_u32(m);
  res = as_u32(__floats2bfloat162_rn(lo - __low2float(m), hi - __high2float(m)));
}

// Online softmax update for one tile; returns the probability fragments for the PV product.
template <class T, int MT>
__device__ __forceinline__ void softmax_tile(float (&s)[4][4], int ntok, float scale_log2, int lane, float& m_run,
                                             float& l_run, float& wsum, float (&o)[MT][4], uint32_t (&pa)[2][2],
                                             uint32_t (&pb)[2][2]) {
  const int t = lane & 3;
  float x[4][2];
  float tmax = -INFINITY;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int tok = 8 * j + 2 * t + e;
      x[j][e] = (tok < ntok) ? s[j][e] * scale_log2 : -INFINITY;
      tmax = fmaxf(tmax, x[j][e]);
    }
  }
  tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
  tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
  const float m_new = fmaxf(m_run, tmax);  // finite: the caller guarantees ntok >= 1
  const float alpha = exp2f(m_run - m_new);
  float rs = 0.f;
  float p[4][2];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      p[j][e] = exp2f(x[j][e] - m_new);
      rs += p[j][e];
    }
  }
  rs += __shfl_xor_sync(0xffffffffu, rs, 1);
  rs += __shfl_xor_sync(0xffffffffu, rs, 2);
  l_run = l_run * alpha + rs;
  wsum = wsum * alpha + rs;
  m_run = m_new;
  // the accumulators hold O^T: column pair (2t, 2t+1) = heads 2t and 2t+1, whose statistics live in
  // the lane quads 2t and 2t+1
  const float a_lo = __shfl_sync(0xffffffffu, alpha, (2 * t) * 4);
  const float a_hi = __shfl_sync(0xffffffffu, alpha, (2 * t + 1) * 4);
#pragma unroll
  for (int i = 0; i < MT; ++i) {
    o[i][0] *= a_lo; o[i][1] *= a_hi; o[i][2] *= a_lo; o[i][3] *= a_hi;
  }
  split_pair<T>(p[0][0], p[0][1], pa[0][0], pb[0][0]);
  split_pair<T>(p[1][0], p[1][1], pa[0][1], pb[0][1]);
  split_pair<T>(p[2][0], p[2][1], pa[1][0], pb[1][0]);
  split_pair<T>(p[3][0], p[3][1], pa[1][1], pb[1][1]);
}

template <class T, int D, int BITS, int GROUP, int TILES>
__global__ void __launch_bounds__(DECODE_WARPS * 32) decode_attn_kernel(const DecodeParams p) {
  using TT = DecodeTraits<T, D, BITS, GROUP, TILES>;
  constexpr int KS = TT::KS, MT = TT::MT;
  const int s = blockIdx.x, hk = blockIdx.y, ul = blockIdx.z;
  const int u = p.unit0 + ul;
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  auto ld = [](const uint4* ptr) { return ld_stream16(ptr); };

  // query fragments: row g of the A operand = head hk*G + g (rows >= G are zero)
  uint32_t qa[KS][2];
  {
    const T* qrow = reinterpret_cast<const T*>(p.q) + ((size_t)ul * p.Hq + (size_t)hk * p.G + g) * D;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      if (g < p.G) {
        qa[ks][0] = *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * t);
        qa[ks][1] = *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * t);
      } else {
        qa[ks][0] = 0u; qa[ks][1] = 0u;
      }
    }
  }

  float m_run = -INFINITY, l_run = 0.f;
  float o[MT][4];
#pragma unroll
  for (int i = 0; i < MT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }

  const int n_live = p.n_live[u];
  const int fill = p.open_fill[u];
  const int stride = p.S * DECODE_WARPS;
  for (int e = s * DECODE_WARPS + wid; e < n_live; e += stride) {
    const uint2 ent = p.entries[(size_t)u * p.EMAX + e];
    const uint32_t kind = ent.x >> ENTRY_KIND_SHIFT;
    const int page = (int)ent.y;
    const int valid = (kind == KIND_OPEN) ? fill : TT::W;
    float wsum = 0.f;
    if (kind != KIND_Q) {
      const char* base = p.fp_pool + ((size_t)u * p.PF + page) * p.fp_page_bytes + (size_t)hk * TT::FP_HEAD_BYTES;
#pragma unroll 1
      for (int tile = 0; tile < TILES; ++tile) {
        const int ntok = valid - 32 * tile;
        if (ntok <= 0) break;
        const uint4* kt = reinterpret_cast<const uint4*>(base + (size_t)tile * 2 * TT::FP_TILE_BYTES);
        const uint4* vt = kt + TT::FP_TILE_BYTES / 16;
        float sacc[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f; }
        qk_fp_tile<T, D>(sacc, qa, kt, lane, ld);
        uint32_t pa[2][2], pb[2][2];
        softmax_tile<T, MT>(sacc, ntok, p.scale_log2, lane, m_run, l_run, wsum, o, pa, pb);
        pv_fp_tile<T, D>(o, pa, pb, vt, lane, ld);
      }
    } else {
      const char* base = p.q_pool + ((size_t)u * p.PQ + page) * p.q_page_bytes + (size_t)hk * TT::Q_HEAD_BYTES;
#pragma unroll 1
      for (int tile = 0; tile < TILES; ++tile) {
        const char* tb = base + (size_t)tile * TT::Q_TILE_STRIDE;
        const uint4* kc = reinterpret_cast<const uint4*>(tb);
        const uint4* vc = reinterpret_cast<const uint4*>(tb + TT::KC_BYTES);
        const uint4* vp = reinterpret_cast<const uint4*>(tb + TT::KC_BYTES + TT::VC_BYTES);
        const uint4* kp = reinterpret_cast<const uint4*>(base + TT::KP_OFF + (size_t)((tile * 32) / GROUP) * TT::KP_BYTES);
        float sacc[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f; }
        qk_q_tile<T, D, BITS>(sacc, qa, kc, kp, lane, ld);
        uint32_t pa[2][2], pb[2][2];
        softmax_tile<T, MT>(sacc, 32, p.scale_log2, lane, m_run, l_run, wsum, o, pa, pb);
        pv_q_tile<T, D, BITS, GROUP>(o, pa, pb, vc, vp, lane, ld);
      }
    }
    if (t == 0 && g < p.G) {
      p.wrec[((size_t)u * p.Hq + (size_t)hk * p.G + g) * p.EMAX + e] = make_float2(wsum, m_run);
    }
  }

  // ---- merge the four warps, write the split's partial ------------------------------------------
  __shared__ float sm_m[DECODE_WARPS][8];
  __shared__ float sm_l[DECODE_WARPS][8];
  __shared__ float sm_o[DECODE_WARPS][8][D + 4];
  if (t == 0) { sm_m[wid][g] = m_run; sm_l[wid][g] = l_run; }
#pragma unroll
  for (int i = 0; i < MT; ++i) {
    sm_o[wid][2 * t][16 * i + g] = o[i][0];
    sm_o[wid][2 * t + 1][16 * i + g] = o[i][1];
    sm_o[wid][2 * t][16 * i + g + 8] = o[i][2];
    sm_o[wid][2 * t + 1][16 * i + g + 8] = o[i][3];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < p.G * D; idx += DECODE_WARPS * 32) {
    const int h = idx / D, ch = idx - h * D;
    float mx = sm_m[0][h];
#pragma unroll
    for (int w = 1; w < DECODE_WARPS; ++w) mx = fmaxf(mx, sm_m[w][h]);
    float acc = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < DECODE_WARPS; ++w) {
      const float mw = sm_m[w][h];
      const float sc = (mw == -INFINITY) ? 0.f : exp2f(mw - mx);
      acc += sm_o[w][h][ch] * sc;
      l += sm_l[w][h] * sc;
    }
    const size_t ph = ((size_t)u * p.Hq + (size_t)hk * p.G + h) * MAX_SPLITS + s;
    p.o_part[ph * D + ch] = acc;
    if (ch == 0) { p.ml[ph * 2] = mx; p.ml[ph * 2 + 1] = l; }
  }
}

template <class T, int D, int BITS, int GROUP, int TILES>
cudaError_t launch_decode_attn(const DecodeParams& p, int n_units, cudaStream_t stream) {
  dim3 grid(p.S, p.Hkv, n_units);
  decode_attn_kernel<T, D, BITS, GROUP, TILES><<<grid, DECODE_WARPS * 32, 0, stream>>>(p);
  return cudaGetLastError();
}

// explicit dispatch table entry points, one per (dtype, D) translation unit
typedef cudaError_t (*decode_launch_fn)(const DecodeParams&, int, cudaStream_t);
decode_launch_fn decode_dispatch_h64(int bits, int group, int tiles);
decode_launch_fn decode_dispatch_h128(int bits, int group, int tiles);
decode_launch_fn decode_dispatch_b64(int bits, int group, int tiles);
decode_launch_fn decode_dispatch_b128(int bits, int group, int tiles);

#define QEVICT_DECODE_DISPATCH(NAME, T, D)                                            \
  decode_launch_fn NAME(int bits, int group, int tiles) {                             \
    if (bits == 4 && group == 32 && tiles == 1) return launch_decode_attn<T, D, 4, 32, 1>; \
    if (bits == 2 && group == 32 && tiles == 1) return launch_decode_attn<T, D, 2, 32, 1>; \
    if (bits == 4 && group == 32 && tiles == 2) return launch_decode_attn<T, D, 4, 32, 2>; \
    if (bits == 2 && group == 32 && tiles == 2) return launch_decode_attn<T, D, 2, 32, 2>; \
    if (bits == 4 && group == 64 && tiles == 2) return launch_decode_attn<T, D, 4, 64, 2>; \
    if (bits == 2 && group == 64 && tiles == 2) return launch_decode_attn<T, D, 2, 64, 2>; \
    return nullptr;                                                                   \
  }

}  // namespace qevict
