// Split-combine kernel: merges the partial (m, l, O) of the splits into the attention output, and turns
// the per-(head, window) softmax numerators into the window mass that Eq. 1 adds to each window's score.
//
// For head h with global maximum M_h and denominator L_h (log2 domain),
//     out_h       = sum_s O_{h,s} 2^{m_{h,s} - M_h} / L_h
//     mass_h(w)   = wsum_h(w) 2^{mref_h(w) - M_h} / L_h
//     score[w]   += sum_{h = 0 .. H_q-1} mass_h(w)          (raw sum over heads, fixed order)
// One warp owns one window: lane h holds head h's share and a fixed shuffle tree adds them, so the score
// update is the same bits every run (no floating-point atomics).
#include "kernels.cuh"

namespace qevict {

namespace {

constexpr int COMBINE_THREADS = 128;
constexpr int MAX_HQ = 128;

template <class T>
__global__ void __launch_bounds__(COMBINE_THREADS) combine_kernel(const KernelArgs a, int S, int e_bound, T* __restrict__ out) {
  const Geometry& g = a.geo;
  // blockIdx.x = chunk * Hkv + KV head: chunk 0 of every KV head also merges the attention output;
  // every CTA owns 4 * NE consecutive work-list entries for the mass update
  const int hk = blockIdx.x % a.geo.Hkv, ul = blockIdx.y, u = a.unit0 + ul, tid = threadIdx.x;
  const int lane = tid & 31, wid = tid >> 5;
  pdl_prologue();
  constexpr int NE = 8;  // work-list entries a warp keeps in registers at a time
  __shared__ float s_m[MAX_HQ], s_invl[MAX_HQ];
  const float* ml = a.st.ml + (size_t)u * g.Hq * MAX_SPLITS * 2;
  const float2* wrec = a.st.wrec + (size_t)u * g.Hq * g.EMAX;
  const uint2* entries = a.st.entries + (size_t)u * g.EMAX;

  // This CTA's slice of the work list (the grid covers the host's upper bound of the list length, so
  // nothing here waits for the length); warp `wid` takes entries e0 + wid, e0 + wid + 4, ...; lane = head.
  const int e0 = blockIdx.x * (4 * NE), e1 = min(min(e_bound, g.EMAX), e0 + 4 * NE);
  const int n = a.st.n_live[u];
  float2 rec[NE];
  uint32_t ewin[NE];
#pragma unroll
  for (int k = 0; k < NE; ++k) {
    const int e = e0 + wid + 4 * k;
    rec[k] = (e < e1 && lane < g.Hq) ? __ldg(wrec + (size_t)lane * g.EMAX + e) : make_float2(0.f, 0.f);
    ewin[k] = (e < e1) ? __ldg(&entries[e].x) : 0u;
  }

  // per-head maximum and denominator over the splits (the (m, l) pairs of a head are contiguous)
  for (int h = tid; h < g.Hq; h += COMBINE_THREADS) {
    const float2* mlh = reinterpret_cast<const float2*>(ml) + (size_t)h * MAX_SPLITS;
    float mx = -INFINITY;
    for (int s0 = 0; s0 < S; s0 += 8) {
      float2 v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = (s0 + k < S) ? __ldg(mlh + s0 + k) : make_float2(-INFINITY, 0.f);
#pragma unroll
      for (int k = 0; k < 8; ++k) mx = fmaxf(mx, v[k].x);
    }
    float l = 0.f;
    for (int s0 = 0; s0 < S; s0 += 8) {
      float2 v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = (s0 + k < S) ? __ldg(mlh + s0 + k) : make_float2(-INFINITY, 0.f);
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (v[k].x != -INFINITY) l += v[k].y * exp2f(v[k].x - mx);
      }
    }
    s_m[h] = mx;
    s_invl[h] = l > 0.f ? 1.f / l : 0.f;
  }
  __syncthreads();

  // attention output of the heads of this KV head
  const float* op = a.st.o_part + (size_t)u * g.Hq * MAX_SPLITS * g.D;
  for (int idx = tid; idx < g.G * g.D && blockIdx.x < g.Hkv; idx += COMBINE_THREADS) {
    const int hl = idx / g.D, ch = idx - hl * g.D, h = hk * g.G + hl;
    const float2* mlh = reinterpret_cast<const float2*>(ml) + (size_t)h * MAX_SPLITS;
    const float mx = s_m[h];
    float acc = 0.f;
    for (int s0 = 0; s0 < S; s0 += 8) {
      float2 v[8];
      float x[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        v[k] = (s0 + k < S) ? __ldg(mlh + s0 + k) : make_float2(-INFINITY, 0.f);
        x[k] = (s0 + k < S) ? __ldg(op + ((size_t)h * MAX_SPLITS + s0 + k) * g.D + ch) : 0.f;
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (v[k].x != -INFINITY) acc += x[k] * exp2f(v[k].x - mx);
      }
    }
    out[((size_t)ul * g.Hq + h) * g.D + ch] = Tr<T>::from_float(acc * s_invl[h]);
  }

  // window mass: lane h holds head h's share; a fixed shuffle tree adds the heads (same order every run)
  auto head_sum = [&](float2 r, int e) -> float {
    float term = 0.f;
    for (int hb = 0; hb < g.Hq; hb += 32) {
      const int h = hb + lane;
      float2 rr = r;
      if (hb > 0) rr = (h < g.Hq) ? __ldg(wrec + (size_t)h * g.EMAX + e) : make_float2(0.f, 0.f);
      if (h < g.Hq) term += rr.x * exp2f(rr.y - s_m[h]) * s_invl[h];
    }
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) term += __shfl_xor_sync(0xffffffffu, term, o2);
    return term;
  };
  float mass[NE], old[NE];
#pragma unroll
  for (int k = 0; k < NE; ++k) {
    const int e = e0 + wid + 4 * k;
    const bool live = e < e1 && e < n;
    old[k] = (live && lane == 0) ? a.st.importance[(size_t)u * g.NW + (ewin[k] & ENTRY_WINDOW_MASK)] : 0.f;
    mass[k] = live ? head_sum(rec[k], e) : 0.f;
  }
#pragma unroll
  for (int k = 0; k < NE; ++k) {
    const int e = e0 + wid + 4 * k;
    if (e < e1 && e < n && lane == 0) {
      a.st.importance[(size_t)u * g.NW + (ewin[k] & ENTRY_WINDOW_MASK)] = old[k] + mass[k];
      a.st.mass_e[(size_t)u * g.EMAX + e] = mass[k];
    }
  }
}

}  // namespace

cudaError_t launch_combine(const KernelArgs& a, int n_splits, int e_bound, void* out, cudaStream_t s) {
  const int chunks = (e_bound + 31) / 32;  // 4 warps x 8 entries per CTA
  dim3 grid(chunks > a.geo.Hkv ? chunks : a.geo.Hkv, a.n_units);
  if (a.geo.dtype == QEVICT_DTYPE_FP16)
    return launch_pdl(combine_kernel<__half>, grid, dim3(COMBINE_THREADS), 0, s, a, n_splits, e_bound, (__half*)out);
  return launch_pdl(combine_kernel<__nv_bfloat16>, grid, dim3(COMBINE_THREADS), 0, s, a, n_splits, e_bound, (__nv_bfloat16*)out);
}

}  // namespace qevict
