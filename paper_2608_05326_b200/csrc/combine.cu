// Split-combine kernel: merges the partial (m, l, O) of the splits into the attention output, and turns
// the per-(head, window) softmax numerators into the window mass that Eq. 1 adds to each window's score.
//
// For head h with global maximum M_h and denominator L_h (log2 domain),
//     out_h       = sum_s O_{h,s} 2^{m_{h,s} - M_h} / L_h
//     mass_h(w)   = wsum_h(w) 2^{mref_h(w) - M_h} / L_h
//     score[w]   += sum_{h = 0 .. H_q-1} mass_h(w)          (raw sum over heads, fixed order)
// One thread owns one window and walks the heads in ascending order, so the score update is
// deterministic (no floating-point atomics).
#include "kernels.cuh"

namespace qevict {

namespace {

constexpr int COMBINE_THREADS = 128;
constexpr int MAX_HQ = 128;

template <class T>
__global__ void __launch_bounds__(COMBINE_THREADS) combine_kernel(const KernelArgs a, int S, T* __restrict__ out) {
  const Geometry& g = a.geo;
  const int hk = blockIdx.x, ul = blockIdx.y, u = a.unit0 + ul, tid = threadIdx.x;
  __shared__ float s_m[MAX_HQ], s_invl[MAX_HQ];
  const float* ml = a.st.ml + (size_t)u * g.Hq * MAX_SPLITS * 2;
  for (int h = tid; h < g.Hq; h += COMBINE_THREADS) {
    float mx = -INFINITY;
    for (int s = 0; s < S; ++s) mx = fmaxf(mx, ml[((size_t)h * MAX_SPLITS + s) * 2]);
    float l = 0.f;
    for (int s = 0; s < S; ++s) {
      const float ms = ml[((size_t)h * MAX_SPLITS + s) * 2];
      if (ms != -INFINITY) l += ml[((size_t)h * MAX_SPLITS + s) * 2 + 1] * exp2f(ms - mx);
    }
    s_m[h] = mx;
    s_invl[h] = l > 0.f ? 1.f / l : 0.f;
  }
  __syncthreads();

  // attention output of the heads of this KV head
  const float* op = a.st.o_part + (size_t)u * g.Hq * MAX_SPLITS * g.D;
  for (int idx = tid; idx < g.G * g.D; idx += COMBINE_THREADS) {
    const int hl = idx / g.D, ch = idx - hl * g.D, h = hk * g.G + hl;
    const float mx = s_m[h];
    float acc = 0.f;
    for (int s = 0; s < S; ++s) {
      const float ms = ml[((size_t)h * MAX_SPLITS + s) * 2];
      if (ms != -INFINITY) acc += op[((size_t)h * MAX_SPLITS + s) * g.D + ch] * exp2f(ms - mx);
    }
    out[((size_t)ul * g.Hq + h) * g.D + ch] = Tr<T>::from_float(acc * s_invl[h]);
  }

  // window mass: this CTA owns a contiguous slice of the unit's work list
  const int n = a.st.n_live[u];
  const int per = (n + g.Hkv - 1) / g.Hkv;
  const int e0 = hk * per, e1 = min(n, e0 + per);
  const float2* wrec = a.st.wrec + (size_t)u * g.Hq * g.EMAX;
  for (int e = e0 + tid; e < e1; e += COMBINE_THREADS) {
    float acc = 0.f;
    // heads in ascending order (fixed summation order); records are fetched eight at a time so that the
    // loads overlap
    for (int h0 = 0; h0 < g.Hq; h0 += 8) {
      float2 r[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        r[k] = (h0 + k < g.Hq) ? wrec[(size_t)(h0 + k) * g.EMAX + e] : make_float2(0.f, 0.f);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (h0 + k < g.Hq) acc += r[k].x * exp2f(r[k].y - s_m[h0 + k]) * s_invl[h0 + k];
      }
    }
    const uint32_t w = a.st.entries[(size_t)u * g.EMAX + e].x & ENTRY_WINDOW_MASK;
    a.st.importance[(size_t)u * g.NW + w] += acc;
    a.st.mass_e[(size_t)u * g.EMAX + e] = acc;
  }
}

}  // namespace

cudaError_t launch_combine(const KernelArgs& a, int n_splits, void* out, cudaStream_t s) {
  dim3 grid(a.geo.Hkv, a.n_units);
  if (a.geo.dtype == QEVICT_DTYPE_FP16)
    combine_kernel<__half><<<grid, COMBINE_THREADS, 0, s>>>(a, n_splits, (__half*)out);
  else
    combine_kernel<__nv_bfloat16><<<grid, COMBINE_THREADS, 0, s>>>(a, n_splits, (__nv_bfloat16*)out);
  return cudaGetLastError();
}

}  // namespace qevict
