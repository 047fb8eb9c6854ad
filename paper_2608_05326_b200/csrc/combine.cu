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

__device__ __forceinline__ float ex2a(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

template <class T>
__global__ void __launch_bounds__(COMBINE_THREADS) combine_kernel(const KernelArgs a, int S, int e_bound, T* __restrict__ out) {
  const Geometry& g = a.geo;
  // every CTA owns 4 * NE (= 16) consecutive work-list entries for the mass update and a slice of the
  // (head, 4-channel) tasks of the output merge; all its global loads are issued before anything waits
  const int ul = blockIdx.y, u = a.unit0 + ul, tid = threadIdx.x;
  const int lane = tid & 31, wid = tid >> 5;
  constexpr int NE = 4;  // work-list entries a warp keeps in registers at a time
  extern __shared__ __align__(16) unsigned char csm[];
  float* s_m = reinterpret_cast<float*>(csm);  // [Hq] global maximum
  float* s_invl = s_m + g.Hq;                  // [Hq] 1 / denominator
  float* s_w = s_invl + g.Hq;                  // [Hq][S] weight of a split in its head's output
  pdl_prologue();
  QE_TRACE_SCOPE(a.trace, 2);
  const float2* ml = reinterpret_cast<const float2*>(a.st.ml) + (size_t)u * g.Hq * MAX_SPLITS;
  const float2* wrec = a.st.wrec + (size_t)u * g.Hq * g.EMAX;
  const uint2* entries = a.st.entries + (size_t)u * g.EMAX;
  const float* op = a.st.o_part + (size_t)u * g.Hq * MAX_SPLITS * g.D;

  // ---- requests: first output task, this CTA's slice of the work list ------------------------------------
  const int D4 = g.D >> 2, n_task = g.Hq * D4, t_stride = gridDim.x * COMBINE_THREADS;
  const int t0 = blockIdx.x * COMBINE_THREADS + tid;
  float4 pre[8];
  {
    const int h = t0 / D4, c4 = t0 - h * D4;
    const float4* src = reinterpret_cast<const float4*>(op + (size_t)h * MAX_SPLITS * g.D) + c4;
#pragma unroll
    for (int k = 0; k < 8; ++k)
      pre[k] = (t0 < n_task && k < S) ? __ldg(src + (size_t)k * D4) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  // (the grid covers the host's upper bound of the list length, so nothing here waits for the length);
  // warp `wid` takes entries e0 + wid, e0 + wid + 4, ...; lane = head
  const int e0 = blockIdx.x * (4 * NE), e1 = min(min(e_bound, g.EMAX), e0 + 4 * NE);
  const int n = a.st.n_live[u];
  float2 rec[NE];
  uint32_t ewin[NE];
#pragma unroll
  for (int k = 0; k < NE; ++k) {
    const int e = e0 + wid + 4 * k;
    rec[k] = (e < e1 && lane < g.Hq) ? __ldg(wrec + (size_t)e * g.Hq + lane) : make_float2(0.f, 0.f);
    ewin[k] = (e < e1) ? __ldg(&entries[e].x) : 0u;
  }

  // ---- per-head maximum, denominator and split weights (one thread per head) ------------------------------
#pragma unroll 1
  for (int h = tid; h < g.Hq; h += COMBINE_THREADS) {
    const float2* p = ml + (size_t)h * MAX_SPLITS;
    float mx = -INFINITY, l = 0.f;
#pragma unroll 1
    for (int s0 = 0; s0 < S; s0 += 8) {
      float2 v[8];
      float cm = -INFINITY;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        v[k] = (s0 + k < S) ? __ldg(p + s0 + k) : make_float2(-INFINITY, 0.f);
        cm = fmaxf(cm, v[k].x);
      }
      const float nm = fmaxf(mx, cm);
      if (nm > -INFINITY) {  // an empty split has m = -inf, l = 0: contributes 0
        l *= ex2a(mx - nm);
#pragma unroll
        for (int k = 0; k < 8; ++k) l += v[k].y * ex2a(v[k].x - nm);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (s0 + k < S) s_w[h * S + s0 + k] = v[k].x;
      mx = nm;
    }
    const float invl = l > 0.f ? 1.f / l : 0.f;
#pragma unroll 1
    for (int sp = 0; sp < S; ++sp) {
      const float m = s_w[h * S + sp];
      s_w[h * S + sp] = m > -INFINITY ? ex2a(m - mx) * invl : 0.f;
    }
    s_m[h] = mx;
    s_invl[h] = invl;
  }
  // old scores of this warp's windows (needs only the entries), requested before the barrier; with Eq. 1 the
  // mass goes straight into the score, with the other ranking functions into the event accumulator
  float* score = g.rank_mode == QEVICT_RANK_CUMULATIVE ? a.st.importance : a.st.event_mass;
  float old[NE];
#pragma unroll
  for (int k = 0; k < NE; ++k) {
    const int e = e0 + wid + 4 * k;
    if (e < e1 && e < n && !QE_IN_RANGE((int)(ewin[k] & ENTRY_WINDOW_MASK) < g.NW, a.st.status, CHECK_BOUNDS_WINDOW)) ewin[k] = 0xFFFFFFFFu;
    old[k] = (e < e1 && e < n && lane == 0 && ewin[k] != 0xFFFFFFFFu) ? score[(size_t)u * g.NW + (ewin[k] & ENTRY_WINDOW_MASK)] : 0.f;
  }
  __syncthreads();

  // ---- attention output: out_h = sum_s w_{h,s} O_{h,s}, four channels per task ----------------------------
#pragma unroll 1
  for (int task = t0; task < n_task; task += t_stride) {
    const int h = task / D4, c4 = task - h * D4;
    const float4* src = reinterpret_cast<const float4*>(op + (size_t)h * MAX_SPLITS * g.D) + c4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
    for (int s0 = 0; s0 < S; s0 += 8) {
      float4 x[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (task == t0 && s0 == 0) x[k] = pre[k];
        else x[k] = (s0 + k < S) ? __ldg(src + (size_t)(s0 + k) * D4) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (s0 + k < S) {
          const float w = s_w[h * S + s0 + k];
          acc.x += x[k].x * w; acc.y += x[k].y * w; acc.z += x[k].z * w; acc.w += x[k].w * w;
        }
      }
    }
    __align__(8) T o4[4] = {Tr<T>::from_float(acc.x), Tr<T>::from_float(acc.y), Tr<T>::from_float(acc.z),
                            Tr<T>::from_float(acc.w)};
    *reinterpret_cast<uint2*>(out + ((size_t)ul * g.Hq + h) * g.D + 4 * c4) = *reinterpret_cast<const uint2*>(o4);
  }

  // ---- window mass: lane h holds head h's share; a fixed shuffle tree adds the heads (same order every
  // run) -------------------------------------------------------------------------------------------------
  auto head_sum = [&](float2 r, int e) -> float {
    float term = 0.f;
#pragma unroll 1
    for (int hb = 0; hb < g.Hq; hb += 32) {
      const int h = hb + lane;
      float2 rr = r;
      if (hb > 0) rr = (h < g.Hq) ? __ldg(wrec + (size_t)e * g.Hq + h) : make_float2(0.f, 0.f);
      if (h < g.Hq) term += rr.x * ex2a(rr.y - s_m[h]) * s_invl[h];
    }
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) term += __shfl_xor_sync(0xffffffffu, term, o2);
    return term;
  };
#pragma unroll
  for (int k = 0; k < NE; ++k) {
    const int e = e0 + wid + 4 * k;
    const bool live = e < e1 && e < n && ewin[k] != 0xFFFFFFFFu;  // (all ones: a window index the checking build refused)
    const float mass = live ? head_sum(rec[k], e) : 0.f;
    if (live && lane == 0) {
      score[(size_t)u * g.NW + (ewin[k] & ENTRY_WINDOW_MASK)] = old[k] + mass;
      a.st.mass_e[(size_t)u * g.EMAX + e] = mass;
    }
  }
}

}  // namespace

cudaError_t launch_combine(const KernelArgs& a, int n_splits, int e_bound, void* out, cudaStream_t s) {
  const int chunks = (e_bound + 15) / 16;  // 4 warps x 4 entries per CTA
  dim3 grid(chunks > a.geo.Hkv ? chunks : a.geo.Hkv, a.n_units);
  const size_t sm = (size_t)a.geo.Hq * 8 + (size_t)a.geo.Hq * n_splits * 4;
  if (a.geo.dtype == QEVICT_DTYPE_FP16)
    return launch_pdl(combine_kernel<__half>, grid, dim3(COMBINE_THREADS), sm, s, a, n_splits, e_bound, (__half*)out);
  return launch_pdl(combine_kernel<__nv_bfloat16>, grid, dim3(COMBINE_THREADS), sm, s, a, n_splits, e_bound, (__nv_bfloat16*)out);
}

}  // namespace qevict
