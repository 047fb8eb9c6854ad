// Prefill window scores on the GPU.
//
// "During prefill, prompt attention initialises the window scores" [Methodology]; the score has Eq. 1's form:
// the attention probability a window's tokens receive, summed over query heads and over the queries that
// observe it.  Here the observers are n_obs queries per head that stand after the prompt, so each attends
// to the whole prompt in full precision:
//     score[w] = sum over observers o, heads h of  sum_{i in w} softmax_i(q_{o,h} . k_i / sqrt(d)).
//
// Three kernels.  The first walks the prompt keys once: a warp takes one 32-token tile (lane = token, the key
// row lives in registers), and for every (observer, head) of its KV head reduces the tile's logits to a
// record {tile maximum, sum of 2^(logit - maximum)}.  The second merges the records per (observer, head)
// into the global maximum and denominator, the third adds up every window's share; all sums run in a fixed
// order.
#include "ctx.h"

namespace qevict {

namespace {

constexpr int SCORE_THREADS = 256;

template <class T>
__global__ void __launch_bounds__(SCORE_THREADS) score_tiles_kernel(const T* __restrict__ k, const T* __restrict__ q_obs,
                                                                    float2* __restrict__ rec, int n_obs, int ctx, int Hq,
                                                                    int Hkv, int D, float scale_log2) {
  extern __shared__ float sq[];  // [n_obs * G][D] queries of this KV head, as float
  const int hk = blockIdx.y, b = blockIdx.z, G = Hq / Hkv, nqh = n_obs * G, NQ = n_obs * Hq;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  for (int i = threadIdx.x; i < nqh * D; i += SCORE_THREADS) {
    const int qi = i / D, c = i - qi * D, o = qi / G, hl = qi - o * G;
    sq[i] = Tr<T>::to_float(q_obs[(((size_t)b * n_obs + o) * Hq + hk * G + hl) * D + c]);
  }
  __syncthreads();
  const int n_tiles = ctx / 32;
  const int tile = blockIdx.x * (SCORE_THREADS / 32) + wid;
  if (tile >= n_tiles) return;
  // this lane's key row
  float kr[128];
  const uint4* src = reinterpret_cast<const uint4*>(k + (((size_t)b * Hkv + hk) * ctx + (size_t)tile * 32 + lane) * D);
#pragma unroll
  for (int v = 0; v < 16; ++v) {
    if (v * 8 < D) {
      const uint4 x = __ldg(src + v);
      const T* e = reinterpret_cast<const T*>(&x);
#pragma unroll
      for (int j = 0; j < 8; ++j) kr[v * 8 + j] = Tr<T>::to_float(e[j]);
    }
  }
  for (int qi = 0; qi < nqh; ++qi) {
    const float* qv = sq + qi * D;
    float acc = 0.f;
#pragma unroll
    for (int c = 0; c < 128; ++c) {
      if (c < D) acc = fmaf(kr[c], qv[c], acc);
    }
    const float x = acc * scale_log2;
    float m = x;
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o2));
    float l = exp2f(x - m);
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o2);
    if (lane == 0) {
      const int o = qi / G, hl = qi - o * G;
      rec[((size_t)b * n_tiles + tile) * NQ + (size_t)o * Hq + hk * G + hl] = make_float2(m, l);
    }
  }
}

// Global maximum and 1 / denominator of every (observer, head): one warp per query, lanes stride over the
// tiles, fixed shuffle trees.
__global__ void __launch_bounds__(SCORE_THREADS) score_stats_kernel(const float2* __restrict__ rec, float2* __restrict__ stats,
                                                                    int NQ, int n_tiles) {
  const int b = blockIdx.y, lane = threadIdx.x & 31;
  const int q = blockIdx.x * (SCORE_THREADS / 32) + (threadIdx.x >> 5);
  if (q >= NQ) return;
  const float2* r = rec + (size_t)b * n_tiles * NQ + q;
  float mx = -INFINITY;
  for (int t = lane; t < n_tiles; t += 32) mx = fmaxf(mx, r[(size_t)t * NQ].x);
#pragma unroll
  for (int o2 = 16; o2 > 0; o2 >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o2));
  float l = 0.f;
  for (int t = lane; t < n_tiles; t += 32) {
    const float2 v = r[(size_t)t * NQ];
    l += v.y * exp2f(v.x - mx);
  }
#pragma unroll
  for (int o2 = 16; o2 > 0; o2 >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o2);
  if (lane == 0) stats[(size_t)b * NQ + q] = make_float2(mx, 1.f / l);
}

// Mass of every window: one warp per window, lanes stride over the (observer, head) pairs of each of its
// tiles, fixed shuffle tree.
__global__ void __launch_bounds__(SCORE_THREADS) score_merge_kernel(const float2* __restrict__ rec, const float2* __restrict__ stats,
                                                                    float* __restrict__ scores, int NQ, int n_tiles,
                                                                    int tiles_per_window) {
  const int b = blockIdx.y, lane = threadIdx.x & 31, n_windows = n_tiles / tiles_per_window;
  const int w = blockIdx.x * (SCORE_THREADS / 32) + (threadIdx.x >> 5);
  if (w >= n_windows) return;
  const float2* st = stats + (size_t)b * NQ;
  float mass = 0.f;
  for (int tt = 0; tt < tiles_per_window; ++tt) {
    const float2* rw = rec + ((size_t)b * n_tiles + (size_t)w * tiles_per_window + tt) * NQ;
    for (int q = lane; q < NQ; q += 32) {
      const float2 v = rw[q], sq = st[q];
      mass += v.y * exp2f(v.x - sq.x) * sq.y;
    }
  }
#pragma unroll
  for (int o2 = 16; o2 > 0; o2 >>= 1) mass += __shfl_xor_sync(0xffffffffu, mass, o2);
  if (lane == 0) scores[(size_t)b * n_windows + w] = mass;
}

}  // namespace

}  // namespace qevict

using namespace qevict;

extern "C" {

QEVICT_API qevict_status qevict_prefill_score_scratch_bytes(qevict_handle h, int32_t n_obs, int32_t ctx_tokens, uint64_t* bytes) {
  if (!h || !bytes || n_obs < 1 || ctx_tokens < 32 || ctx_tokens % 32) return QEVICT_ERR_INVALID_ARG;
  *bytes = (uint64_t)h->geo.batch * ((uint64_t)(ctx_tokens / 32) + 1) * n_obs * h->geo.Hq * sizeof(float2);
  return QEVICT_OK;
}

QEVICT_API qevict_status qevict_prefill_score(qevict_handle h, const void* k, const void* q_obs, int32_t n_obs, int32_t ctx_tokens,
                                              float* window_scores, void* scratch, uint64_t scratch_bytes, void* stream) {
  if (!h) return QEVICT_ERR_INVALID_ARG;
  const Geometry& g = h->geo;
  auto bad = [&](const char* msg) { h->last_error = msg; return QEVICT_ERR_INVALID_ARG; };
  if (!k || !q_obs || !window_scores || !scratch) return bad("k, q_obs, window_scores and scratch must not be NULL");
  if (n_obs < 1 || n_obs > 64) return bad("n_obs must be in 1..64");
  if (ctx_tokens < g.W || ctx_tokens % g.W || ctx_tokens > h->cfg.max_context) return bad("ctx_tokens must be a multiple of window within max_context");
  uint64_t need = 0;
  qevict_prefill_score_scratch_bytes(h, n_obs, ctx_tokens, &need);
  if (scratch_bytes < need) { h->last_error = "scratch too small: see qevict_prefill_score_scratch_bytes"; return QEVICT_ERR_NO_MEMORY; }
  const int nqh = n_obs * g.G, NQ = n_obs * g.Hq, n_tiles = ctx_tokens / 32;
  const size_t sm_a = (size_t)nqh * g.D * sizeof(float);
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = cudaSetDevice(h->cfg.device);
  float2* rec = static_cast<float2*>(scratch);
  dim3 grid((n_tiles + SCORE_THREADS / 32 - 1) / (SCORE_THREADS / 32), g.Hkv, g.batch);
  if (e == cudaSuccess && g.dtype == QEVICT_DTYPE_FP16) {
    if (sm_a > 48 * 1024) e = cudaFuncSetAttribute(score_tiles_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_a);
    if (e == cudaSuccess)
      score_tiles_kernel<__half><<<grid, SCORE_THREADS, sm_a, s>>>((const __half*)k, (const __half*)q_obs, rec, n_obs, ctx_tokens,
                                                                   g.Hq, g.Hkv, g.D, g.scale_log2);
  } else if (e == cudaSuccess) {
    if (sm_a > 48 * 1024) e = cudaFuncSetAttribute(score_tiles_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_a);
    if (e == cudaSuccess)
      score_tiles_kernel<__nv_bfloat16><<<grid, SCORE_THREADS, sm_a, s>>>((const __nv_bfloat16*)k, (const __nv_bfloat16*)q_obs, rec,
                                                                          n_obs, ctx_tokens, g.Hq, g.Hkv, g.D, g.scale_log2);
  }
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e == cudaSuccess) {
    float2* stats = rec + (size_t)g.batch * n_tiles * NQ;  // after the records
    const int wpb = SCORE_THREADS / 32, n_windows = ctx_tokens / g.W;
    score_stats_kernel<<<dim3((NQ + wpb - 1) / wpb, g.batch), SCORE_THREADS, 0, s>>>(rec, stats, NQ, n_tiles);
    score_merge_kernel<<<dim3((n_windows + wpb - 1) / wpb, g.batch), SCORE_THREADS, 0, s>>>(rec, stats, window_scores, NQ, n_tiles,
                                                                                       g.W / 32);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) { h->last_error = std::string("prefill_score: ") + cudaGetErrorString(e); return QEVICT_ERR_CUDA; }
  h->launches += 3;
  return QEVICT_OK;
}

}  // extern "C"
