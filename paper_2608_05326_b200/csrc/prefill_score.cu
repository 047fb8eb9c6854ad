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

// ---- the same tile records on the 5th-generation tensor cores ---------------------------------------------
// logits[128 tokens][NP queries] = K[128][D] . Q^T[D][NP] is a dense contraction: one tcgen05.mma chain per CTA
// (M = 128, N = NP, D / 16 steps of K = 16), operands in shared memory in the canonical K-major layout without
// swizzle -- 8-row x 16-byte core matrices, 128 bytes each, SBO between 8-row groups, LBO between the two
// 16-byte halves of a K = 16 step -- written with plain stores, accumulator in tensor memory (128 lanes x NP
// fp32 columns), read back with tcgen05.ld so that lane = token, exactly as the shuffle reductions want it.
// Every wait is bounded; a wait that runs out records CHECK_COPY_TIMEOUT and the CTA frees its tensor memory
// and leaves.
__device__ __forceinline__ uint32_t sm_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  // start address, leading and stride byte offsets in 16-byte units; version 1; no swizzle
  return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

template <class T>
__global__ void __launch_bounds__(128) score_tiles_tc_kernel(const T* __restrict__ k, const T* __restrict__ q_obs,
                                                             float2* __restrict__ rec, int32_t* __restrict__ status, int n_obs,
                                                             int ctx, int Hq, int Hkv, int D, int NP, float scale_log2) {
  extern __shared__ __align__(128) unsigned char tsm[];
  unsigned char* sA = tsm;                        // [D/8] column blocks of 16 core matrices (the 128-token block)
  constexpr uint32_t LBO_A = 16 * 128 + 16;       // bytes between the column blocks of the key operand
  unsigned char* sB = tsm + (D / 8) * LBO_A;      // [D/8][NP/8] core matrices of the queries
  uint64_t* mbar = reinterpret_cast<uint64_t*>(sB + (size_t)NP * D * 2);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(mbar + 1);
  const int hk = blockIdx.y, b = blockIdx.z, G = Hq / Hkv, nqh = n_obs * G, NQ = n_obs * Hq;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int tok0 = blockIdx.x * 128, n_tiles = ctx / 32;

  if (wid == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sm_u32(tmem_slot)), "r"((uint32_t)NP) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(sm_u32(mbar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // keys: consecutive threads take consecutive 16-byte pieces of the rows (coalesced); piece c8 of row r goes
  // to core matrix (c8, r / 8), row r % 8.  The column blocks are LBO_A apart: one extra 16 bytes per block
  // spreads a warp's stores over all banks.
  {
    const int ppr = D / 8;  // pieces per row
    const T* kb = k + (((size_t)b * Hkv + hk) * ctx + tok0) * D;
    for (int idx = tid; idx < 128 * ppr; idx += 128) {
      const int r = idx / ppr, c8 = idx - r * ppr;
      const uint4 v = tok0 + r < ctx ? __ldg(reinterpret_cast<const uint4*>(kb) + idx) : make_uint4(0u, 0u, 0u, 0u);
      *reinterpret_cast<uint4*>(sA + ((size_t)c8 * LBO_A + (size_t)(r >> 3) * 128 + (r & 7) * 16)) = v;
    }
  }
  // queries (rows past the last one are zero)
  for (int i = tid; i < NP * (D / 8); i += 128) {
    const int qi = i / (D / 8), c8 = i - qi * (D / 8);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (qi < nqh) {
      const int o = qi / G, hl = qi - o * G;
      v = __ldg(reinterpret_cast<const uint4*>(q_obs + (((size_t)b * n_obs + o) * Hq + hk * G + hl) * D) + c8);
    }
    *reinterpret_cast<uint4*>(sB + ((size_t)(c8 * (NP / 8) + (qi >> 3)) * 128 + (qi & 7) * 16)) = v;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // plain stores -> operands of the tensor core
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;

  if (tid == 0) {
    // instruction descriptor: fp32 accumulator, 16-bit inputs of type T, both operands K-major, N = NP, M = 128
    const uint32_t fmt = Tr<T>::MAGIC == 0x64006400u ? 0u : 1u;  // 0 = fp16, 1 = bf16
    const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(NP >> 3) << 17) | ((128u >> 4) << 24);
    const uint32_t a0 = sm_u32(sA), b0 = sm_u32(sB);
    for (int ks = 0; ks < D / 16; ++ks) {
      const uint64_t da = umma_desc(a0 + (uint32_t)(2 * ks) * LBO_A, LBO_A, 128u);
      const uint64_t db = umma_desc(b0 + (uint32_t)(2 * ks * (NP / 8)) * 128u, (uint32_t)(NP / 8) * 128u, 128u);
      const uint32_t acc = ks > 0 ? 1u : 0u;
      asm volatile(
          "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
          "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}\n" ::"r"(tmem),
          "l"(da), "l"(db), "r"(idesc), "r"(acc), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
          : "memory");
    }
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(sm_u32(mbar)) : "memory");
  }
  // bounded wait for the products
  bool ok = false;
  for (uint32_t it = 0; it < (1u << 18) && !ok; ++it) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(done) : "r"(sm_u32(mbar)), "r"(0u) : "memory");
    ok = done != 0;
  }
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (!ok && tid == 0) record_check(status, CHECK_COPY_TIMEOUT);
  const int tile = blockIdx.x * 4 + wid;
  if (ok && tile < n_tiles) {
    for (int c0 = 0; c0 < NP && c0 < nqh; c0 += 32) {
      uint32_t v[32];
      const uint32_t taddr = tmem + ((uint32_t)(wid * 32) << 16) + (uint32_t)c0;
      asm volatile(
          "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, "
          "%19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
          : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
            "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]),
            "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
            "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
          : "r"(taddr)
          : "memory");
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      // Lane = token, v[j] = logit of query c0 + j.  Both reductions run over the lanes for all 32 queries at
      // once: a butterfly in which every step halves the values a lane still carries (31 shuffles instead of
      // 160) and leaves lane L with the result of query c0 + L.
      float x[32], r[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) { x[j] = __uint_as_float(v[j]) * scale_log2; r[j] = x[j]; }
#pragma unroll
      for (int st = 16; st >= 1; st >>= 1) {
        const bool upper = (lane & st) != 0;
#pragma unroll
        for (int j = 0; j < st; ++j) {
          const float keep = upper ? r[j + st] : r[j], send = upper ? r[j] : r[j + st];
          r[j] = fmaxf(keep, __shfl_xor_sync(0xffffffffu, send, st));
        }
      }
      const float m_mine = r[0];  // maximum of query c0 + lane over the tile
#pragma unroll
      for (int j = 0; j < 32; ++j) r[j] = exp2f(x[j] - __shfl_sync(0xffffffffu, m_mine, j));
#pragma unroll
      for (int st = 16; st >= 1; st >>= 1) {
        const bool upper = (lane & st) != 0;
#pragma unroll
        for (int j = 0; j < st; ++j) {
          const float keep = upper ? r[j + st] : r[j], send = upper ? r[j] : r[j + st];
          r[j] = keep + __shfl_xor_sync(0xffffffffu, send, st);
        }
      }
      const int qi = c0 + lane;
      if (qi < nqh) {
        const int o = qi / G, hl = qi - o * G;
        rec[((size_t)b * n_tiles + tile) * NQ + (size_t)o * Hq + hk * G + hl] = make_float2(m_mine, r[0]);
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (wid == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)NP) : "memory");
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
  // pre-RoPE keys: room for a rotated copy of the prompt keys behind the records
  if (h->geo.rope_base > 0.f) *bytes = ((*bytes + 255) & ~(uint64_t)255) + (uint64_t)h->geo.batch * h->geo.Hkv * ctx_tokens * h->geo.D * 2;
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
  DeviceGuard guard(h->cfg.device);
  cudaError_t e = guard.err;
  float2* rec = static_cast<float2*>(scratch);
  if (g.rope_base > 0.f) {
    // the keys are pre-RoPE: the scores are taken over a rotated copy (prompt positions 0 .. ctx_tokens - 1)
    const uint64_t rec_bytes = ((uint64_t)g.batch * ((uint64_t)n_tiles + 1) * n_obs * g.Hq * sizeof(float2) + 255) & ~(uint64_t)255;
    void* k_rot = static_cast<char*>(scratch) + rec_bytes;
    if (e == cudaSuccess) e = launch_rope_rotate_prompt(g, k, k_rot, (long)g.batch * g.Hkv, ctx_tokens, s);
    k = k_rot;
    h->launches += 1;
  }
  if (nqh <= 128 && ctx_tokens % 128 == 0) {
    // tensor-core path: NP = queries padded to a power of two (tensor-memory columns)
    const int NP = nqh <= 32 ? 32 : (nqh <= 64 ? 64 : 128);
    const size_t sm_t = (size_t)(g.D / 8) * (16 * 128 + 16) + (size_t)NP * g.D * 2 + 16;
    dim3 tgrid(ctx_tokens / 128, g.Hkv, g.batch);
    if (e == cudaSuccess && g.dtype == QEVICT_DTYPE_FP16) {
      e = cudaFuncSetAttribute(score_tiles_tc_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_t);
      if (e == cudaSuccess)
        score_tiles_tc_kernel<__half><<<tgrid, 128, sm_t, s>>>((const __half*)k, (const __half*)q_obs, rec, h->st.status, n_obs,
                                                                ctx_tokens, g.Hq, g.Hkv, g.D, NP, g.scale_log2);
    } else if (e == cudaSuccess) {
      e = cudaFuncSetAttribute(score_tiles_tc_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_t);
      if (e == cudaSuccess)
        score_tiles_tc_kernel<__nv_bfloat16><<<tgrid, 128, sm_t, s>>>((const __nv_bfloat16*)k, (const __nv_bfloat16*)q_obs, rec,
                                                                       h->st.status, n_obs, ctx_tokens, g.Hq, g.Hkv, g.D, NP,
                                                                       g.scale_log2);
    }
  } else {
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
