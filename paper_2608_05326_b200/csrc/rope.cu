// Rotation table of pre-RoPE keys [Migration-Stable Quantization: keys are kept in the pre-RoPE domain with their
// absolute positions; RoPE is reapplied after dequantization].  Built once per cache: for every block of 32
// positions, (cos, sin)(p * theta_i), theta_i = base^(-2 i / d), rounded to the execution datatype from a
// float64 evaluation, stored in the order the attention kernel's key fragments want them (see rope_fragments in
// decode_attn.cuh): vector ((ks' * 2 + mt) * 2 + half) * 32 + lane = {C r, S r, C r+1, S r+1}, r = 2 * half,
// where register r covers token row g + 8 (r & 1) of token block mt and channels 16 ks' + 8 (r >> 1) + 2t, +1.
#include "kernels.cuh"

namespace qevict {

namespace {

template <class T> __device__ __forceinline__ T from_double(double x);
template <> __device__ __forceinline__ __half from_double<__half>(double x) { return __double2half(x); }
template <> __device__ __forceinline__ __nv_bfloat16 from_double<__nv_bfloat16>(double x) { return __double2bfloat16(x); }

template <class T>
__device__ __forceinline__ uint32_t pack_pair(T lo, T hi) {
  typename Tr<T>::T2 v;
  v.x = lo; v.y = hi;
  return *reinterpret_cast<const uint32_t*>(&v);
}

// (cos, sin)(pos * base^(-2 i / d)) from a float64 evaluation, rounded once to T
template <class T>
__device__ __forceinline__ void rope_cos_sin(double pos, int i, int D, double base, T& c, T& s) {
  const double ang = pos * pow(base, -2.0 * (double)i / (double)D);
  c = from_double<T>(cos(ang));
  s = from_double<T>(sin(ang));
}

template <class T>
__global__ void rope_table_kernel(uint4* __restrict__ table, int n_blocks, int D, double base) {
  const int vecs = (D / 32) * 2 * 2 * 32;  // per block of 32 positions
  const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long)n_blocks * vecs) return;
  const int blk = (int)(idx / vecs), v = (int)(idx - (long)blk * vecs);
  const int lane = v & 31, half = (v >> 5) & 1, mt = (v >> 6) & 1, ksp = v >> 7;
  const int g = lane >> 2, t = lane & 3;
  uint32_t out[4];
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    const int r = 2 * half + rr;
    const double pos = (double)(blk * 32 + 16 * mt + g + 8 * (r & 1));
    T c[2], s[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) rope_cos_sin<T>(pos, 16 * ksp + 8 * (r >> 1) + 2 * t + e, D, base, c[e], s[e]);
    out[2 * rr] = pack_pair<T>(c[0], c[1]);
    out[2 * rr + 1] = pack_pair<T>(s[0], s[1]);
  }
  table[idx] = make_uint4(out[0], out[1], out[2], out[3]);
}

// Prompt keys [rows = batch * H_kv][ctx][d], pre-RoPE -> rotated for positions 0 .. ctx-1, in the same arithmetic
// as the attention kernel (every product and sum rounded to T on its own).  One thread per (row, position, pair).
template <class T>
__global__ void rope_rotate_prompt_kernel(const T* __restrict__ k, T* __restrict__ out, long n_pairs, int ctx, int D, double base) {
  using T2 = typename Tr<T>::T2;
  const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_pairs) return;
  const int h = D / 2, i = (int)(idx % h);
  const long tok = idx / h;  // row * ctx + position
  const int pos = (int)(tok % ctx);
  T c, s;
  rope_cos_sin<T>((double)pos, i, D, base, c, s);
  const T x = k[tok * D + i], y = k[tok * D + i + h];
  // the packed operations of the attention kernel, one lane of them
  T2 X, Y, C, S;
  X.x = x; X.y = x; Y.x = y; Y.y = y; C.x = c; C.y = c; S.x = s; S.y = s;
  const T2 xr = __hsub2_rn(__hmul2_rn(X, C), __hmul2_rn(Y, S));
  const T2 yr = __hadd2_rn(__hmul2_rn(Y, C), __hmul2_rn(X, S));
  out[tok * D + i] = xr.x;
  out[tok * D + i + h] = yr.x;
}

}  // namespace

cudaError_t launch_rope_rotate_prompt(const Geometry& g, const void* k, void* out, long rows, int ctx, cudaStream_t s) {
  const long n_pairs = rows * ctx * (g.D / 2);
  const unsigned grid = (unsigned)((n_pairs + 255) / 256);
  if (g.dtype == QEVICT_DTYPE_FP16)
    rope_rotate_prompt_kernel<__half><<<grid, 256, 0, s>>>((const __half*)k, (__half*)out, n_pairs, ctx, g.D, (double)g.rope_base);
  else
    rope_rotate_prompt_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)k, (__nv_bfloat16*)out, n_pairs, ctx, g.D,
                                                                  (double)g.rope_base);
  return cudaGetLastError();
}

cudaError_t launch_rope_table(const Geometry& g, const State& st, cudaStream_t s) {
  if (!(g.rope_base > 0.f)) return cudaSuccess;
  const int n_blocks = g.NW * g.tiles;
  const long total = (long)n_blocks * (g.D / 32) * 2 * 2 * 32;
  const unsigned grid = (unsigned)((total + 255) / 256);
  if (g.dtype == QEVICT_DTYPE_FP16) rope_table_kernel<__half><<<grid, 256, 0, s>>>(st.rope_table, n_blocks, g.D, (double)g.rope_base);
  else rope_table_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(st.rope_table, n_blocks, g.D, (double)g.rope_base);
  return cudaGetLastError();
}

}  // namespace qevict
