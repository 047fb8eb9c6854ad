// Shared declarations of the qevict CUDA library: geometry, device state, small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/qevict.h"

namespace qevict {

// entry kinds of the decode work list
enum : uint32_t { KIND_FP = 0u, KIND_Q = 1u, KIND_OPEN = 2u };
static constexpr int ENTRY_KIND_SHIFT = 28;
static constexpr uint32_t ENTRY_WINDOW_MASK = (1u << ENTRY_KIND_SHIFT) - 1u;

// device status word values (first failure wins)
enum : int {
  CHECK_OK = 0,
  CHECK_FP_POOL_EXHAUSTED = 1,
  CHECK_Q_POOL_EXHAUSTED = 2,
  CHECK_ENTRY_OVERFLOW = 3,
  CHECK_WINDOW_OVERFLOW = 4,
  CHECK_COPY_TIMEOUT = 5,
  // checking build only (-DQEVICT_DEBUG_BOUNDS): an index read from a table was out of range; the access was skipped
  CHECK_BOUNDS_ENTRY = 6,    // work-list entry (kind, window or page)
  CHECK_BOUNDS_PAGE = 7,     // page id in a window table or a list
  CHECK_BOUNDS_WINDOW = 8,   // window index
  CHECK_BOUNDS_RECORD = 9,   // migration record
};

static constexpr int TILE_TOKENS = 32;    // tokens per attention tile
static constexpr int DECODE_WARPS = 4;    // warps per decode CTA
static constexpr int MAX_SPLITS = 64;

// Geometry derived from the configuration (host and device).
struct Geometry {
  int batch, n_layers, n_units;
  int Hq, Hkv, G, D, dtype, W, bits, group, Kf, Kq;
  int NW;        // max windows per unit
  int PF, PQ;    // pages per unit in the full-precision / quantized pool
  int EMAX;      // max entries of a unit's work list
  int aged_cap;  // filled windows that may wait for a routing event
  int n_sink, n_recent;  // protected windows: sink prefix, recent region (besides the open window)
  int rank_mode;     // QEVICT_RANK_*
  int one_way;       // 1: a Quantized window never returns to the Full tier
  float rope_base;   // > 0: stored keys are pre-RoPE, rotated by the attention kernel
  float rank_param;  // lambda or p
  int Kfp;       // K_f + n_sink + n_recent: windows that may need a full-precision page in one event
  int tiles;     // W / 32
  // full-precision page: [H_kv][tile]{K tile, V tile}, each tile 32 x D elements, fragment-major
  uint32_t fp_tile_bytes, fp_head_bytes, fp_page_bytes;
  // quantized page: [H_kv]{ [tile]{K codes, V codes, V params}, K params x (W/group) }
  uint32_t q_kc_bytes, q_vc_bytes, q_vp_bytes, q_tile_stride, q_kp_bytes, q_kp_off, q_head_bytes, q_page_bytes;
  float scale_log2;  // softmax scale * log2(e)
};

// Device pointers of one cache (all arrays are [n_units][...]).
struct State {
  uint8_t* tier;        // [NW]
  uint8_t* ledger;      // [NW]
  int32_t* fp_page;     // [NW]
  int32_t* q_page;      // [NW]
  float* importance;    // [NW]
  float* event_mass;    // [NW] mass since the last routing event (ranking functions other than Eq. 1)
  float* knorm_acc;     // [1] sum of the key norms of the open window's tokens (key-norm ranking)
  int32_t* fp_owner;    // [PF] window holding the page, -1 free
  int32_t* q_owner;     // [PQ]
  int32_t* n_windows;   // [1]
  int32_t* open_window; // [1] -1 if none
  int32_t* open_fill;   // [1]
  int32_t* n_live;      // [1] entries in the work list
  uint2* entries;       // [EMAX] {window | kind << 28, page}
  int4* copy_list;      // [Kf] {window, dst fp page, 0, 0} (prefill only)
  int32_t* n_copy;
  int4* mig_queue;      // [PF + Kq + Kf] records of two int4 per unit; the units of one call share the run
                        // that starts at its first unit (record format: see the migration kernel)
  int32_t* mig_count;   // [n_layers][2] (not per unit) entries queued by the routing event; events alternate
                        // between the two counters, and the migration kernel clears the one the next event uses
  unsigned long long* counters;  // [4] promotions, quantizations, reactivations, deletions
  char* fp_pool;        // [PF] pages
  char* q_pool;         // [PQ] pages
  float* o_part;        // [Hq][MAX_SPLITS][D]
  float* ml;            // [Hq][MAX_SPLITS][2]
  float2* wrec;         // [EMAX][Hq] {window exp-sum, reference max (log2 domain)}
  float* mass_e;        // [EMAX] last step's mass per entry
  int32_t* status;      // [1] (shared by all units)
  uint4* rope_table;    // [NW * tiles] blocks of cos / sin pairs in the key tile's fragment order (shared by all units)
#ifdef QEVICT_TRACE
  unsigned long long* trace;  // [TRACE_CALLS + 1] call blocks (shared by all units)
#endif
};

template <class T> struct Tr;
template <> struct Tr<__half> {
  using T2 = __half2;
  static constexpr uint32_t MAGIC = 0x64006400u;  // 1024.0 in both halves: 1024 + code is exact
  static constexpr int MANT = 10, EXP_BIAS = 15;   // significand bits, exponent bias
  static __device__ __forceinline__ __half from_float(float x) { return __float2half_rn(x); }
  static __device__ __forceinline__ float to_float(__half x) { return __half2float(x); }
};
template <> struct Tr<__nv_bfloat16> {
  using T2 = __nv_bfloat162;
  static constexpr uint32_t MAGIC = 0x43004300u;  // 128.0 in both halves: 128 + code is exact
  static constexpr int MANT = 7, EXP_BIAS = 127;   // significand bits, exponent bias
  static __device__ __forceinline__ __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
  static __device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
};

template <class T2> __device__ __forceinline__ T2 as_t2(uint32_t x) {
  T2 r;
  *reinterpret_cast<uint32_t*>(&r) = x;
  return r;
}
template <class T2> __device__ __forceinline__ uint32_t as_u32(T2 x) { return *reinterpret_cast<uint32_t*>(&x); }

// (a & b) | c in one LOP3: pulls two codes out of a packed word and plants them in the significands of MAGIC.
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;\n" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// Dequantize two codes held in the low bits of each 16-bit half of `x` (already OR-ed with MAGIC):
// value = RNE_T(code * s + z), one correctly rounded fused multiply-add in the execution datatype.
template <class T> __device__ __forceinline__ uint32_t dequant2(uint32_t x, uint32_t s2, uint32_t z2) {
  using T2 = typename Tr<T>::T2;
  T2 c = __hsub2(as_t2<T2>(x), as_t2<T2>(Tr<T>::MAGIC));  // exact
  return as_u32(__hfma2(c, as_t2<T2>(s2), as_t2<T2>(z2)));
}

// Two codes of BITS bits at bit position `pos` of each 16-bit half of `w` -> two dequantized values.  A code that
// lies wholly inside the significand field of T needs no shift to become a number: planted at significand bit p
// under the exponent of 2^(MANT - p), the half reads 2^(MANT - p) + code, and subtracting that power of two
// leaves the code, exactly.  So only every CAP-th bit position costs a shift (CAP = the multiple of BITS that
// fits the significand: 6 of 7 bits for 2-bit codes in bf16), and the shifted word serves CAP / BITS positions.
// `pos` must be a compile-time constant after unrolling.
template <class T, int BITS>
__device__ __forceinline__ uint32_t dequant_at(uint32_t w, int pos, uint32_t s2, uint32_t z2) {
  using T2 = typename Tr<T>::T2;
  constexpr int MANT = Tr<T>::MANT, CAP = (MANT / BITS) * BITS;
  const int sh = (pos / CAP) * CAP, p = pos - sh;
  const uint32_t mask = (((1u << BITS) - 1u) << p) * 0x00010001u;
  const uint32_t magic = ((uint32_t)(Tr<T>::EXP_BIAS + MANT - p) << MANT) * 0x00010001u;
  const T2 c = __hsub2(as_t2<T2>(and_or(w >> sh, mask, magic)), as_t2<T2>(magic));  // exact
  return as_u32(__hfma2(c, as_t2<T2>(s2), as_t2<T2>(z2)));
}

// D = A(16x16, row) * B(16x8, col) + D, fp32 accumulate.
template <class T>
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1);
template <>
__device__ __forceinline__ void mma16816<__half>(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                 uint32_t a3, uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
template <>
__device__ __forceinline__ void mma16816<__nv_bfloat16>(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                        uint32_t a3, uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
  uint4 r;
  asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// Pull `bytes` (multiple of 16, 16-byte aligned) starting at `p` into L2; no completion to wait for.
__device__ __forceinline__ void prefetch_l2(const void* p, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(p), "r"(bytes) : "memory");
}

__device__ __forceinline__ void record_check(int32_t* status, int code) { atomicCAS(status, 0, code); }

// Checking build (-DQEVICT_DEBUG_BOUNDS, a library of its own): every page id, window index, work-list entry and
// migration record that a kernel reads from a table is range-checked before it is used as an index; a value out
// of range records a code in the device status word and the access is skipped -- no trap, no assert, the context
// stays usable.  The pools start filled with a NaN pattern in that build, so a read of a page nobody wrote
// surfaces in the results.  In the normal build QE_IN_RANGE is the constant true and costs nothing.
#ifdef QEVICT_DEBUG_BOUNDS
#define QE_IN_RANGE(cond, status, code) ((cond) ? true : (record_check((status), (code)), false))
#else
#define QE_IN_RANGE(cond, status, code) true
#endif

// Programmatic dependent launch: the kernels of a step are enqueued with launch_pdl and begin with
// pdl_prologue().  The prologue first lets the next kernel of the stream start scheduling its CTAs, then
// waits until every earlier kernel has completed and its writes are visible -- so launch latency and CTA
// ramp-up of kernel n+1 overlap the tail of kernel n, while all data dependencies stay intact.
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
}

// Kernel timeline (tracing build only, -DQEVICT_TRACE).  The workspace then carries, for each of the first
// TRACE_CALLS API calls since the timeline was last read, one block per step kernel (0 append, 1 attention,
// 2 combine, 3 route, 4 migrate) of per-SM {earliest warp start, latest warp end} in %globaltimer nanoseconds;
// each warp issues two fire-and-forget reductions on its own SM's pair, so nothing waits on the stamps.
// Block TRACE_CALLS is a sink for the calls beyond the capacity.  In the normal build QE_TRACE_SCOPE is empty.
constexpr int STATUS_BYTES = 256;
#ifdef QEVICT_TRACE
constexpr int TRACE_CALLS = 512;
constexpr int TRACE_KERNELS = 5;
constexpr int TRACE_SMS = 160;  // >= SMs of the device; %smid is folded into the range
constexpr size_t TRACE_CALL_WORDS = (size_t)TRACE_KERNELS * TRACE_SMS * 2;
constexpr size_t TRACE_BYTES = (TRACE_CALLS + 1) * TRACE_CALL_WORDS * 8;
struct TraceScope {
  unsigned long long* slot;
  static __device__ __forceinline__ unsigned long long now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
  }
  __device__ __forceinline__ TraceScope(unsigned long long* call_block, int k) {
    uint32_t smid;
    asm("mov.u32 %0, %%smid;" : "=r"(smid));
    slot = call_block + ((size_t)k * TRACE_SMS + smid % TRACE_SMS) * 2;
    if ((threadIdx.x & 31) == 0) atomicMin(slot, now());
  }
  __device__ __forceinline__ ~TraceScope() {
    if ((threadIdx.x & 31) == 0) atomicMax(slot + 1, now());
  }
};
#define QE_TRACE_SCOPE(block, k) TraceScope qe_trace_scope(block, k)
#else
#define QE_TRACE_SCOPE(block, k)
#endif

template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// ---- kernels launched by the host API (defined in the .cu files) -------------------------------
struct LaunchCtx {
  Geometry geo;
  State st;        // pointers of unit 0; per-unit strides are implied by the geometry
  cudaStream_t stream;
};

}  // namespace qevict
