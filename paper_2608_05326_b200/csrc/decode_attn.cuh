// Tiered split-KV flash-decode kernel.
//
// One decode step attends every query head over the accessible tokens of its unit [attention
// equation of the Methodology] and records, per (query head, window), the window's softmax
// numerator, from which the combine kernel forms the window mass of Eq. 1.
//
// Work decomposition: CTA = (split, KV head, unit), 4 warps.  Warp `wid` of split `s` owns one contiguous
// run of the work list; the routing kernel interleaves Full and Quantized windows in the list in
// proportion to their numbers (recent windows last), so every warp alternates between bandwidth-heavy
// 16-bit tiles and arithmetic-heavy low-bit tiles all the way through its walk.  Each
// warp runs an independent online softmax over its windows; the four warps are merged in shared
// memory and the CTA writes one partial (m, l, O) per query head of its KV head.
//
// Data movement: every warp owns a ring of shared-memory slots (two; three with pre-RoPE keys).  Lane 0 streams the warp's
// pages into the ring with bulk asynchronous copies (cp.async.bulk, completion counted on one
// mbarrier per slot) one piece ahead of the math; a page is stored fragment-major (layout.cuh),
// so a piece is one contiguous run in global memory and every lane reads its operands from shared
// memory with conflict-free 16-byte loads.  Waits on the mbarriers are bounded: a wait that runs out
// records CHECK_COPY_TIMEOUT, the warp stops issuing, drains what it has in flight and returns.
//
// Per 32-token tile:  S^T = K Q^T with tokens on the M side of mma.m16n8k16, channels on K and the (<= 8)
// grouped heads on N (all 16 rows of every product are useful), softmax in fp32 in the log2 domain,
// O^T += V^T P^T with channels on M, tokens on K and heads on N; the probability fragments are turned
// from (token, head) into (head, token) operands by 8x8 register transposes (movmatrix).  The
// probabilities enter it as a 16-bit value plus its rounding residual; with at most 4 heads per KV
// head the residuals ride in the unused N columns 4..7 of the same product (PACK), otherwise they take
// a second product.  A quantized tile is read as packed words, and codes become operands in
// registers with one exact subtract and one fused multiply-add per pair.
//
// Pre-RoPE keys (ROPE instantiations) [Migration-Stable Quantization: keys in the pre-RoPE domain with their
// absolute positions, RoPE reapplied after dequantization]: the ring has a third slot, into which the
// rotation block of the tile's 32 positions follows the piece that holds the keys; the key fragments of
// k-steps ks and ks + KS/2 (rotation partners sit in the same lane and register) are rotated in registers,
// full-precision tiles as loaded and low-bit tiles after dequantization, before the products.
#pragma once

#include <atomic>

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
  float2* wrec;           // [n_units][EMAX][Hq]
  int32_t* status;
  int unit0, S, Hq, Hkv, G, EMAX, PF, PQ, NW;
  int e_bound;            // upper bound of every unit's work-list length (host's mirror of the window counts)
  uint32_t fp_page_bytes, q_page_bytes;
  float scale_log2;
  const char* rope;       // pre-RoPE keys: blocks of cos / sin pairs, one per 32 positions, in the key tile's fragment order
#ifdef QEVICT_TRACE
  unsigned long long* trace;  // this call's block of the kernel timeline
#endif
};

static constexpr uint32_t WAIT_LIMIT = 1u << 20;  // mbarrier try_wait attempts before giving up

template <class T, int D, int BITS, int GROUP, int TILES, bool ROPE>
struct DecodeTraits {
  // ring slots per warp: with pre-RoPE keys a tile's rotation block sits in the ring beside the key tile
  static constexpr int NSLOT = ROPE ? 3 : 2;
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
  // a ring slot holds a full-precision key tile or value tile, or a whole quantized tile
  // (key codes, value codes, value params as they lie in the page, then the key params)
  static constexpr uint32_t SLOT_BYTES = FP_TILE_BYTES;
  static constexpr uint32_t ROPE_BLOCK_BYTES = 32 * (D / 2) * 4;  // (cos, sin) of 32 positions x d/2 frequencies
  static_assert(ROPE_BLOCK_BYTES <= SLOT_BYTES, "a rotation block must fit a slot");
  static constexpr uint32_t RING_BYTES = DECODE_WARPS * NSLOT * SLOT_BYTES;
  static constexpr uint32_t SMEM_BYTES = RING_BYTES + DECODE_WARPS * NSLOT * 8;
  static_assert(Q_TILE_STRIDE + KP_BYTES <= SLOT_BYTES, "a quantized tile must fit a slot");
  static_assert(8 * (D + 4) * 4 + 64 <= NSLOT * SLOT_BYTES, "merge buffer must fit the warp's ring");
};

// ---- shared-memory / mbarrier / bulk-copy primitives -------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint4 lds16(uint32_t addr) {
  uint4 r;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
  return r;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait; false if the phase did not complete within WAIT_LIMIT attempts.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  return false;
}
// Pages are read once per step and a step reads several times the L2's capacity, so the copies carry an
// evict-first policy: the stream of pages then leaves the small tables, the partials and the code of the
// step's other kernels in L2 instead of flushing them every step.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}

// The same without a cache hint: the rotation table of pre-RoPE keys is shared by every unit and KV head and
// should stay in L2.
__device__ __forceinline__ void bulk_g2s_plain(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// ---- S^T = K Q^T ---------------------------------------------------------------------------------------
// Tokens on M (two blocks of 16), channels on K, the (<= 8) grouped heads on N.  s[mt] = {(token g, head 2t),
// (token g, head 2t+1), (token g+8, head 2t), (token g+8, head 2t+1)} of token block mt.
// A full-precision key tile (32 tokens) from a ring slot.
template <class T, int D>
__device__ __forceinline__ void qk_fp_tile(float (&s)[2][4], const uint32_t (&qa)[D / 16][2], uint32_t slot, int lane) {
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      const uint4 kv = lds16(slot + ((ks * 2 + mt) * 32 + lane) * 16);
      mma16816<T>(s[mt], kv.x, kv.y, kv.z, kv.w, qa[ks][0], qa[ks][1]);
    }
  }
}

// Key part of a quantized tile: codes at `slot`, parameters at `kp`.  One 16-byte code vector covers two
// k-steps (four with 2-bit codes) for both token blocks and is fetched right before it is used.
template <class T, int D, int BITS>
__device__ __forceinline__ void qk_q_tile(float (&s)[2][4], const uint32_t (&qa)[D / 16][2], uint32_t slot, uint32_t kp,
                                          int lane) {
  constexpr int KS = D / 16;
  constexpr int KPV = (BITS == 4) ? 2 : 4;  // k-steps per code vector
  const int t = lane & 3;
#pragma unroll
  for (int v = 0; v < KS / KPV; ++v) {
    const uint4 cv = lds16(slot + (v * 32 + lane) * 16);
    const uint32_t cw[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
    for (int kk = 0; kk < KPV; ++kk) {
      const int ks = v * KPV + kk;
      const uint4 pr = lds16(kp + (ks * 4 + t) * 16);  // {s,z} of channels 2t,2t+1 and of channels 2t+8,2t+9
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const uint32_t w = (BITS == 4) ? cw[kk * 2 + mt] : cw[kk];
        const int sh = (BITS == 4) ? 0 : mt * 8;
        const uint32_t a0 = dequant_at<T, BITS>(w, sh + 0 * BITS, pr.x, pr.y);
        const uint32_t a1 = dequant_at<T, BITS>(w, sh + 1 * BITS, pr.x, pr.y);
        const uint32_t a2 = dequant_at<T, BITS>(w, sh + 2 * BITS, pr.z, pr.w);
        const uint32_t a3 = dequant_at<T, BITS>(w, sh + 3 * BITS, pr.z, pr.w);
        mma16816<T>(s[mt], a0, a1, a2, a3, qa[ks][0], qa[ks][1]);
      }
    }
  }
}

// ---- pre-RoPE keys: S^T = R(K) Q^T ---------------------------------------------------------------------------
// The partner of channel c < d/2 is channel c + d/2: the same lane, the same register, KS/2 k-steps further on.
// A rotation block holds, for k-step ks' < KS/2 and token block mt, two 16-byte vectors per lane:
// {C r0, S r0, C r1, S r1} and {C r2, S r2, C r3, S r3}, C / S = the (cos, sin) pairs of register r's two channels
// at register r's token row.  x' = RN(RN(x c) - RN(y s)), y' = RN(RN(y c) + RN(x s)) in the execution datatype,
// every operation rounded on its own (the _rn intrinsics are never contracted into a fused multiply-add).
template <class T>
__device__ __forceinline__ void rope_pair(uint32_t& x, uint32_t& y, uint32_t c, uint32_t s) {
  using T2 = typename Tr<T>::T2;
  const T2 X = as_t2<T2>(x), Y = as_t2<T2>(y), C = as_t2<T2>(c), S = as_t2<T2>(s);
  x = as_u32(__hsub2_rn(__hmul2_rn(X, C), __hmul2_rn(Y, S)));
  y = as_u32(__hadd2_rn(__hmul2_rn(Y, C), __hmul2_rn(X, S)));
}
template <class T>
__device__ __forceinline__ void rope_fragments(uint4& a, uint4& b, uint32_t rslot, int ksp, int mt, int lane) {
  const uint4 c0 = lds16(rslot + (((ksp * 2 + mt) * 2 + 0) * 32 + lane) * 16);
  const uint4 c1 = lds16(rslot + (((ksp * 2 + mt) * 2 + 1) * 32 + lane) * 16);
  rope_pair<T>(a.x, b.x, c0.x, c0.y);
  rope_pair<T>(a.y, b.y, c0.z, c0.w);
  rope_pair<T>(a.z, b.z, c1.x, c1.y);
  rope_pair<T>(a.w, b.w, c1.z, c1.w);
}

template <class T, int D>
__device__ __forceinline__ void qk_fp_tile_rope(float (&s)[2][4], const uint32_t (&qa)[D / 16][2], uint32_t slot,
                                                uint32_t rslot, int lane) {
  constexpr int KS = D / 16;
#pragma unroll
  for (int ksp = 0; ksp < KS / 2; ++ksp) {
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      uint4 a = lds16(slot + ((ksp * 2 + mt) * 32 + lane) * 16);
      uint4 b = lds16(slot + (((ksp + KS / 2) * 2 + mt) * 32 + lane) * 16);
      rope_fragments<T>(a, b, rslot, ksp, mt, lane);
      mma16816<T>(s[mt], a.x, a.y, a.z, a.w, qa[ksp][0], qa[ksp][1]);
      mma16816<T>(s[mt], b.x, b.y, b.z, b.w, qa[ksp + KS / 2][0], qa[ksp + KS / 2][1]);
    }
  }
}

template <class T, int D, int BITS>
__device__ __forceinline__ void qk_q_tile_rope(float (&s)[2][4], const uint32_t (&qa)[D / 16][2], uint32_t slot, uint32_t kp,
                                               uint32_t rslot, int lane) {
  constexpr int KS = D / 16;
  constexpr int KPV = (BITS == 4) ? 2 : 4;  // k-steps per code vector
  const int t = lane & 3;
  uint32_t cw[KS / KPV][4];
#pragma unroll
  for (int v = 0; v < KS / KPV; ++v) {
    const uint4 cv = lds16(slot + (v * 32 + lane) * 16);
    cw[v][0] = cv.x; cw[v][1] = cv.y; cw[v][2] = cv.z; cw[v][3] = cv.w;
  }
  auto fragment = [&](int ks, int mt, const uint4& pr) -> uint4 {
    const uint32_t w = (BITS == 4) ? cw[ks / KPV][(ks % KPV) * 2 + mt] : cw[ks / KPV][ks % KPV];
    const int sh = (BITS == 4) ? 0 : mt * 8;
    uint4 a;
    a.x = dequant_at<T, BITS>(w, sh + 0 * BITS, pr.x, pr.y);
    a.y = dequant_at<T, BITS>(w, sh + 1 * BITS, pr.x, pr.y);
    a.z = dequant_at<T, BITS>(w, sh + 2 * BITS, pr.z, pr.w);
    a.w = dequant_at<T, BITS>(w, sh + 3 * BITS, pr.z, pr.w);
    return a;
  };
#pragma unroll
  for (int ksp = 0; ksp < KS / 2; ++ksp) {
    const uint4 pra = lds16(kp + (ksp * 4 + t) * 16), prb = lds16(kp + ((ksp + KS / 2) * 4 + t) * 16);
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      uint4 a = fragment(ksp, mt, pra), b = fragment(ksp + KS / 2, mt, prb);
      rope_fragments<T>(a, b, rslot, ksp, mt, lane);
      mma16816<T>(s[mt], a.x, a.y, a.z, a.w, qa[ksp][0], qa[ksp][1]);
      mma16816<T>(s[mt], b.x, b.y, b.z, b.w, qa[ksp + KS / 2][0], qa[ksp + KS / 2][1]);
    }
  }
}

// ---- O^T += V^T P^T ----------------------------------------------------------------------------------------
// A full-precision value tile from a ring slot.
template <class T, int D, bool PACK>
__device__ __forceinline__ void pv_fp_tile(float (&o)[D / 16][4], const uint32_t (&pa)[2][2], const uint32_t (&pb)[2][2],
                                           uint32_t slot, int lane) {
#pragma unroll
  for (int ks = 0; ks < 2; ++ks) {
#pragma unroll
    for (int i = 0; i < D / 16; ++i) {
      const uint4 vv = lds16(slot + ((i * 2 + ks) * 32 + lane) * 16);
      mma16816<T>(o[i], vv.x, vv.y, vv.z, vv.w, pa[ks][0], pa[ks][1]);
      if (!PACK) mma16816<T>(o[i], vv.x, vv.y, vv.z, vv.w, pb[ks][0], pb[ks][1]);
    }
  }
}

// Value part of a quantized tile: codes at `slot`, parameters at `slot + VC_BYTES`.  One 16-byte code
// vector covers two channel blocks (four with 2-bit codes) and is fetched right before it is used.
template <class T, int D, int BITS, int GROUP, bool PACK>
__device__ __forceinline__ void pv_q_tile(float (&o)[D / 16][4], const uint32_t (&pa)[2][2], const uint32_t (&pb)[2][2],
                                          uint32_t slot, int lane) {
  constexpr int MT = D / 16;
  constexpr uint32_t VC_BYTES = 32 * D * BITS / 8;
  constexpr int IPV = (BITS == 4) ? 2 : 4;  // channel blocks (of 16) per code vector
  const int t = lane & 3;
  const uint32_t vp = slot + VC_BYTES;
  uint4 pr0 = make_uint4(0u, 0u, 0u, 0u), pr1 = pr0;
#pragma unroll
  for (int v = 0; v < MT / IPV; ++v) {
    const uint4 cv = lds16(slot + (v * 32 + lane) * 16);
    const uint32_t vw[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
    for (int ii = 0; ii < IPV; ++ii) {
      const int i = v * IPV + ii;
      if ((16 * i) % GROUP == 0) {  // a new channel group starts: its per-token parameters
        const int gc = (16 * i) / GROUP;
        pr0 = lds16(vp + ((gc * 2 + 0) * 4 + t) * 16);  // tokens 0..15:  {s,z} low octet, {s,z} high octet
        pr1 = lds16(vp + ((gc * 2 + 1) * 4 + t) * 16);  // tokens 16..31
      }
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        const uint4 pr = ks ? pr1 : pr0;
        const uint32_t w = (BITS == 4) ? vw[ii * 2 + ks] : vw[ii];
        const int sh = (BITS == 4) ? 0 : ks * 8;
        const uint32_t a0 = dequant_at<T, BITS>(w, sh + 0 * BITS, pr.x, pr.y);
        const uint32_t a1 = dequant_at<T, BITS>(w, sh + 1 * BITS, pr.x, pr.y);
        const uint32_t a2 = dequant_at<T, BITS>(w, sh + 2 * BITS, pr.z, pr.w);
        const uint32_t a3 = dequant_at<T, BITS>(w, sh + 3 * BITS, pr.z, pr.w);
        mma16816<T>(o[i], a0, a1, a2, a3, pa[ks][0], pa[ks][1]);
        if (!PACK) mma16816<T>(o[i], a0, a1, a2, a3, pb[ks][0], pb[ks][1]);
      }
    }
  }
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

// Transpose an 8x8 block of 16-bit elements held one row pair per lane (row = lane / 4, columns
// 2 * (lane % 4) and +1): turns probabilities indexed (token, head) into the (head, token) operand of PV.
__device__ __forceinline__ uint32_t transpose8x8(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}

// Online softmax update for one tile.  A lane owns heads 2t and 2t+1 (index 0 / 1 of m_run, l_part, wsum)
// and tokens g, g+8, g+16, g+24 of the tile; the reference exponent m_run of a head is the same in the 8 lanes
// of equal t, while l_part and wsum are the lane's own share of the sums (added over the 8 lanes by the caller,
// once per window and once at the end).  m_run is a reference, not necessarily the maximum: a tile whose
// logits stay below m_run + REF_SLACK keeps it (its probabilities are then at most 2^REF_SLACK, far inside
// the range of every format they pass through), so the common tile costs no reduction over lanes and no
// rescaling; only a tile that exceeds the slack moves the reference to the true maximum so far.
// With PACK the query heads sit in columns 0..3 of the products and once more in columns 4..7, so lanes
// t >= 2 see the same logits as lanes t - 2 and contribute the rounding residuals of the same probabilities.
// Leaves the probability fragments for the PV product in pa / pb.
constexpr float REF_SLACK = 8.f;
template <class T, int MT, bool PACK>
__device__ __forceinline__ void softmax_tile(float (&s)[2][4], int ntok, float scale_log2, int lane, float (&m_run)[2],
                                             float (&l_part)[2], float (&wsum)[2], float (&o)[MT][4],
                                             uint32_t (&pa)[2][2], uint32_t (&pb)[2][2]) {
  const int g = lane >> 2;
  float x[2][2][2];  // raw logits, [token block][row half][head]; the softmax scale is folded into the exponent below
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      x[mt][r][0] = s[mt][2 * r];
      x[mt][r][1] = s[mt][2 * r + 1];
    }
  }
  if (ntok < 32) {  // only the open window has unfilled token slots
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        if (16 * mt + 8 * r + g >= ntok) { x[mt][r][0] = -INFINITY; x[mt][r][1] = -INFINITY; }
      }
    }
  }
  float lm[2];  // the lane's largest scaled logit per head (the scale is positive)
#pragma unroll
  for (int h = 0; h < 2; ++h) lm[h] = fmaxf(fmaxf(x[0][0][h], x[0][1][h]), fmaxf(x[1][0][h], x[1][1][h])) * scale_log2;
  if (__any_sync(0xffffffffu, lm[0] > m_run[0] + REF_SLACK || lm[1] > m_run[1] + REF_SLACK)) {
    float alpha[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float tmax = lm[h];
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 4));
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 8));
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 16));
      const float m_new = fmaxf(m_run[h], tmax);  // finite: the caller guarantees ntok >= 1
      alpha[h] = ex2(m_run[h] - m_new);
      l_part[h] *= alpha[h];
      wsum[h] *= alpha[h];
      m_run[h] = m_new;
    }
    // the accumulators hold O^T with the lane's own two heads as its columns
#pragma unroll
    for (int i = 0; i < MT; ++i) {
      o[i][0] *= alpha[0]; o[i][1] *= alpha[1]; o[i][2] *= alpha[0]; o[i][3] *= alpha[1];
    }
  }
  float p[2][2][2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float rs = 0.f;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        p[mt][r][h] = ex2(fmaf(x[mt][r][h], scale_log2, -m_run[h]));
        rs += p[mt][r][h];
      }
    }
    l_part[h] += rs;
    wsum[h] += rs;
  }
  // probabilities as (token, head) pairs -> 16-bit value + residual -> transposed into the B operand
  // (k = token, n = head): block (mt, r) becomes register r of k-step mt
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      uint32_t main, res;
      split_pair<T>(p[mt][r][0], p[mt][r][1], main, res);
      if (PACK) {
        // columns 0..3 carry the probabilities, columns 4..7 their residuals, in the same product
        pa[mt][r] = transpose8x8((lane & 3) >= 2 ? res : main);
      } else {
        pa[mt][r] = transpose8x8(main);
        pb[mt][r] = transpose8x8(res);
      }
    }
  }
}

// sum over the 8 lanes of equal lane % 4
__device__ __forceinline__ float sum_over_g(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 4);
  v += __shfl_xor_sync(0xffffffffu, v, 8);
  v += __shfl_xor_sync(0xffffffffu, v, 16);
  return v;
}

template <class T, int D, int BITS, int GROUP, int TILES, bool PACK, bool ROPE>
__global__ void __launch_bounds__(DECODE_WARPS * 32, ROPE ? 2 : 3) decode_attn_kernel(const DecodeParams p) {
  using TT = DecodeTraits<T, D, BITS, GROUP, TILES, ROPE>;
  constexpr int KS = TT::KS, MT = TT::MT, NSLOT = TT::NSLOT;
  extern __shared__ __align__(128) unsigned char smem[];
  const int s = blockIdx.x, hk = blockIdx.y, ul = blockIdx.z;
  const int u = p.unit0 + ul;
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const uint32_t ring = smem_u32(smem) + wid * NSLOT * TT::SLOT_BYTES;
  const uint32_t bars = smem_u32(smem) + TT::RING_BYTES + wid * NSLOT * 8;
  pdl_prologue();
  QE_TRACE_SCOPE(p.trace, 1);
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NSLOT; ++i) mbar_init(bars + i * 8, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncwarp();

  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // heads 2t and 2t+1
  float o[MT][4];
#pragma unroll
  for (int i = 0; i < MT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }

  // Every warp of the (unit, KV head) takes one contiguous run of the work list: the list interleaves Full and
  // Quantized windows in proportion, so any run holds the same mix of 16-bit and low-bit pages (a strided walk
  // would alias with the interleaving period for some split counts).  The runs are cut from the host's upper
  // bound of the list length, so the entries are fetched without waiting for the length itself (the slots
  // exist up to EMAX; what lies past the end is masked afterwards): start-up costs one global round trip.
  const int n_warps = p.S * DECODE_WARPS, gw = s * DECODE_WARPS + wid;
  const int run = p.e_bound / n_warps, extra = p.e_bound - run * n_warps;
  const int first = gw * run + min(gw, extra), my_cap = run + (gw < extra ? 1 : 0);  // <= 32: the host picks S so
  uint2 my_ent = make_uint2(0u, 0u);
  if (lane < my_cap && first + lane < p.EMAX) my_ent = p.entries[(size_t)u * p.EMAX + first + lane];
  const int n_live = p.n_live[u];
  const int fill = p.open_fill[u];
  int my_n = max(0, min(my_cap, n_live - first));
  // the runs cover the host's bound of the list length: a longer list would be attended to only in part
  if (n_live > p.e_bound && s == 0 && threadIdx.x == 0) record_check(p.status, CHECK_ENTRY_OVERFLOW);
#ifdef QEVICT_DEBUG_BOUNDS
  {  // an entry with an impossible kind, window or page ends the warp's run before it
    const uint32_t kind = my_ent.x >> ENTRY_KIND_SHIFT, win = my_ent.x & ENTRY_WINDOW_MASK;
    const bool bad = lane < my_n && (kind > KIND_OPEN || win >= (uint32_t)p.NW || my_ent.y >= (uint32_t)(kind == KIND_Q ? p.PQ : p.PF));
    const unsigned bad_lanes = __ballot_sync(0xffffffffu, bad);
    if (bad_lanes) {
      if (lane == 0) record_check(p.status, CHECK_BOUNDS_ENTRY);
      my_n = min(my_n, __ffs(bad_lanes) - 1);
    }
  }
#endif
  if (lane >= my_n) my_ent = make_uint2(0u, 0u);

  // ---- producer: pieces are issued in consumption order into slots 0,1,..,NSLOT-1,0,.. ------------------
  // pieces per tile: full precision = key tile, value tile; quantized = the whole tile; with pre-RoPE keys the
  // tile's rotation block follows the piece that holds the keys
  int pr_ci = 0, pr_tile = 0, pr_part = 0, issued = 0, consumed = 0;
  bool dead = false, pr_isq = false;
  uint32_t pr_win = 0;
  const char* pr_base = nullptr;  // page of the producer's current entry (this KV head), set on its first piece
  const char* const fp_unit = p.fp_pool + (size_t)u * p.PF * p.fp_page_bytes + (size_t)hk * TT::FP_HEAD_BYTES;
  const char* const q_unit = p.q_pool + (size_t)u * p.PQ * p.q_page_bytes + (size_t)hk * TT::Q_HEAD_BYTES;
  const uint64_t l2pol = l2_evict_first_policy();
  auto issue_next = [&]() {  // warp-collective
    if (pr_ci >= my_n || dead) return;  // every piece of every entry of this warp has been issued
    if (pr_tile == 0 && pr_part == 0) {
      const uint32_t ex = __shfl_sync(0xffffffffu, my_ent.x, pr_ci), ey = __shfl_sync(0xffffffffu, my_ent.y, pr_ci);
      pr_isq = (ex >> ENTRY_KIND_SHIFT) == KIND_Q;
      pr_win = ex & ENTRY_WINDOW_MASK;
      pr_base = pr_isq ? q_unit + (size_t)ey * p.q_page_bytes : fp_unit + (size_t)ey * p.fp_page_bytes;
    }
    const bool is_rope = ROPE && pr_part == 1;
    if (lane == 0) {
      const int slot = issued % NSLOT;
      const uint32_t dst = ring + slot * TT::SLOT_BYTES, bar = bars + slot * 8;
      if (is_rope) {
        mbar_expect_tx(bar, TT::ROPE_BLOCK_BYTES);
        bulk_g2s_plain(dst, p.rope + ((size_t)pr_win * TILES + pr_tile) * TT::ROPE_BLOCK_BYTES, TT::ROPE_BLOCK_BYTES, bar);
      } else if (!pr_isq) {
        const int half = pr_part ? 1 : 0;  // key tile, then value tile
        mbar_expect_tx(bar, TT::FP_TILE_BYTES);
        bulk_g2s(dst, pr_base + (size_t)(pr_tile * 2 + half) * TT::FP_TILE_BYTES, TT::FP_TILE_BYTES, bar, l2pol);
      } else {
        mbar_expect_tx(bar, TT::Q_TILE_STRIDE + TT::KP_BYTES);
        bulk_g2s(dst, pr_base + (size_t)pr_tile * TT::Q_TILE_STRIDE, TT::Q_TILE_STRIDE, bar, l2pol);
        bulk_g2s(dst + TT::Q_TILE_STRIDE, pr_base + TT::KP_OFF + (size_t)((pr_tile * 32) / GROUP) * TT::KP_BYTES, TT::KP_BYTES, bar, l2pol);
      }
    }
    ++issued;
    if (++pr_part == (pr_isq ? 1 : 2) + (ROPE ? 1 : 0)) {
      pr_part = 0;
      if (++pr_tile == TILES) { pr_tile = 0; ++pr_ci; }
    }
  };
  // wait for the piece `ahead` places after the next one in order; returns its slot address
  auto acquire = [&](int ahead = 0) -> uint32_t {
    const int k = consumed + ahead, slot = k % NSLOT;
    if (!dead && !mbar_wait(bars + slot * 8, (k / NSLOT) & 1)) {
      dead = true;
      if (lane == 0) record_check(p.status, CHECK_COPY_TIMEOUT);
    }
    return ring + slot * TT::SLOT_BYTES;
  };
  auto release = [&]() {  // all lanes have read the slot: hand it back to the producer
    ++consumed;
    __syncwarp();
    issue_next();
  };
#pragma unroll 1
  for (int i = 0; i < NSLOT; ++i) issue_next();

  // query fragments: column g of the B operand = head hk*G + g (columns >= G are zero)
  uint32_t qa[KS][2];
  {
    // with PACK (at most 4 heads per KV head) the heads fill columns 0..3 and, again, columns 4..7
    const int gh = PACK ? (g & 3) : g;
    const T* qrow = reinterpret_cast<const T*>(p.q) + ((size_t)ul * p.Hq + (size_t)hk * p.G + gh) * D;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      if (gh < p.G) {
        qa[ks][0] = *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * t);
        qa[ks][1] = *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * t);
      } else {
        qa[ks][0] = 0u; qa[ks][1] = 0u;
      }
    }
  }


#pragma unroll 1
  for (int ci = 0; ci < my_n; ++ci) {
    const uint32_t ex = __shfl_sync(0xffffffffu, my_ent.x, ci);
    const uint32_t kind = ex >> ENTRY_KIND_SHIFT;
    const int e = first + ci;
    const int valid = (kind == KIND_OPEN) ? fill : TT::W;
    float wsum[2] = {0.f, 0.f};
#pragma unroll 1
    for (int tile = 0; tile < TILES; ++tile) {
      const int ntok = min(32, valid - 32 * tile);
      float sacc[2][4];
#pragma unroll
      for (int j = 0; j < 2; ++j) { sacc[j][0] = sacc[j][1] = sacc[j][2] = sacc[j][3] = 0.f; }
      uint32_t pa[2][2], pb[2][2];
      if (kind != KIND_Q) {
        uint32_t sl = acquire();
        if (ROPE) {
          const uint32_t rs = acquire(1);
          if (!dead && ntok > 0) {
            qk_fp_tile_rope<T, D>(sacc, qa, sl, rs, lane);
            softmax_tile<T, MT, PACK>(sacc, ntok, p.scale_log2, lane, m_run, l_run, wsum, o, pa, pb);
          }
          release();
        } else if (!dead && ntok > 0) {
          qk_fp_tile<T, D>(sacc, qa, sl, lane);
          softmax_tile<T, MT, PACK>(sacc, ntok, p.scale_log2, lane, m_run, l_run, wsum, o, pa, pb);
        }
        release();
        sl = acquire();
        if (!dead && ntok > 0) pv_fp_tile<T, D, PACK>(o, pa, pb, sl, lane);
        release();
      } else {
        const uint32_t sl = acquire();
        const uint32_t rs = ROPE ? acquire(1) : 0u;
        if (!dead) {
          if (ROPE) qk_q_tile_rope<T, D, BITS>(sacc, qa, sl, sl + TT::Q_TILE_STRIDE, rs, lane);
          else qk_q_tile<T, D, BITS>(sacc, qa, sl, sl + TT::Q_TILE_STRIDE, lane);
          softmax_tile<T, MT, PACK>(sacc, 32, p.scale_log2, lane, m_run, l_run, wsum, o, pa, pb);
          pv_q_tile<T, D, BITS, GROUP, PACK>(o, pa, pb, sl + TT::KC_BYTES, lane);
        }
        release();
        if (ROPE) release();
      }
    }
    wsum[0] = sum_over_g(wsum[0]);
    wsum[1] = sum_over_g(wsum[1]);
    if (g == 0) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (2 * t + h < p.G) p.wrec[((size_t)u * p.EMAX + e) * p.Hq + hk * p.G + 2 * t + h] = make_float2(wsum[h], m_run[h]);
      }
    }
  }
  if (dead) {
    // give the copies still in flight a bounded time to land before the shared memory is reused
    for (int k = consumed; k < issued; ++k) mbar_wait(bars + (k % NSLOT) * 8, (k / NSLOT) & 1);
  }

  // ---- merge the four warps (each parks its state in its own, now idle, ring), write the partial ------
  // per-warp layout: float o[8][D + 4], then float m[8], float l[8]
  constexpr int OSTR = D + 4;
  float* my_o = reinterpret_cast<float*>(smem + wid * NSLOT * TT::SLOT_BYTES);
  float* my_ml = my_o + 8 * OSTR;
  l_run[0] = sum_over_g(l_run[0]);
  l_run[1] = sum_over_g(l_run[1]);
  if (g == 0) { my_ml[2 * t] = m_run[0]; my_ml[2 * t + 1] = m_run[1]; my_ml[8 + 2 * t] = l_run[0]; my_ml[8 + 2 * t + 1] = l_run[1]; }
#pragma unroll
  for (int i = 0; i < MT; ++i) {
    my_o[(2 * t) * OSTR + 16 * i + g] = o[i][0];
    my_o[(2 * t + 1) * OSTR + 16 * i + g] = o[i][1];
    my_o[(2 * t) * OSTR + 16 * i + g + 8] = o[i][2];
    my_o[(2 * t + 1) * OSTR + 16 * i + g + 8] = o[i][3];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < p.G * D; idx += DECODE_WARPS * 32) {
    const int h = idx / D, ch = idx - h * D;
    float mw[DECODE_WARPS];
    float mx = -INFINITY;
#pragma unroll
    for (int w = 0; w < DECODE_WARPS; ++w) {
      const float* wo = reinterpret_cast<const float*>(smem + w * NSLOT * TT::SLOT_BYTES);
      mw[w] = wo[8 * OSTR + h];
      mx = fmaxf(mx, mw[w]);
    }
    float acc = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < DECODE_WARPS; ++w) {
      const float* wo = reinterpret_cast<const float*>(smem + w * NSLOT * TT::SLOT_BYTES);
      const float sc = (mw[w] == -INFINITY) ? 0.f : ex2(mw[w] - mx);
      float ov = wo[h * OSTR + ch];
      if (PACK) ov += wo[(h + 4) * OSTR + ch];  // residual columns
      acc += ov * sc;
      l += wo[8 * OSTR + 8 + h] * sc;
    }
    const size_t ph = ((size_t)u * p.Hq + (size_t)hk * p.G + h) * MAX_SPLITS + s;
    p.o_part[ph * D + ch] = acc;
    if (ch == 0) { p.ml[ph * 2] = mx; p.ml[ph * 2 + 1] = l; }
  }
}

template <class T, int D, int BITS, int GROUP, int TILES, bool PACK, bool ROPE>
cudaError_t launch_decode_attn(const DecodeParams& p, int n_units, cudaStream_t stream) {
  using TT = DecodeTraits<T, D, BITS, GROUP, TILES, ROPE>;
  // the shared-memory attribute of a kernel is kept per device: set it the first time this instantiation is
  // launched on the current device (one bit per device ordinal; ordinals past 63 set it every time)
  static std::atomic<unsigned long long> prepared{0ull};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = dev < 64 ? 1ull << dev : 0ull;
  if (!(prepared.load(std::memory_order_acquire) & bit) || !bit) {
    e = cudaFuncSetAttribute(decode_attn_kernel<T, D, BITS, GROUP, TILES, PACK, ROPE>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TT::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    prepared.fetch_or(bit, std::memory_order_release);
  }
  dim3 grid(p.S, p.Hkv, n_units);
  return launch_pdl(decode_attn_kernel<T, D, BITS, GROUP, TILES, PACK, ROPE>, grid, dim3(DECODE_WARPS * 32), TT::SMEM_BYTES, stream, p);
}

// explicit dispatch table entry points, one per (dtype, D) translation unit
typedef cudaError_t (*decode_launch_fn)(const DecodeParams&, int, cudaStream_t);
decode_launch_fn decode_dispatch_h64(int bits, int group, int tiles, int heads_per_kv, bool rope);
decode_launch_fn decode_dispatch_h128(int bits, int group, int tiles, int heads_per_kv, bool rope);
decode_launch_fn decode_dispatch_b64(int bits, int group, int tiles, int heads_per_kv, bool rope);
decode_launch_fn decode_dispatch_b128(int bits, int group, int tiles, int heads_per_kv, bool rope);

#define QEVICT_DECODE_CASE(T, D, B, G, TL)    \
  if (bits == B && group == G && tiles == TL) \
    return rope ? (heads_per_kv <= 4 ? launch_decode_attn<T, D, B, G, TL, true, true> : launch_decode_attn<T, D, B, G, TL, false, true>) \
                : (heads_per_kv <= 4 ? launch_decode_attn<T, D, B, G, TL, true, false> : launch_decode_attn<T, D, B, G, TL, false, false>);

#define QEVICT_DECODE_DISPATCH(NAME, T, D)                                  \
  decode_launch_fn NAME(int bits, int group, int tiles, int heads_per_kv, bool rope) { \
    QEVICT_DECODE_CASE(T, D, 4, 32, 1)                                      \
    QEVICT_DECODE_CASE(T, D, 2, 32, 1)                                      \
    QEVICT_DECODE_CASE(T, D, 4, 32, 2)                                      \
    QEVICT_DECODE_CASE(T, D, 2, 32, 2)                                      \
    QEVICT_DECODE_CASE(T, D, 4, 64, 2)                                      \
    QEVICT_DECODE_CASE(T, D, 2, 64, 2)                                      \
    return nullptr;                                                         \
  }

}  // namespace qevict
