// Fragment-major page layouts.
//
// A page is stored in the order in which the decode kernel's tensor-core fragments consume it, so
// that every warp-wide 16-byte load is one contiguous 512-byte run and lands in registers (or
// shared memory) already in mma.m16n8k16 operand order.  A 32-token tile of keys is the A operand of
// S^T = K Q^T (m = token, k = channel); a 32-token tile of values is the A operand of O^T = V^T P^T
// (m = channel, k = token).  With lane = 4*g + t:
//
//   key tile, 16-byte vector (ks, mt), ks = channel/16, mt = token/16:
//       lane holds tokens 16mt + 8*rh + g, channels 16ks + 8*hi + 2t + e at element (hi*2 + rh)*2 + e
//   value tile, 16-byte vector (i, ks), i = channel/16, ks = token/16:
//       lane holds channel 16i + 8*ah + g, tokens 16ks + 8*hi + 2t + e at element (hi*2 + ah)*2 + e
//
// Quantized codes use the same (vector, lane, element) coordinates with one code per element, packed
// so that (word >> shift) & mask yields the two codes of a 16-bit pair in the low bits of each half.
// Parameters (scale, zero) are stored as pairs matching the element pairs they multiply.
#pragma once

#include <stdint.h>

namespace qevict {

#if defined(__CUDACC__)
#define QE_HD __host__ __device__ __forceinline__
#else
#define QE_HD inline
#endif

// element offset inside a full-precision key tile
QE_HD int fpk_off(int tk, int ch, int D) {
  (void)D;
  const int mt = tk >> 4, rh = (tk >> 3) & 1, g = tk & 7;
  const int ks = ch >> 4, hi = (ch >> 3) & 1, t = (ch & 7) >> 1, e = ch & 1;
  const int lane = g * 4 + t;
  return ((ks * 2 + mt) * 32 + lane) * 8 + (hi * 2 + rh) * 2 + e;
}

// element offset inside a full-precision value tile
QE_HD int fpv_off(int tk, int ch) {
  const int i = ch >> 4, ah = (ch >> 3) & 1, g = ch & 7;
  const int ks = tk >> 4, hi = (tk >> 3) & 1, t = (tk & 7) >> 1, e = tk & 1;
  const int lane = g * 4 + t;
  return ((i * 2 + ks) * 32 + lane) * 8 + (hi * 2 + ah) * 2 + e;
}

struct CodePos {
  int word;   // 32-bit word offset inside the tile's code block
  int shift;  // bit position of the code inside the word
};

QE_HD int code_word_off(int widx, int lane) { return ((widx >> 2) * 32 + lane) * 4 + (widx & 3); }

// key codes of a tile
QE_HD CodePos kcode_pos(int tk, int ch, int D, int bits) {
  (void)D;
  const int mt = tk >> 4, rh = (tk >> 3) & 1, g = tk & 7;
  const int ks = ch >> 4, hi = (ch >> 3) & 1, t = (ch & 7) >> 1, e = ch & 1;
  const int lane = g * 4 + t;
  const int a = hi * 2 + rh;
  CodePos p;
  if (bits == 4) {
    p.word = code_word_off(ks * 2 + mt, lane);
    p.shift = 4 * a + 16 * e;
  } else {
    p.word = code_word_off(ks, lane);
    p.shift = 2 * (mt * 4 + a) + 16 * e;
  }
  return p;
}

// value codes of a tile
QE_HD CodePos vcode_pos(int tk, int ch, int bits) {
  const int i = ch >> 4, ah = (ch >> 3) & 1, g = ch & 7;
  const int ks = tk >> 4, hi = (tk >> 3) & 1, t = (tk & 7) >> 1, e = tk & 1;
  const int lane = g * 4 + t;
  const int a = hi * 2 + ah;
  CodePos p;
  if (bits == 4) {
    p.word = code_word_off(i * 2 + ks, lane);
    p.shift = 4 * a + 16 * e;
  } else {
    p.word = code_word_off(i, lane);
    p.shift = 2 * (ks * 4 + a) + 16 * e;
  }
  return p;
}

// key parameters of one group of tokens: element offsets (16-bit units) of scale and zero of channel ch
QE_HD int kparam_off(int ch, int is_zero) {
  const int ks = ch >> 4, hi = (ch >> 3) & 1, t = (ch & 7) >> 1, e = ch & 1;
  return (ks * 4 + t) * 8 + (hi * 2 + is_zero) * 2 + e;
}

// value parameters of a tile: scale and zero of (token tk, channel group gc)
QE_HD int vparam_off(int tk, int gc, int is_zero) {
  const int ks = tk >> 4, hi = (tk >> 3) & 1, t = (tk & 7) >> 1, e = tk & 1;
  return ((gc * 2 + ks) * 4 + t) * 8 + (hi * 2 + is_zero) * 2 + e;
}

}  // namespace qevict
