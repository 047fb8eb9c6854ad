// Fragment-major page layouts.
//
// A page is stored in the order in which the decode kernel's tensor-core fragments consume it, so
// that every warp-wide 16-byte load is one contiguous 512-byte run and lands in registers (or
// shared memory) already in mma.m16n8k16 operand order.  A 32-token tile of keys is the B operand of
// S = Q K^T (k = channel, n = token); a 32-token tile of values is the A operand of O^T = V^T P^T
// (m = channel, k = token).  With lane = 4*g + t:
//
//   key tile, 16-byte vector (j, c), j = token/8, c = channel/32:
//       lane holds token 8j+g, channels 32c + 16*ks + 8*hi + 2t + e   at element ks*4 + hi*2 + e
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
  const int j = tk >> 3, g = tk & 7;
  const int c = ch >> 5, r = ch & 31;
  const int ks = r >> 4, hi = (r >> 3) & 1, t = (r & 7) >> 1, e = r & 1;
  const int lane = g * 4 + t;
  return ((j * (D >> 5) + c) * 32 + lane) * 8 + ks * 4 + hi * 2 + e;
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
  const int j = tk >> 3, g = tk & 7;
  const int c = ch >> 5, r = ch & 31;
  const int ks = r >> 4, hi = (r >> 3) & 1, t = (r & 7) >> 1, e = r & 1;
  const int lane = g * 4 + t;
  const int m = ks * 2 + hi;
  CodePos p;
  // word index = channel-group * 4 + token block: one 16-byte vector holds the four token blocks of a
  // channel group, so the attention kernel fetches the codes of one k-step pair at a time
  if (bits == 4) {
    p.word = code_word_off(c * 4 + j, lane);
    p.shift = 4 * m + 16 * e;
  } else {
    p.word = code_word_off((c >> 1) * 4 + j, lane);
    p.shift = 2 * ((c & 1) * 4 + m) + 16 * e;
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
  const int c = ch >> 5, r = ch & 31;
  const int ks = r >> 4, hi = (r >> 3) & 1, t = (r & 7) >> 1, e = r & 1;
  return ((c * 2 + ks) * 4 + t) * 8 + (hi * 2 + is_zero) * 2 + e;
}

// value parameters of a tile: scale and zero of (token tk, channel group gc)
QE_HD int vparam_off(int tk, int gc, int is_zero) {
  const int ks = tk >> 4, hi = (tk >> 3) & 1, t = (tk & 7) >> 1, e = tk & 1;
  return ((gc * 2 + ks) * 4 + t) * 8 + (hi * 2 + is_zero) * 2 + e;
}

}  // namespace qevict
