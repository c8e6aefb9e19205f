// Device-side building blocks of the quantized-Adam step kernels (sm_100a).
//
// Arithmetic contract: every floating-point step of the method is one IEEE-754
// binary32 operation with round-to-nearest-even, written with the explicit
// __f*_rn intrinsics so that the compiler can neither contract a multiply and an
// add into an FMA nor substitute an approximate division or square root.
// Subnormals are kept (the library is built without flush-to-zero).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace qadam {

constexpr int kAlign = 128;        // elements: segment starts, tile starts and tile lengths are multiples
constexpr int kThreads = 256;      // threads per CTA in every kernel
constexpr int kRows = 4;           // float4 rows per thread and tile
constexpr int kRowElems = kThreads * 4;          // 1024 elements per CTA-wide row
constexpr int kTileElems = kRows * kRowElems;    // 4096 elements per tile

// A tile is a run of at most kTileElems padded elements inside one segment.
struct __align__(16) Tile {
  long long off;   // first element (padded layout), multiple of kAlign
  int count;       // elements, multiple of kAlign
  int seg;         // segment the run belongs to
};

// How a level index is decided and what a level is worth (Section 5.1's set G).
enum GMode : int {
  G_TERNARY = 0,   // {0, 1}                     (kg = 0, either grid)
  G_FIVE = 1,      // {0, 1/2, 1}                (kg = 1, either grid)
  G_POW2 = 2,      // {0, 2^-k, ..., 1}          (kg >= 2, geometric)
  G_UNIFORM = 3,   // {0, 1/2^k, 2/2^k, ..., 1}  (kg >= 2, uniform)
  G_IDENTITY = 4,  // Q_g = identity
  G_STOCHASTIC = 5 // {0, 1} chosen at random with probability |u| / |u|_inf (worker side only:
                   // the codes it emits are ternary codes and are decoded as such)
};

struct Hyper {
  float beta, theta, eps;
  float one_minus_beta, one_minus_theta;   // fl(1 - beta), fl(1 - theta), rounded once on the host
};

__device__ __forceinline__ float exp2i(int e) {          // 2^e, -126 <= e <= 127
  return __int_as_float((e + 127) << 23);
}

// v_t = theta v + (1-theta) g^2 ;  m_t = beta m + (1-beta) g      (Algorithm 1 / 3)
__device__ __forceinline__ void moments(const Hyper& h, float g, float& m, float& v) {
  const float gg = __fmul_rn(g, g);
  v = __fadd_rn(__fmul_rn(h.theta, v), __fmul_rn(h.one_minus_theta, gg));
  m = __fadd_rn(__fmul_rn(h.beta, m), __fmul_rn(h.one_minus_beta, g));
}

// alpha_t m / sqrt(v + eps)      (epsilon inside the root, no bias correction)
// A zero numerator is frequent (a coordinate whose decoded updates have all been
// level 0 keeps m = 0 exactly) and would send the IEEE division down its slow
// special-case path; +-0 / den = +-0 for the positive den here, so the numerator is
// returned as it is and the divider is fed a harmless 1 in its place.
__device__ __forceinline__ float adam_step(const Hyper& h, float m, float v, float alpha) {
  const float num = __fmul_rn(alpha, m);
  const float den = __fsqrt_rn(__fadd_rn(v, h.eps));
  const bool zero = num == 0.0f;
  const float q = __fdiv_rn(zero ? 1.0f : num, den);
  return zero ? num : q;
}

// Index (0..L) of the level of G nearest to y = |u| / |u|_inf: the number of
// midpoints between neighbouring levels that lie strictly below y, so a tie goes
// to the level nearer zero.  y may be NaN (0/0 for an all-zero segment): every
// comparison is then false and the index is 0.
template <int MODE>
__device__ __forceinline__ int level_index(float y, int k, int L) {
  if constexpr (MODE == G_TERNARY) {
    return y > 0.5f ? 1 : 0;
  } else if constexpr (MODE == G_FIVE) {
    return (y > 0.25f ? 1 : 0) + (y > 0.75f ? 1 : 0);
  } else if constexpr (MODE == G_POW2) {
    // levels 0, 2^-k, 2^(1-k), ..., 1: midpoints 2^(-k-1), then 3*2^(c-3-k), c = 2..L
    float t = exp2i(-k - 1);
    int c = y > t ? 1 : 0;
    t = __fmul_rn(3.0f, t);
    for (int cc = 2; cc <= L; ++cc) {
      c += y > t ? 1 : 0;
      t = __fmul_rn(t, 2.0f);
    }
    return c;
  } else {
    // levels c / 2^k: midpoints (c - 1/2) / 2^k.  With z = y 2^k (exact) the count
    // of c' >= 1 with z > c' - 1/2 is ceil(z - 1/2), and z - 1/2 is exact wherever
    // its rounding could matter (z >= 1/4).
    const float z = __fmul_rn(y, exp2i(k));
    int c = (int)ceilf(__fadd_rn(z, -0.5f));
    c = c < 0 ? 0 : c;
    return c > L ? L : c;
  }
}

// Magnitude of level c of G (exactly representable).
template <int MODE>
__device__ __forceinline__ float level_value(int c, int k) {
  if constexpr (MODE == G_TERNARY) {
    return c ? 1.0f : 0.0f;
  } else if constexpr (MODE == G_FIVE) {
    return 0.5f * (float)c;
  } else if constexpr (MODE == G_POW2) {
    return c ? exp2i(c - 1 - k) : 0.0f;
  } else {
    return __fmul_rn((float)c, exp2i(-k));
  }
}

// What Q_g needs of a segment's scale s = |u|_inf, computed once per tile rather than per
// coordinate.  The level of a coordinate is decided by y = fl(|u| / s) against the midpoints
// of G; the fast paths below settle that decision without dividing for all but a sliver of
// values and fall back to the division inside the sliver, so the result is always the one
// the division gives.
struct GradScale {
  float s;
  float inv;      // fl(1 / s), times 2^k for the uniform grid
  float half;     // ternary: s / 2 (exact) and the upper end of the sliver above it
  float half_hi;
  bool fast;      // s is an ordinary number (not zero, tiny, Inf or NaN): the fast paths apply
};
template <int MODE>
__device__ __forceinline__ GradScale grad_scale(float s, int k) {
  GradScale g;
  g.s = s;
  g.fast = s >= 1e-30f && s < 3.0e38f;
  g.half = __fmul_rn(0.5f, s);
  g.half_hi = __fmul_rn(g.half, 1.000000476837158203125f);          // 1 + 2^-21
  g.inv = 0.0f;
  if constexpr (MODE == G_FIVE || MODE == G_POW2 || MODE == G_UNIFORM) {
    if (g.fast) {
      g.inv = __fdiv_rn(1.0f, s);
      if constexpr (MODE == G_UNIFORM) g.inv = __fmul_rn(g.inv, exp2i(k));      // exact
    }
  }
  return g;
}

// One coordinate of Q_g and of the error update:  given u and the segment's scale
// s = |u|_inf, returns the code (level index + L) and writes e' = u - Q_g(u).
template <int MODE>
__device__ __forceinline__ unsigned quantize_grad(float u, const GradScale& gs, int k, int L, float& e_next) {
  const float s = gs.s;
  const float a = fabsf(u);
  const bool neg = u < 0.0f;
  if constexpr (MODE == G_TERNARY) {
    // The decision is y = fl(|u| / s) > 1/2.  |u| <= s/2 gives a quotient <= 1/2 (s/2 is exact
    // for a normal s), and |u| > (s/2)(1 + 2^-21) gives a quotient whose rounding stays above
    // 1/2.  Only values inside that band, and tiny or non-finite scales, take the division.
    bool one;
    if (a <= gs.half && gs.fast) {
      one = false;
    } else if (a > gs.half_hi && gs.fast) {
      one = true;
    } else {
      one = __fdiv_rn(a, s) > 0.5f;
    }
    const float deq = one ? (neg ? -s : s) : 0.0f;
    e_next = __fsub_rn(u, deq);
    return one ? (neg ? 0u : 2u) : 1u;
  }
  int c;
  bool decided = false;
  if constexpr (MODE == G_FIVE || MODE == G_POW2) {
    // Geometric levels 0, 2^-k, ..., 1: the midpoints are 2^(-k-1) and 1.5 * 2^j, so the level
    // index is read off the exponent of y and of whether its fraction reaches 1.5.
    // y' = fl(|u| * fl(1/s)) is within 2^-22 (relative) of y; unless y' lies within 2^-19 of a
    // midpoint (fraction near 1 or near 1.5) both give the same index.
    const int kk = MODE == G_FIVE ? 1 : k;
    if (gs.fast) {
      const float yp = __fmul_rn(a, gs.inv);
      const unsigned yb = __float_as_uint(yp);
      const unsigned m = yb & 0x7fffffu;
      const bool near = (m - 0x3ffff0u) <= 0x20u || m <= 0x10u || m >= 0x7fffefu;
      if (!near) {
        const int e15 = (int)((yb + 0x00400000u) >> 23) - 127;      // exponent, plus one when the fraction is >= 1.5
        const int upper = e15 + kk;
        c = (yp > exp2i(-kk - 1) ? 1 : 0) + (upper > 0 ? upper : 0);
        c = c > L ? L : c;
        decided = true;
      }
    }
  } else if constexpr (MODE == G_UNIFORM) {
    // Uniform levels c / 2^k: the index is ceil(z - 1/2) with z = y 2^k.  z' = |u| * fl(2^k / s)
    // is within 2^-22 (relative) of z; unless z' - 1/2 lies within 2^-15 of an integer (z <= 64)
    // both give the same index.
    if (gs.fast) {
      const float t = __fadd_rn(__fmul_rn(a, gs.inv), -0.5f);
      const float ct = ceilf(t);
      const float w = __fsub_rn(ct, t);                              // in [0, 1)
      if (w > 6.1035156e-05f && w < 0.99993896f) {
        c = (int)ct;
        c = c < 0 ? 0 : (c > L ? L : c);
        decided = true;
      }
    }
  }
  if (!decided) {
    const float y = __fdiv_rn(a, s);
    c = level_index<MODE>(y, k, L);
  }
  float deq = 0.0f;                                   // level 0 carries no sign
  if (c != 0) {
    const float mag = __fmul_rn(s, level_value<MODE>(c, k));
    deq = neg ? -mag : mag;
  }
  e_next = __fsub_rn(u, deq);
  return (unsigned)(neg ? L - c : L + c);
}

// A lane's 4 two-bit codes, given as one byte, stored as part of its warp's row of 128 codes
// (32 bytes): two shuffle steps gather four lanes' bytes into a word, which lanes 0, 4, ..., 28
// store.  Every lane of the warp must call this.  row_dst: address of the row's first code.
__device__ __forceinline__ void store_row_of_code_bytes(unsigned byte, void* row_dst, int lane) {
  unsigned w = byte | (__shfl_down_sync(0xffffffffu, byte, 1) << 8);
  w |= __shfl_down_sync(0xffffffffu, w, 2) << 16;
  if ((lane & 3) == 0) reinterpret_cast<unsigned*>(row_dst)[lane >> 2] = w;
}

// sat(d * 2^127): 1 for every positive d >= 2^-127 (every positive float difference the callers
// form), 0 for zero, negative values and NaN.  One instruction on the fp32 pipe in place of a
// comparison and a select on the integer pipe.
__device__ __forceinline__ float positive_as_one(float d) {
  float r;
  asm("mul.rn.sat.f32 %0, %1, 0f7F000000;" : "=f"(r) : "f"(d));
  return r;
}

// Ternary Q_g of 4 consecutive coordinates of one lane, the error update, and the lane's byte of
// packed codes (code = level index + 1, coordinate c in bits 2c, 2c + 1).  Same decisions as
// quantize_grad<G_TERNARY>: level 1 iff fl(|u| / s) > 1/2, settled without dividing outside the
// sliver (s/2, (s/2)(1 + 2^-21)], by the division inside it and for scales that are not ordinary
// numbers.  Outside the sliver everything runs on the fp32 pipe (the integer pipe, at half its
// rate, is what the quantize kernels are otherwise bound by): [|u| > t] is sat((|u| - t) 2^127),
// exact because the difference of two nearby floats is exact and at least 2^-125 for the scales
// that take this path; the codes are gathered by exact multiply-adds and read out of a mantissa.
__device__ __forceinline__ unsigned quantize_ternary4(const float (&u)[4], const GradScale& gs, float (&e_next)[4]) {
  const float s = gs.s;
  float up[4];
  if (gs.fast) {
    float band = 0.0f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float a = fabsf(u[c]);
      up[c] = positive_as_one(__fsub_rn(a, gs.half_hi));
      band = __fadd_rn(band, __fsub_rn(positive_as_one(__fsub_rn(a, gs.half)), up[c]));
    }
    if (band != 0.0f) {                       // some |u| lies inside the sliver: the division decides
#pragma unroll
      for (int c = 0; c < 4; ++c) up[c] = __fdiv_rn(fabsf(u[c]), s) > 0.5f ? 1.0f : 0.0f;
    }
  } else {
#pragma unroll
    for (int c = 0; c < 4; ++c) up[c] = __fdiv_rn(fabsf(u[c]), s) > 0.5f ? 1.0f : 0.0f;
  }
  float cf[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const float sign1 = __uint_as_float((__float_as_uint(u[c]) & 0x80000000u) | 0x3f800000u);   // +-1 with u's sign
    // up * (+-s) + (+0): +-s for level +-1 and +0 (never -0) for level 0, as the definition has it
    const float deq = __fmaf_rn(up[c], __fmul_rn(sign1, s), 0.0f);
    e_next[c] = __fsub_rn(u[c], deq);
    cf[c] = __fmaf_rn(up[c], sign1, 1.0f);                                                     // 0, 1 or 2
  }
  const float packed = __fmaf_rn(__fmaf_rn(__fmaf_rn(cf[3], 4.0f, cf[2]), 4.0f, cf[1]), 4.0f, cf[0]);
  return __float_as_uint(__fadd_rn(packed, 8388608.0f)) & 0xffu;
}

// Five-level Q_g (levels 0, 1/2, 1 times the scale, k_g = 1 of the geometric grid) of 4
// consecutive coordinates of one lane, the error update, and the lane's 12 bits of packed codes
// (code = level index + 2, coordinate c in bits 3c .. 3c + 2).  Same decisions as
// quantize_grad<G_FIVE>: index [y > 1/4] + [y > 3/4] with y = fl(|u| / s).  y' = fl(|u| fl(1/s)) is
// within 2^-22 (relative) of y, so y' above t (1 + 2^-20) or at most t (1 - 2^-20) settles the
// comparison with the midpoint t; a y' in between sends the lane's four coordinates to the
// division.  As in quantize_ternary4 the comparisons are saturated differences on the fp32 pipe
// (a positive difference of y' and a threshold is at least 2^-26), the dequantized value is
// index * (+-s/2), exact, and the codes are gathered by exact multiply-adds.
__device__ __forceinline__ unsigned quantize_five4(const float (&u)[4], const GradScale& gs, float (&e_next)[4]) {
  const float s = gs.s;
  float idx[4];                                // level index 0, 1 or 2 as a float
  bool divide = !gs.fast;
  if (gs.fast) {
    float band = 0.0f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float yp = __fmul_rn(fabsf(u[c]), gs.inv);
      const float up1 = positive_as_one(__fsub_rn(yp, 0.25000023841857910156f));     // 1/4 (1 + 2^-20)
      const float lo1 = positive_as_one(__fsub_rn(yp, 0.24999976158142089844f));     // 1/4 (1 - 2^-20)
      const float up3 = positive_as_one(__fsub_rn(yp, 0.75000071525573730469f));     // 3/4 (1 + 2^-20)
      const float lo3 = positive_as_one(__fsub_rn(yp, 0.74999928474426269531f));     // 3/4 (1 - 2^-20)
      idx[c] = __fadd_rn(up1, up3);
      band = __fadd_rn(band, __fadd_rn(__fsub_rn(lo1, up1), __fsub_rn(lo3, up3)));
    }
    divide = band != 0.0f;
  }
  if (divide) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float y = __fdiv_rn(fabsf(u[c]), s);
      idx[c] = (y > 0.25f ? 1.0f : 0.0f) + (y > 0.75f ? 1.0f : 0.0f);
    }
  }
  float cf[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const float sign1 = __uint_as_float((__float_as_uint(u[c]) & 0x80000000u) | 0x3f800000u);   // +-1 with u's sign
    // index * (+-s/2) + (+0): the level's value (s/2 and s are exact) and +0, never -0, for level 0.
    // A scale so small that s/2 is not exact takes fl(s * level) as the definition has it.
    const float deq = gs.fast ? __fmaf_rn(idx[c], __fmul_rn(sign1, gs.half), 0.0f)
                              : (idx[c] == 0.0f ? 0.0f : __fmul_rn(__fmul_rn(s, __fmul_rn(0.5f, idx[c])), sign1));
    e_next[c] = __fsub_rn(u[c], deq);
    cf[c] = __fmaf_rn(idx[c], sign1, 2.0f);                                                     // 0 .. 4
  }
  const float packed = __fmaf_rn(__fmaf_rn(__fmaf_rn(cf[3], 8.0f, cf[2]), 8.0f, cf[1]), 8.0f, cf[0]);
  return __float_as_uint(__fadd_rn(packed, 8388608.0f)) & 0xfffu;
}

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3",
// SC 2011), from its published definition: ten rounds over a counter of four 32-bit words
// under a key of two; a round multiplies words 0 and 2 by fixed odd constants, keeps both
// halves of the products and mixes in the other words and the key; the key words grow by two
// Weyl constants after every round.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const unsigned hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const unsigned hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

// One coordinate of the stochastic ternary operator (the method Section 5.1 compares with):
// level 1 with probability y = fl(|u| / s), decided by r < y with r the top 24 bits of the
// coordinate's random word times 2^-24; returns the code and writes e' = u - Q(u).
__device__ __forceinline__ unsigned quantize_grad_stochastic(float u, float s, unsigned word, float& e_next) {
  bool one = false;
  if (s > 0.0f) {
    const float r = __fmul_rn((float)(word >> 8), 5.9604644775390625e-08f);    // exact
    one = r < __fdiv_rn(fabsf(u), s);
  }
  const bool neg = u < 0.0f;
  const float deq = one ? (neg ? -s : s) : 0.0f;
  e_next = __fsub_rn(u, deq);
  return one ? (neg ? 0u : 2u) : 1u;
}

// One coordinate of Q_x (Section 5.1): nearest point of the grid c / 2^(kx+1),
// |c| <= 2^kx, ties toward zero, clipped.  Returns the code c + 2^kx; xq is Q_x(x).
__device__ __forceinline__ unsigned quantize_weight(float x, int kx, float& xq) {
  if (kx == 0) {
    // grid {-1/2, 0, 1/2}: the single midpoint is 1/4 (z = 2|x| > 1/2), ties toward zero
    const bool far = fabsf(x) > 0.25f;
    const bool neg = x < 0.0f;
    xq = far ? (neg ? -0.5f : 0.5f) : 0.0f;
    return far ? (neg ? 0u : 2u) : 1u;
  }
  const int L = 1 << kx;
  float z = __fmul_rn(fabsf(x), exp2i(kx + 1));        // exact
  z = fminf(z, (float)L);
  int c = (int)ceilf(__fadd_rn(z, -0.5f));
  c = c < 0 ? 0 : c;
  const bool neg = x < 0.0f;
  xq = 0.0f;
  if (c != 0) {
    const float mag = __fmul_rn((float)c, exp2i(-(kx + 1)));   // exact
    xq = neg ? -mag : mag;
  }
  return (unsigned)(neg ? L - c : L + c);
}

// ---------------------------------------------------------------------------
// Packing one warp-row: 32 lanes x 4 consecutive elements = 128 codes of B bits,
// i.e. 4*B 32-bit words of the little-endian bit stream, written by lanes
// 0..4B-1 as one coalesced store.  Every lane of the warp must call this.
// row_dst: address of the row's first code (the row starts on a multiple of 128
// elements, so it is 16*B-byte aligned).
// ---------------------------------------------------------------------------
__host__ __device__ constexpr int cgcd(int a, int b) { return b == 0 ? a : cgcd(b, a % b); }

// The same for code widths up to 8 bits with the lane's four codes already gathered into one
// field of 4 * B bits.
template <int B>
__device__ __forceinline__ void pack_row_store_fields(unsigned field, void* row_dst, int lane) {
  static_assert(B >= 2 && B <= 8, "code width");
  constexpr int F = 4 * B;                               // 8..32 bits per lane
  constexpr int G = cgcd(32, F);
  constexpr int J = (F - G + 32 + F - 1) / F;            // fields a 32-bit word can touch
  const int bit0 = 32 * lane;
  const int l0 = bit0 / F;
  const int sh = bit0 - l0 * F;
  unsigned long long acc = 0;
#pragma unroll
  for (int j = 0; j < J; ++j) {
    const int src = l0 + j > 31 ? 31 : l0 + j;
    const unsigned f = __shfl_sync(0xffffffffu, field, src);
    acc |= (unsigned long long)f << (j * F);
  }
  if (lane < F) reinterpret_cast<unsigned*>(row_dst)[lane] = (unsigned)(acc >> sh);
}

template <int B>
__device__ __forceinline__ void pack_row_store(unsigned c0, unsigned c1, unsigned c2, unsigned c3,
                                               void* row_dst, int lane) {
  static_assert(B >= 2 && B <= 16, "code width");
  if constexpr (B == 16) {
    reinterpret_cast<uint2*>(row_dst)[lane] = make_uint2(c0 | (c1 << 16), c2 | (c3 << 16));
  } else if constexpr (B > 8) {
    // 4*B bits per lane (36..60): gather through shared-memory-free 64-bit shuffles
    constexpr int F = 4 * B;                               // field width per lane
    const unsigned long long field = (unsigned long long)c0 | ((unsigned long long)c1 << B) |
                                     ((unsigned long long)c2 << (2 * B)) |
                                     ((unsigned long long)c3 << (3 * B));
    // words per row = F (<= 60): each lane produces up to two words
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int w = lane + 32 * half;
      const int bit0 = 32 * w;
      const int l0 = bit0 / F;
      const int sh = bit0 - l0 * F;                        // < F
      const unsigned long long f0 = __shfl_sync(0xffffffffu, field, l0 > 31 ? 31 : l0);
      const unsigned long long f1 = __shfl_sync(0xffffffffu, field, l0 + 1 > 31 ? 31 : l0 + 1);
      // bits [sh, sh+32) of the F-bit f0 followed by f1
      unsigned long long lo = f0 >> sh;
      const int have = F - sh;                             // bits contributed by f0 (>= 1)
      if (have < 32) lo |= f1 << have;
      if (w < F) reinterpret_cast<unsigned*>(row_dst)[w] = (unsigned)lo;
    }
  } else {
    pack_row_store_fields<B>(c0 | (c1 << B) | (c2 << (2 * B)) | (c3 << (3 * B)), row_dst, lane);
  }
}

// Dispatch on a run-time width.
__device__ __forceinline__ void pack_row_store_rt(int bits, unsigned c0, unsigned c1, unsigned c2,
                                                  unsigned c3, void* row_dst, int lane) {
  switch (bits) {
    case 2: pack_row_store<2>(c0, c1, c2, c3, row_dst, lane); break;
    case 3: pack_row_store<3>(c0, c1, c2, c3, row_dst, lane); break;
    case 4: pack_row_store<4>(c0, c1, c2, c3, row_dst, lane); break;
    case 5: pack_row_store<5>(c0, c1, c2, c3, row_dst, lane); break;
    case 6: pack_row_store<6>(c0, c1, c2, c3, row_dst, lane); break;
    case 7: pack_row_store<7>(c0, c1, c2, c3, row_dst, lane); break;
    case 8: pack_row_store<8>(c0, c1, c2, c3, row_dst, lane); break;
    case 9: pack_row_store<9>(c0, c1, c2, c3, row_dst, lane); break;
    case 10: pack_row_store<10>(c0, c1, c2, c3, row_dst, lane); break;
    case 11: pack_row_store<11>(c0, c1, c2, c3, row_dst, lane); break;
    case 12: pack_row_store<12>(c0, c1, c2, c3, row_dst, lane); break;
    case 13: pack_row_store<13>(c0, c1, c2, c3, row_dst, lane); break;
    case 14: pack_row_store<14>(c0, c1, c2, c3, row_dst, lane); break;
    case 15: pack_row_store<15>(c0, c1, c2, c3, row_dst, lane); break;
    default: pack_row_store<16>(c0, c1, c2, c3, row_dst, lane); break;
  }
}

// The 4*bits-bit field of this lane (its 4 consecutive codes) out of a packed
// warp-row; bits <= 8.  row_src: address of the row's first code.
__device__ __forceinline__ unsigned unpack_row_field(const void* row_src, int bits, int lane) {
  const int F = 4 * bits;
  const unsigned* words = reinterpret_cast<const unsigned*>(row_src);
  const int bit = F * lane;
  const int w = bit >> 5;
  const unsigned lo = __ldg(words + w);
  const unsigned hi = __ldg(words + (w + 1 < F ? w + 1 : w));
  const unsigned v = __funnelshift_r(lo, hi, bit & 31);
  return F == 32 ? v : (v & ((1u << F) - 1u));
}

// Packed binary32 arithmetic (two independent lanes per instruction, sm_100).
// Each lane rounds exactly like the scalar operation.  Caution: unlike the scalar
// forms, a packed multiply whose result feeds a packed add IS fused into a packed
// fused multiply-add by the assembler, explicit rounding mode or not (measured on
// sm_100a, CUDA 12.9): never feed mul2_rn into add2_rn where both roundings matter.
__device__ __forceinline__ unsigned long long pack_f2(float2 a) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a.x), "f"(a.y));
  return r;
}
__device__ __forceinline__ float2 unpack_f2(unsigned long long r) {
  float2 a;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a.x), "=f"(a.y) : "l"(r));
  return a;
}
__device__ __forceinline__ float2 add2_rn(float2 a, float2 b) {
  unsigned long long r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(pack_f2(a)), "l"(pack_f2(b)));
  return unpack_f2(r);
}
__device__ __forceinline__ float2 mul2_rn(float2 a, float2 b) {
  unsigned long long r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(pack_f2(a)), "l"(pack_f2(b)));
  return unpack_f2(r);
}
__device__ __forceinline__ float2 fma2_rn(float2 a, float2 b, float2 c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(pack_f2(a)), "l"(pack_f2(b)), "l"(pack_f2(c)));
  return unpack_f2(r);
}

__device__ __forceinline__ unsigned warp_max(unsigned v) {
  return __reduce_max_sync(0xffffffffu, v);
}

}  // namespace qadam
