// Device-side building blocks of the numeric contract shared by all kernels of the library:
// every binary32 value that feeds a quantizer is produced by individually rounded IEEE operations in a
// fixed order, so that integer codes do not depend on compiler contraction or on the launch shape.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace mixaq {

constexpr int WS = 7;         // window side
constexpr int WT = 49;        // tokens per window
constexpr int HEAD_DIM = 32;

struct AQ {                   // activation quantizer in kernel-friendly form
  float scale, inv_scale, zpf, qmaxf;
  int zp, bits;
};

// ---- the floating-point primitives work on two values at once (sm_100 packed binary32 arithmetic) ----------------
// __ffma2_rn / __fadd2_rn / __fmul2_rn round each lane like the scalar instruction, so every result below is
// bit-identical to the scalar function applied to .x and .y; one packed instruction takes one issue slot where two
// scalar ones take two, which is what the issue-bound epilogues need.  a - b is written fma(b, -1, a): b * -1 is
// exact, so the single rounding is that of the subtraction.
// Caution: unlike the scalar _rn intrinsics, a packed multiply whose result feeds a packed add directly has been seen
// contracted into one packed fused multiply-add (one rounding instead of two, even with --fmad=false).  Wherever the
// contract wants the product rounded before the add, an instruction must sit between the two (a clamp) or the product
// must be formed by scalar multiplies (an empty asm statement between them does not help).
__device__ __forceinline__ float2 f2(float a) { return make_float2(a, a); }
__device__ __forceinline__ float2 sub2(float2 a, float2 b) { return __ffma2_rn(b, f2(-1.0f), a); }

// 2^t by a round-to-nearest split t = n + f and a degree-5 polynomial in f (Horner, fused multiply-adds);
// n goes straight into the exponent field.  Valid for t in [-125, 127].
__device__ __forceinline__ float2 exp2_core2(float2 t) {
  const float2 r = __fadd2_rn(t, f2(12582912.0f));
  const float2 nf = __fadd2_rn(r, f2(-12582912.0f));
  const float2 f = sub2(t, nf);
  float2 p = f2(__uint_as_float(0x3aafc47du));
  p = __ffma2_rn(p, f, f2(__uint_as_float(0x3c1e883du)));
  p = __ffma2_rn(p, f, f2(__uint_as_float(0x3d635716u)));
  p = __ffma2_rn(p, f, f2(__uint_as_float(0x3e75fc83u)));
  p = __ffma2_rn(p, f, f2(__uint_as_float(0x3f317219u)));
  p = __ffma2_rn(p, f, f2(__uint_as_float(0x3f800001u)));
  return make_float2(__uint_as_float(__float_as_uint(p.x) + (__float_as_uint(r.x) << 23)),
                     __uint_as_float(__float_as_uint(p.y) + (__float_as_uint(r.y) << 23)));
}

// GELU(v) = max(v,0) - a*Phi(-a), a = min(|v|, 5); log2 Phi(-a) is a degree-7 polynomial on [0,5].
__device__ __forceinline__ float2 gelu_f2(float2 v) {
  const float2 a = make_float2(fminf(fabsf(v.x), 5.0f), fminf(fabsf(v.y), 5.0f));
  float2 q = f2(__uint_as_float(0xb5d6f9e3u));
  q = __ffma2_rn(q, a, f2(__uint_as_float(0x38729e20u)));
  q = __ffma2_rn(q, a, f2(__uint_as_float(0xba6dcc74u)));
  q = __ffma2_rn(q, a, f2(__uint_as_float(0x3c0a3aedu)));
  q = __ffma2_rn(q, a, f2(__uint_as_float(0xbd5c93e3u)));
  q = __ffma2_rn(q, a, f2(__uint_as_float(0xbeeac5d4u)));
  q = __ffma2_rn(q, a, f2(__uint_as_float(0xbf935b8fu)));
  q = __ffma2_rn(q, a, f2(__uint_as_float(0xbf7fffbeu)));
  const float2 h = __fmul2_rn(a, exp2_core2(q));
  return sub2(make_float2(fmaxf(v.x, 0.0f), fmaxf(v.y, 0.0f)), h);
}

// magic patterns of two values (see quant_magic)
__device__ __forceinline__ void quant_magic2(float2 x, float inv_scale, float lo, float hi, uint32_t& m0, uint32_t& m1) {
  float2 t = __fmul2_rn(x, f2(inv_scale));
  t = make_float2(fminf(fmaxf(t.x, lo), hi), fminf(fmaxf(t.y, lo), hi));
  t = __fadd2_rn(t, f2(12582912.0f));
  m0 = __float_as_uint(t.x); m1 = __float_as_uint(t.y);
}

// q = clamp(rne(x*inv_scale) + zp, 0, qmax), evaluated without a rounding or conversion instruction:
// rne is monotone and fixes integers, so clamping BEFORE rounding to the integer bounds [-zp, qmax-zp] gives the
// same code; adding 1.5*2^23 then rounds to nearest-even exactly (|t| <= 255) and leaves 0x4B400000 + rne(t) in
// the bit pattern.  quant_magic returns that pattern; the code is pattern - 0x4B400000 + zp.
constexpr uint32_t kMagicBits = 0x4B400000u;
__device__ __forceinline__ uint32_t quant_magic(float x, const AQ& q) {
  float t = __fmul_rn(x, q.inv_scale);
  t = fminf(fmaxf(t, -q.zpf), q.qmaxf - q.zpf);
  return __float_as_uint(__fadd_rn(t, 12582912.0f));
}
__device__ __forceinline__ uint32_t quant_code(float x, const AQ& q) {
  return quant_magic(x, q) - kMagicBits + (uint32_t)q.zp;
}
// Additive constant that turns sum_i pattern_i << (bits*i) into the packed word of the codes (the per-code
// offsets zp - 0x4B400000 are folded into one 32-bit constant; every code fits its field, so nothing carries).
__device__ __forceinline__ uint32_t pack_const(int zp, int bits) {
  // sum over the fields of k << shift = k * (sum of 2^shift) modulo 2^32
  const uint32_t k = (uint32_t)zp - kMagicBits;
  return k * (bits == 8 ? 0x01010101u : (bits == 4 ? 0x11111111u : 0x55555555u));
}
// NC (16 or 32) consecutive codes of one row, given as magic patterns, packed and stored with one or two vector
// stores (dst is NC*BITS/8-byte aligned).
template <int BITS, int NC>
__device__ __forceinline__ void store_magic(uint8_t* dst, const uint32_t (&m)[NC], uint32_t kpack) {
  constexpr int PER = 32 / BITS, WORDS = NC / PER;   // codes per word, words
  uint32_t w[WORDS];
#pragma unroll
  for (int i = 0; i < WORDS; ++i) {
    uint32_t v = kpack;
#pragma unroll
    for (int e = 0; e < PER; ++e) v += m[PER * i + e] << (BITS * e);
    w[i] = v;
  }
  if (WORDS == 8) {
    reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
    reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4 % WORDS], w[5 % WORDS], w[6 % WORDS], w[7 % WORDS]);
  } else if (WORDS == 4) {
    reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1 % WORDS], w[2 % WORDS], w[3 % WORDS]);
  } else if (WORDS == 2) {
    reinterpret_cast<uint2*>(dst)[0] = make_uint2(w[0], w[1 % WORDS]);
  } else {
    reinterpret_cast<uint32_t*>(dst)[0] = w[0];
  }
}

// Sum over a warp by the butterfly of the contract (offsets 16, 8, 4, 2, 1); every lane ends with the
// same bits because binary32 addition is commutative.
__device__ __forceinline__ float warp_sum_butterfly(float v) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) v = __fadd_rn(v, __shfl_xor_sync(0xffffffffu, v, off));
  return v;
}

// LayerNorm statistics of R rows, each held as NPL values per lane (lane l holds channels l, l+32, ...).
// The sums follow the contract (per-lane partial sums in channel order, then the butterfly); the divisions and the
// square root, which are expensive instruction sequences, run once for all R rows: lane r serves row r and the
// results are broadcast.
template <int NPL, int R>
__device__ __forceinline__ void ln_stats_rows(const float (&x)[R][NPL], float fC, float (&mean)[R], float (&rstd)[R]) {
  const int lane = threadIdx.x & 31;
  float tot = 0.0f;
#pragma unroll
  for (int r = 0; r < R; ++r) {
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < NPL; ++i) s = __fadd_rn(s, x[r][i]);
    s = warp_sum_butterfly(s);
    if (lane == r) tot = s;
  }
  const float mean_l = __fdiv_rn(tot, fC);
#pragma unroll
  for (int r = 0; r < R; ++r) mean[r] = __shfl_sync(0xffffffffu, mean_l, r);
  float vt = 0.0f;
#pragma unroll
  for (int r = 0; r < R; ++r) {
    float v = 0.0f;
#pragma unroll
    for (int i = 0; i < NPL; ++i) { float d = __fsub_rn(x[r][i], mean[r]); v = __fmaf_rn(d, d, v); }
    v = warp_sum_butterfly(v);
    if (lane == r) vt = v;
  }
  const float var_l = __fdiv_rn(vt, fC);
  const float rstd_l = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(var_l, 1e-5f)));
#pragma unroll
  for (int r = 0; r < R; ++r) rstd[r] = __shfl_sync(0xffffffffu, rstd_l, r);
}
template <int NPL>
__device__ __forceinline__ void ln_stats(const float (&x)[NPL], float fC, float& mean, float& rstd) {
  float xs[1][NPL], m[1], r[1];
#pragma unroll
  for (int i = 0; i < NPL; ++i) xs[0][i] = x[i];
  ln_stats_rows<NPL, 1>(xs, fC, m, r);
  mean = m[0]; rstd = r[0];
}

__device__ __forceinline__ float ln_apply(float x, float mean, float rstd, float g, float b) {
  return __fmaf_rn(__fmul_rn(__fsub_rn(x, mean), rstd), g, b);
}

// Store the codes of one row that a warp holds in the lane-strided layout (lane l: channels l + 32*i).
// bits = 8: one byte per code.  bits = 4 / 2: neighbouring lanes are merged into bytes, little end first.
template <int NPL>
__device__ __forceinline__ void store_codes_lane_strided(uint8_t* row, const uint32_t (&code)[NPL], int bits, int lane) {
#pragma unroll
  for (int i = 0; i < NPL; ++i) {
    uint32_t c = code[i];
    if (bits == 8) {
      row[lane + 32 * i] = (uint8_t)c;
    } else if (bits == 4) {
      uint32_t hi = __shfl_down_sync(0xffffffffu, c, 1);
      if ((lane & 1) == 0) row[(lane + 32 * i) >> 1] = (uint8_t)(c | (hi << 4));
    } else {  // 2 bits
      uint32_t c1 = __shfl_down_sync(0xffffffffu, c, 1);
      uint32_t c2 = __shfl_down_sync(0xffffffffu, c, 2);
      uint32_t c3 = __shfl_down_sync(0xffffffffu, c, 3);
      if ((lane & 3) == 0) row[(lane + 32 * i) >> 2] = (uint8_t)(c | (c1 << 2) | (c2 << 4) | (c3 << 6));
    }
  }
}

// Eight 4-bit codes of one word -> eight bytes (two words), little end first: mask the even and the odd nibbles
// into byte lanes, then interleave them with two byte permutes.
__device__ __forceinline__ void expand_nibbles(uint32_t v, uint32_t& lo, uint32_t& hi) {
  const uint32_t x = v & 0x0F0F0F0Fu;            // codes 0, 2, 4, 6
  const uint32_t y = (v >> 4) & 0x0F0F0F0Fu;     // codes 1, 3, 5, 7
  lo = __byte_perm(x, y, 0x5140);                // x0 y0 x1 y1
  hi = __byte_perm(x, y, 0x7362);                // x2 y2 x3 y3
}
// Eight 2-bit codes in the low half of v -> eight nibbles (bit spread in three shift-or-mask steps).
__device__ __forceinline__ uint32_t spread_pairs(uint32_t t) {
  t = (t | (t << 8)) & 0x00FF00FFu;
  t = (t | (t << 4)) & 0x0F0F0F0Fu;
  t = (t | (t << 2)) & 0x33333333u;
  return t;
}

// Unpack 32 consecutive codes (one k-group) from packed storage (global or shared) into 32 bytes (eight words).
__device__ __forceinline__ void load_codes_32(const uint8_t* src, int bits, uint32_t (&w)[8]) {
  if (bits == 8) {
    uint4 a = reinterpret_cast<const uint4*>(src)[0], b = reinterpret_cast<const uint4*>(src)[1];
    w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
  } else if (bits == 4) {
    uint4 a = reinterpret_cast<const uint4*>(src)[0];
    expand_nibbles(a.x, w[0], w[1]);
    expand_nibbles(a.y, w[2], w[3]);
    expand_nibbles(a.z, w[4], w[5]);
    expand_nibbles(a.w, w[6], w[7]);
  } else {
    uint2 a = reinterpret_cast<const uint2*>(src)[0];
    expand_nibbles(spread_pairs(a.x & 0xFFFFu), w[0], w[1]);
    expand_nibbles(spread_pairs(a.x >> 16), w[2], w[3]);
    expand_nibbles(spread_pairs(a.y & 0xFFFFu), w[4], w[5]);
    expand_nibbles(spread_pairs(a.y >> 16), w[6], w[7]);
  }
}

}  // namespace mixaq
