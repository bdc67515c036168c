// Fused window attention of one branch batch (MixA-Q Section 3.1: multi-head self-attention inside each
// non-overlapping 7x7 window; Figure 2a "Attn High" / "Attn Low"):
//   S_int = (q - z_q)(k - z_k)^T  (int32)  ->  S = fma(S_int, s_q*s_k/sqrt(d), relpos_bias) [+ shift mask]
//   P = softmax_row(S) in binary32  ->  P codes (unsigned, step 1/(2^b-1))
//   O_int = P_codes (v - z_v) (int32)  ->  O = O_int * s_p*s_v  ->  codes of the proj input quantizer.
//
// One CTA of four warps per (window slot, head): the warps stage q, k and v together, then warp i owns query rows
// 16i .. 16i+15.  Both products run on the integer tensor cores of the warp
// (mma.sync m16n8k32, u8 x u8 -> s32; 49 tokens padded to 64 query rows x 56 key columns).  The 49 x 32 problem is
// far too small for a 128-row tcgen05 tile and is bound by the softmax arithmetic, not by the MMA rate.
// The softmax runs on the accumulator fragments: a quad of lanes holds one row, lane t of the quad owns columns
// 8g+2t, 8g+2t+1 -- exactly the four interleaved partial sums of the numeric contract.  The P codes go from
// accumulator layout to A-operand layout without leaving the thread: the key index of P.V is permuted
// consistently on both operands (V^T is staged in shared memory with its columns in that order).
#include "kernels.h"

namespace mixaq {

namespace {

constexpr int ATT_WARPS = 4;
constexpr int QK_LD = 12;     // words per staged q / k row (8 used; 12 keeps fragment reads conflict-free)
constexpr int VT_LD = 20;     // words per row of V^T (16 used)

struct WarpSmem {
  uint32_t q[64][QK_LD];      // query rows (one code per byte), rows >= 49 zero
  uint32_t k[56][QK_LD];      // key rows
  uint32_t vt[32][VT_LD];     // V^T: row e, 64 key positions in the permuted order of pos()
  int rq[64];                 // per query row:  -z_k * sum_d q + 32 z_q z_k
  int ck[56];                 // per key column: -z_q * sum_d k
  uint32_t o[4][16][8];       // per warp: staging of 16 output rows x 32 codes (one per byte)
  uint8_t reg[64];            // shift region of every token
};

__device__ __forceinline__ int dp4a_uu(uint32_t a, uint32_t b, int c) {
  int d;
  asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

__device__ __forceinline__ void mma_u8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ int shift_region(int pos, int L, int shift) {
  return pos < L - WS ? 0 : (pos < L - shift ? 1 : 2);
}

// Position of key j inside V^T rows: within each group of 32 keys, the MMA's k index 4t+u (u = 0..3) of lane t
// holds the P code of accumulator tile 2*0+(u>>1), column 2t+(u&1); k index 16+4t+u that of tiles 2, 3.
__device__ __forceinline__ int pos(int j) {
  const int jj = j & 31, nt = jj >> 3, c = jj & 7, t = c >> 1, u0 = c & 1;
  const int kappa = nt < 2 ? 4 * t + 2 * nt + u0 : 16 + 4 * t + 2 * (nt - 2) + u0;
  return (j & 32) + kappa;
}

// pack eight bytes (two words) into eight nibbles, little end first
__device__ __forceinline__ uint32_t pack_nibbles(uint32_t lo, uint32_t hi) {
  const uint32_t x = __byte_perm(lo, hi, 0x6420);   // codes 0, 2, 4, 6
  const uint32_t y = __byte_perm(lo, hi, 0x7531);   // codes 1, 3, 5, 7
  return x | (y << 4);
}
// eight nibbles -> eight 2-bit codes in the low half
__device__ __forceinline__ uint32_t squeeze_pairs(uint32_t t) {
  t = (t | (t >> 2)) & 0x0F0F0F0Fu;
  t = (t | (t >> 4)) & 0x00FF00FFu;
  t = (t | (t >> 8)) & 0x0000FFFFu;
  return t;
}

// TAPS: the debug taps (softmax output, P codes, P.V accumulators) are compiled in only for calls that ask for them
template <bool SHIFTED, bool TAPS>
__global__ void __launch_bounds__(ATT_WARPS * 32, 8) k_attention(AttnArgs a) {
  __shared__ __align__(16) WarpSmem sm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int slots_hi = a.br[0].slots;
  const long wg = (long)blockIdx.x;
  int slot = (int)(wg / a.heads);
  const int h = (int)(wg - (long)slot * a.heads);
  const bool is_hi = slot < slots_hi;
  const AttnBranch& br = is_hi ? a.br[0] : a.br[1];
  if (!is_hi) slot -= slots_hi;
  const int bits = br.bits, cbits = br.cbits, C = a.C;     // range of a code, bits it occupies in memory
  const long row_bytes = (long)3 * C * cbits / 8;
  const int zq = br.q.zp, zk = br.k.zp, zv = br.v.zp;

  // ---- stage q, k (rows) and v (transposed, permuted) of this head, one code per byte: 3 x 64 row items ----
  int wy = 0, wx = 0;
  if (SHIFTED) { const int w = br.win[slot]; wy = w / a.nwx; wx = w - wy * a.nwx; }
  for (int item = threadIdx.x; item < 3 * 64; item += ATT_WARPS * 32) {
    const int sec = item >> 6, r = item & 63;
    const uint8_t* src = br.qkv + ((long)slot * WT + r) * row_bytes + (long)(sec * C + h * HEAD_DIM) * cbits / 8;
    uint32_t w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (r < WT) load_codes_32(src, cbits, w);
    if (sec < 2) {
      int s = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) s = dp4a_uu(w[e], 0x01010101u, s);
      if (sec == 0) {
        *reinterpret_cast<uint4*>(&sm.q[r][0]) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(&sm.q[r][4]) = make_uint4(w[4], w[5], w[6], w[7]);
        sm.rq[r] = r < WT ? -zk * s + HEAD_DIM * zq * zk : 0;
        int reg = 0;
        if (SHIFTED && r < WT) {
          const int i = r / WS, j = r - i * WS;
          reg = shift_region(wy * WS + i, a.Hp, a.shift) * 3 + shift_region(wx * WS + j, a.Wp, a.shift);
        }
        sm.reg[r] = (uint8_t)reg;
      } else if (r < 56) {
        *reinterpret_cast<uint4*>(&sm.k[r][0]) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(&sm.k[r][4]) = make_uint4(w[4], w[5], w[6], w[7]);
        sm.ck[r] = -zq * s;
      }
    } else {
      uint8_t* vtb = reinterpret_cast<uint8_t*>(&sm.vt[0][0]);
      const int p = pos(r);
#pragma unroll
      for (int e = 0; e < 32; ++e) vtb[e * (VT_LD * 4) + p] = (uint8_t)(w[e >> 2] >> (8 * (e & 3)));
    }
  }
  __syncthreads();

  // ---- key fragments, per-column terms and regions of this lane's 14 columns (fixed over the query tiles) ----
  uint32_t kb0[7], kb1[7];
  int ckj[7][2];
  uint32_t regj_lo = 0, regj_hi = 0;          // 4 bits per column: columns of tiles 0..3 in lo, 4..6 in hi
#pragma unroll
  for (int nt = 0; nt < 7; ++nt) {
    kb0[nt] = sm.k[8 * nt + g][t];
    kb1[nt] = sm.k[8 * nt + g][4 + t];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int j = 8 * nt + 2 * t + u;
      ckj[nt][u] = sm.ck[j];
      if (SHIFTED) {
        const uint32_t rj = sm.reg[j];
        if (nt < 4) regj_lo |= rj << (4 * (2 * nt + u)); else regj_hi |= rj << (4 * (2 * (nt - 4) + u));
      }
    }
  }
  const float alpha = br.alpha, so = br.so;
  const int pmax = (1 << bits) - 1;
  const float pmaxf = (float)pmax;
  const AQ oq = br.o;
  const float kLog2e = 1.44269504088896340736f;
  const float4* relf = reinterpret_cast<const float4*>(a.relbias) + (long)h * (4 * 7 * 32) + lane;
  const long m_base = (long)slot * WT;
  const long out_row_bytes = (long)C * cbits / 8;

  {
    const int mt = warp;
    // ---- S = Q K^T for 16 query rows ----
    uint32_t qa[4];
    qa[0] = sm.q[16 * mt + g][t];     qa[1] = sm.q[16 * mt + g + 8][t];
    qa[2] = sm.q[16 * mt + g][4 + t]; qa[3] = sm.q[16 * mt + g + 8][4 + t];
    int c[7][4];
#pragma unroll
    for (int nt = 0; nt < 7; ++nt) {
      c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0;
      mma_u8(c[nt], qa, kb0[nt], kb1[nt]);
    }
    const int nrows = mt < 3 ? 2 : 1;           // rows 56..63 do not exist: skip the upper half of the last tile
    uint32_t pa[2][4];                          // P codes as A fragments of the two 32-key steps
    int psum[2] = {0, 0};
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) { pa[ks][0] = pa[ks][1] = pa[ks][2] = pa[ks][3] = 0; }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      if (r < nrows) {
        const int i = 16 * mt + g + 8 * r;
        const int rqi = sm.rq[i];
        uint32_t xlo = 0, xhi = 0;
        if (SHIFTED) { const uint32_t ri = sm.reg[i] * 0x11111111u; xlo = regj_lo ^ ri; xhi = regj_hi ^ ri; }
        // the two columns a lane holds per key tile are handled as a pair (packed binary32 arithmetic, lane-wise
        // the same operations as the scalar contract)
        float2 lg[7];
        float mx = -3.0e38f;
#pragma unroll
        for (int nt = 0; nt < 7; ++nt) {
          const float4 rb = __ldg(relf + (mt * 7 + nt) * 32);
          const float2 sf = make_float2(__int2float_rn(c[nt][2 * r] + rqi + ckj[nt][0]),
                                        __int2float_rn(c[nt][2 * r + 1] + rqi + ckj[nt][1]));
          float2 v = __ffma2_rn(sf, f2(alpha), r == 0 ? make_float2(rb.x, rb.y) : make_float2(rb.z, rb.w));
          if (SHIFTED) {
            const uint32_t x0 = nt < 4 ? (xlo >> (4 * (2 * nt))) & 15u : (xhi >> (4 * (2 * (nt - 4)))) & 15u;
            const uint32_t x1 = nt < 4 ? (xlo >> (4 * (2 * nt + 1))) & 15u : (xhi >> (4 * (2 * (nt - 4) + 1))) & 15u;
            v = __fadd2_rn(v, make_float2(x0 != 0 ? -100.0f : 0.0f, x1 != 0 ? -100.0f : 0.0f));
          }
          lg[nt] = v;
          // key columns 49..55 do not exist: of tile 6 only column 0 of lane t = 0
          if (nt < 6 || t == 0) mx = fmaxf(mx, v.x);
          if (nt < 6) mx = fmaxf(mx, v.y);
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        // exponentials and this lane's partial sum in column order (the partial of index t of the contract)
        float part = 0.0f;
#pragma unroll
        for (int nt = 0; nt < 7; ++nt) {
          float2 tt = __fmul2_rn(sub2(lg[nt], f2(mx)), f2(kLog2e));
          tt = make_float2(fmaxf(tt.x, -125.0f), fmaxf(tt.y, -125.0f));
          float2 e = exp2_core2(tt);
          if (!(nt < 6 || t == 0)) e.x = 0.0f;
          if (!(nt < 6)) e.y = 0.0f;
          lg[nt] = e;
          part = __fadd_rn(__fadd_rn(part, e.x), e.y);
        }
        const float s1 = __fadd_rn(part, __shfl_xor_sync(0xffffffffu, part, 1));
        const float sum = __fadd_rn(s1, __shfl_xor_sync(0xffffffffu, s1, 2));
        const float inv = __fdiv_rn(1.0f, sum);
        // P codes: clamp(rne(p * pmax), 0, pmax); byte u of A register (ks, r [+2]) is tile 4ks + [2 +] (u>>1), column u&1.
        // The clamp never acts: 0 <= e_j <= sum, so p * pmax lies in [0, pmax * (1 + 2^-22)] and rounds into 0 .. pmax;
        // it is left out.  The rounded values stay in their "1.5 * 2^23 + code" patterns: the patterns are added into
        // the A registers shifted into place and the bias they carry is taken out once per register.
        uint32_t acc_pa[4] = {0u, 0u, 0u, 0u};
        uint32_t ps_raw = 0u;
#pragma unroll
        for (int nt = 0; nt < 7; ++nt) {
          const float2 pr = __fmul2_rn(lg[nt], f2(inv));          // the softmax output itself
          if (TAPS && br.tap_probs) {
            const int j0 = 8 * nt + 2 * t;
            float* tp = br.tap_probs + (((long)slot * a.heads + h) * WT + i) * WT;
            if (i < WT && j0 < WT) tp[j0] = pr.x;
            if (i < WT && j0 + 1 < WT) tp[j0 + 1] = pr.y;
          }
          // two roundings (product, then the add that rounds to an integer).  The products are scalar multiplies: a
          // packed multiply feeding a packed add gets contracted into one fused operation, which rounds once and
          // differs at exact .5 ties
          const float2 tq = __fadd2_rn(make_float2(__fmul_rn(pr.x, pmaxf), __fmul_rn(pr.y, pmaxf)), f2(12582912.0f));
          const uint32_t pat[2] = {__float_as_uint(tq.x), __float_as_uint(tq.y)};
          const int ks = nt >> 2, sub = nt & 3;
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            ps_raw += pat[u];
            acc_pa[2 * ks + (sub >> 1)] += pat[u] << (8 * (2 * (sub & 1) + u));
            if (TAPS && br.tap_p) {
              const int j = 8 * nt + 2 * t + u;
              if (i < WT && j < WT) br.tap_p[(((long)slot * a.heads + h) * WT + i) * WT + j] = (uint8_t)(pat[u] - kMagicBits);
            }
          }
        }
        // register (ks, half): four patterns (three for ks = 1, half = 1: tiles 4..6 only); the low byte of a pattern's
        // bias 0x4B400000 is zero, so shifted into a byte lane it only reaches higher bytes, which the sum drops
        // beyond bit 31: bias of a register = sum over its lanes of (0x4B400000 << 8 lane) mod 2^32
        constexpr uint32_t kBias4 = kMagicBits + (kMagicBits << 8) + (kMagicBits << 16) + (kMagicBits << 24);
        constexpr uint32_t kBias2 = kMagicBits + (kMagicBits << 8);
        pa[0][r] = acc_pa[0] - kBias4;  pa[0][r + 2] = acc_pa[1] - kBias4;
        pa[1][r] = acc_pa[2] - kBias4;  pa[1][r + 2] = acc_pa[3] - kBias2;
        int ps = (int)(ps_raw - 14u * kMagicBits);
        ps += __shfl_xor_sync(0xffffffffu, ps, 1);
        ps += __shfl_xor_sync(0xffffffffu, ps, 2);
        psum[r] = ps;
      }
    }
    // ---- O = P V for the 16 rows: two 32-key steps, four 8-column tiles of the head dimension ----
    int d[4][4];
#pragma unroll
    for (int ne = 0; ne < 4; ++ne) {
      d[ne][0] = d[ne][1] = d[ne][2] = d[ne][3] = 0;
#pragma unroll
      for (int ks = 0; ks < 2; ++ks)
        mma_u8(d[ne], pa[ks], sm.vt[8 * ne + g][8 * ks + t], sm.vt[8 * ne + g][8 * ks + 4 + t]);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int i = 16 * mt + g + 8 * r;
#pragma unroll
      for (int ne = 0; ne < 4; ++ne) {
        const int o0 = d[ne][2 * r] - zv * psum[r], o1 = d[ne][2 * r + 1] - zv * psum[r];
        if (TAPS && br.tap_pv && r < nrows && i < WT) {
          int* tp = br.tap_pv + (m_base + i) * C + h * HEAD_DIM + 8 * ne + 2 * t;
          tp[0] = o0; tp[1] = o1;
        }
        // O = O_int * s_p*s_v, then the proj-input quantizer, both columns of the lane at once
        uint32_t m0, m1;
        quant_magic2(__fmul2_rn(make_float2(__int2float_rn(o0), __int2float_rn(o1)), f2(so)), oq.inv_scale, -oq.zpf,
                     oq.qmaxf - oq.zpf, m0, m1);
        const uint32_t kz = (uint32_t)oq.zp - kMagicBits;
        reinterpret_cast<uint16_t*>(&sm.o[warp][g + 8 * r][0])[4 * ne + t] = (uint16_t)((m0 + kz) | ((m1 + kz) << 8));
      }
    }
    __syncwarp();
    if (lane < 16) {
      const int i = 16 * mt + lane;
      if (i < WT) {
        const uint4 w0 = *reinterpret_cast<const uint4*>(&sm.o[warp][lane][0]);
        const uint4 w1 = *reinterpret_cast<const uint4*>(&sm.o[warp][lane][4]);
        uint8_t* dst = br.out + (m_base + i) * out_row_bytes + (long)h * HEAD_DIM * cbits / 8;
        if (cbits == 8) {
          reinterpret_cast<uint4*>(dst)[0] = w0;
          reinterpret_cast<uint4*>(dst)[1] = w1;
        } else {
          const uint32_t n0 = pack_nibbles(w0.x, w0.y), n1 = pack_nibbles(w0.z, w0.w);
          const uint32_t n2 = pack_nibbles(w1.x, w1.y), n3 = pack_nibbles(w1.z, w1.w);
          if (cbits == 4) {
            reinterpret_cast<uint4*>(dst)[0] = make_uint4(n0, n1, n2, n3);
          } else {
            reinterpret_cast<uint2*>(dst)[0] = make_uint2(squeeze_pairs(n0) | (squeeze_pairs(n1) << 16),
                                                          squeeze_pairs(n2) | (squeeze_pairs(n3) << 16));
          }
        }
      }
    }
  }
}

}  // namespace

void launch_attention(const AttnArgs& a, cudaStream_t st) {
  const long problems = (long)(a.br[0].slots + a.br[1].slots) * a.heads;
  if (problems == 0) return;
  const unsigned grid = (unsigned)problems;
  const bool taps = a.br[0].tap_p || a.br[0].tap_pv || a.br[0].tap_probs || a.br[1].tap_p || a.br[1].tap_pv || a.br[1].tap_probs;
  if (a.shift > 0) {
    if (taps) k_attention<true, true><<<grid, ATT_WARPS * 32, 0, st>>>(a);
    else      k_attention<true, false><<<grid, ATT_WARPS * 32, 0, st>>>(a);
  } else {
    if (taps) k_attention<false, true><<<grid, ATT_WARPS * 32, 0, st>>>(a);
    else      k_attention<false, false><<<grid, ATT_WARPS * 32, 0, st>>>(a);
  }
  ++g_launches;
}

}  // namespace mixaq
