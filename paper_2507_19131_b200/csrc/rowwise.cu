// Memory-bound row kernels: gather + LayerNorm + quantize + bit-pack (both branches in one launch),
// the patch-merging gather, and the pass-through copy of pruned windows (MixA-Q Section 3.2 / 3.4).
// Two LayerNorm kernels with the same summation tree: one warp per row (lane l holds channels l, l+32, l+64, ...,
// every load a full 128-byte line) and, for large batches of narrow rows, 4 or 8 lanes per row with vector loads.
#include "kernels.h"
#include <type_traits>

namespace mixaq {

// R rows per warp are in flight together: their loads are issued before any of the reductions starts.
// A CTA works for one branch only (the first `blocks_hi` CTAs take the high batch), so the branch's constants
// (gamma, beta, quantizer) are fetched once per warp and no per-row selection is left in the loop.
template <int NPL, int R>
__global__ void __launch_bounds__(256) k_ln_quant(LnBranch hi, LnBranch lo, int blocks_hi) {
  const int C = NPL * 32;
  const int lane = threadIdx.x & 31;
  const bool is_hi = (int)blockIdx.x < blocks_hi;
  const LnBranch& br = is_hi ? hi : lo;
  const int M = br.M;
  const int m_base = (((is_hi ? blockIdx.x : blockIdx.x - blocks_hi) * (blockDim.x >> 5)) + (threadIdx.x >> 5)) * R;
  if (m_base >= M) return;
  const float* __restrict__ src = br.src;
  const int32_t* __restrict__ rowsrc = br.rowsrc;
  long srow[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int m = m_base + r;
    srow[r] = -1;
    if (m < M) srow[r] = rowsrc ? (long)rowsrc[m] : (long)m;
  }
  float x[R][NPL];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const float* row = src + (srow[r] < 0 ? 0 : srow[r]) * C + lane;
#pragma unroll
    for (int i = 0; i < NPL; ++i) x[r][i] = srow[r] < 0 ? 0.0f : __ldg(row + 32 * i);
  }
  float gam[NPL], bet[NPL];
#pragma unroll
  for (int i = 0; i < NPL; ++i) { gam[i] = __ldg(br.gamma + lane + 32 * i); bet[i] = __ldg(br.beta + lane + 32 * i); }
  const AQ q = br.q;
  const int row_bytes = C * q.bits / 8;
  float mean[R], rstd[R];
  ln_stats_rows<NPL, R>(x, (float)C, mean, rstd);
  const uint32_t zcode = quant_code(0.0f, q);      // pad token: zero after the normalisation
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int m = m_base + r;
    if (m >= M) break;
    uint32_t code[NPL];
#pragma unroll
    for (int i = 0; i < NPL; ++i)
      code[i] = srow[r] < 0 ? zcode : quant_code(ln_apply(x[r][i], mean[r], rstd[r], gam[i], bet[i]), q);
    store_codes_lane_strided<NPL>(br.out + (long)m * row_bytes, code, q.bits, lane);
  }
}

// The same LayerNorm for large batches of narrow rows: G lanes share a row and a warp works on 32/G rows at once.
// Lane j of a row's group owns the partial sums of indices P*j .. P*j+P-1 (P = 32/G) of the 32 interleaved
// partials, i.e. of every 32-channel group the P contiguous channels 32i + P*j ..: vector loads, whole bytes of
// codes per lane, and the butterfly (offsets 16, 8, 4, 2, 1 on the partial index) becomes log2(G) exchanges
// between lanes followed by a tree inside the lane -- the same additions in the same order.
// MERGE: the rows are the output tokens of a patch merging: channel group i of a row comes from input neighbour
// i / (NG/4) (order (0,0), (1,0), (0,1), (1,1)); neighbours outside the map are zeros that take part in the LayerNorm.
template <int NG, int G, bool MERGE>
__global__ void __launch_bounds__(256, (NG * (32 / G) > 24 ? 2 : 4)) k_ln_quant_g(LnBranch hi, LnBranch lo, int blocks_hi) {
  constexpr int C = NG * 32, P = 32 / G, ROWS = 32 / G;     // channels, partials per lane, rows per warp
  constexpr int VEC = P >= 4 ? 4 : 2;                       // floats per load
  static_assert(P >= 2 && (!MERGE || NG % 4 == 0), "unsupported lane split");
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int j = lane % G, rw = lane / G;
  const bool is_hi = (int)blockIdx.x < blocks_hi;
  const LnBranch& br = is_hi ? hi : lo;
  const int M = br.M;
  const int blk = is_hi ? blockIdx.x : blockIdx.x - blocks_hi;
  const int m0 = (blk * 8 + warp) * ROWS;
  if (m0 >= M) return;
  const int m = m0 + rw;
  const AQ q = br.q;
  const int bits = q.bits;
  long srow = -1;
  if (m < M) srow = (MERGE || !br.rowsrc) ? (long)m : (long)br.rowsrc[m];
  // source rows: one (gather / plain) or the four input neighbours (merge); -1: zeros
  long nsrc[MERGE ? 4 : 1];
  if (MERGE) {
    const int H2 = (br.mgH + 1) / 2, W2 = (br.mgW + 1) / 2;
    const int mm = m < M ? m : 0;
    const int b = mm / (H2 * W2), r2 = mm - b * (H2 * W2), y2 = r2 / W2, x2 = r2 - y2 * W2;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      const int yy = 2 * y2 + (g & 1), xx = 2 * x2 + (g >> 1);
      nsrc[MERGE ? g : 0] = (m < M && yy < br.mgH && xx < br.mgW) ? ((long)b * br.mgH + yy) * br.mgW + xx : -1;
    }
  } else {
    nsrc[0] = srow;
  }
  float x[NG][P];
#pragma unroll
  for (int i = 0; i < NG; ++i) {
    constexpr int GPN = MERGE ? NG / 4 : NG;                 // channel groups per source row
    const long sr = nsrc[MERGE ? i / GPN : 0];
    const float* src = br.src + (sr < 0 ? 0 : sr) * (GPN * 32) + 32 * (i % GPN) + P * j;
#pragma unroll
    for (int v = 0; v < P / VEC; ++v) {
      if (VEC == 4) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        if (sr >= 0) a = __ldg(reinterpret_cast<const float4*>(src) + v);
        x[i][4 * v] = a.x; x[i][4 * v + 1] = a.y; x[i][4 * v + 2] = a.z; x[i][4 * v + 3] = a.w;
      } else {
        float2 a = make_float2(0.f, 0.f);
        if (sr >= 0) a = __ldg(reinterpret_cast<const float2*>(src) + v);
        x[i][2 * v] = a.x; x[i][2 * v + 1] = a.y;
      }
    }
  }
  // partial sums in channel order, then the butterfly: lanes first (offsets 16 .. P), then inside the lane
  auto reduce32 = [&](float (&p)[P]) -> float {
#pragma unroll
    for (int o = G / 2; o >= 1; o >>= 1)
#pragma unroll
      for (int k = 0; k < P; ++k) p[k] = __fadd_rn(p[k], __shfl_xor_sync(0xffffffffu, p[k], o));
#pragma unroll
    for (int o = P / 2; o >= 1; o >>= 1)
#pragma unroll
      for (int k = 0; k < o; ++k) p[k] = __fadd_rn(p[k], p[k + o]);
    return p[0];
  };
  // neighbouring partials are summed as pairs (packed binary32 arithmetic: each lane adds in the same order)
  float p[P];
#pragma unroll
  for (int k = 0; k < P; k += 2) {
    float2 s = f2(0.0f);
#pragma unroll
    for (int i = 0; i < NG; ++i) s = __fadd2_rn(s, make_float2(x[i][k], x[i][k + 1]));
    p[k] = s.x; p[k + 1] = s.y;
  }
  const float mean = __fdiv_rn(reduce32(p), (float)C);
#pragma unroll
  for (int k = 0; k < P; k += 2) {
    float2 v = f2(0.0f);
#pragma unroll
    for (int i = 0; i < NG; ++i) { const float2 d = sub2(make_float2(x[i][k], x[i][k + 1]), f2(mean)); v = __ffma2_rn(d, d, v); }
    p[k] = v.x; p[k + 1] = v.y;
  }
  const float var = __fdiv_rn(reduce32(p), (float)C);
  const float rstd = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(var, 1e-5f)));
  if (m >= M) return;
  // the normalisation, the quantizer and the packing with the bit width as a compile-time constant (a CTA works for
  // one branch, so the switch is uniform)
  auto finish = [&](auto bits_tag) {
    constexpr int BITS = decltype(bits_tag)::value;
    constexpr int PER = 32 / BITS;                     // codes per 32-bit word
    uint8_t* out = br.out + (long)m * (C * BITS / 8) + (P * j) * BITS / 8;
    const uint32_t kpack = pack_const(q.zp, BITS);
    // a pad token is zero after the normalisation: all its codes are the code of zero
    uint32_t zw0 = kpack, zw1 = kpack;
    {
      const uint32_t zpat = quant_magic(0.0f, q);
#pragma unroll
      for (int k = 0; k < P; ++k) { if (k < PER) zw0 += zpat << (BITS * k); else zw1 += zpat << (BITS * (k - PER)); }
    }
#pragma unroll
    for (int i = 0; i < NG; ++i) {
      uint32_t w0 = kpack, w1 = kpack;
#pragma unroll
      for (int v4 = 0; v4 < P / VEC; ++v4) {
        float gg[4], bb[4];
        if (VEC == 4) {
          const float4 g4 = __ldg(reinterpret_cast<const float4*>(br.gamma + 32 * i + P * j) + v4);
          const float4 b4 = __ldg(reinterpret_cast<const float4*>(br.beta + 32 * i + P * j) + v4);
          gg[0] = g4.x; gg[1] = g4.y; gg[2] = g4.z; gg[3] = g4.w; bb[0] = b4.x; bb[1] = b4.y; bb[2] = b4.z; bb[3] = b4.w;
        } else {
          const float2 g2 = __ldg(reinterpret_cast<const float2*>(br.gamma + 32 * i + P * j) + v4);
          const float2 b2 = __ldg(reinterpret_cast<const float2*>(br.beta + 32 * i + P * j) + v4);
          gg[0] = g2.x; gg[1] = g2.y; gg[2] = gg[3] = 0.f; bb[0] = b2.x; bb[1] = b2.y; bb[2] = bb[3] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < VEC; e += 2) {
          const int k = VEC * v4 + e;
          // y = fma((x - mean) * rstd, gamma, beta) on two channels, then their magic patterns
          const float2 d = __fmul2_rn(sub2(make_float2(x[i][k], x[i][k + 1]), f2(mean)), f2(rstd));
          const float2 y = __ffma2_rn(d, make_float2(gg[e], gg[e + 1]), make_float2(bb[e], bb[e + 1]));
          uint32_t pat[2];
          quant_magic2(y, q.inv_scale, -q.zpf, q.qmaxf - q.zpf, pat[0], pat[1]);
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            if (k + u < PER) w0 += pat[u] << (BITS * (k + u));
            else             w1 += pat[u] << (BITS * (k + u - PER));
          }
        }
      }
      if (srow < 0) { w0 = zw0; w1 = zw1; }
      // P codes of BITS bits: P*BITS/8 whole bytes (the launcher only picks G with P*BITS >= 8)
      uint8_t* dst = out + 32 * i * BITS / 8;
      constexpr int NBYTES = P * BITS / 8;
      if (NBYTES == 8) *reinterpret_cast<uint2*>(dst) = make_uint2(w0, w1);
      else if (NBYTES == 4) *reinterpret_cast<uint32_t*>(dst) = w0;
      else if (NBYTES == 2) *reinterpret_cast<uint16_t*>(dst) = (uint16_t)w0;
      else *dst = (uint8_t)w0;
    }
  };
  if (bits == 8) finish(std::integral_constant<int, 8>{});
  else if (bits == 4) finish(std::integral_constant<int, 4>{});
  else finish(std::integral_constant<int, 2>{});
}

// patch merging: token (b, y2, x2) of the output gathers (2y2+dy, 2x2+dx) for (dy,dx) = (0,0),(1,0),(0,1),(1,1)
// in this order along the channel axis; neighbours outside the map are zeros (they do take part in the LN).
template <int NPL>   // NPL = 4C/32
__global__ void __launch_bounds__(256) k_merge_gather(MergeGatherArgs a) {
  const int K = NPL * 32;
  const int C = K / 4;
  int H2 = (a.H + 1) / 2, W2 = (a.W + 1) / 2;
  long tok = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  if (tok >= (long)a.B * H2 * W2) return;
  int b = (int)(tok / ((long)H2 * W2));
  int r = (int)(tok - (long)b * H2 * W2);
  int y2 = r / W2, x2 = r - y2 * W2;
  float x[NPL];
#pragma unroll
  for (int i = 0; i < NPL; ++i) {
    int c = lane + 32 * i;
    int g = c / C, cc = c - g * C;
    int yy = 2 * y2 + (g & 1), xx = 2 * x2 + (g >> 1);
    x[i] = (yy < a.H && xx < a.W) ? __ldg(a.x + (((long)b * a.H + yy) * a.W + xx) * C + cc) : 0.0f;
  }
  float mean, rstd;
  ln_stats<NPL>(x, (float)K, mean, rstd);
  uint32_t code[NPL];
  AQ q = a.q;
#pragma unroll
  for (int i = 0; i < NPL; ++i) {
    int c = lane + 32 * i;
    code[i] = quant_code(ln_apply(x[i], mean, rstd, __ldg(a.gamma + c), __ldg(a.beta + c)), q);
  }
  store_codes_lane_strided<NPL>(a.out + tok * (K * q.bits / 8), code, q.bits, lane);
}

__global__ void __launch_bounds__(256) k_copy_rows(const float* __restrict__ x, float* __restrict__ y,
                                                   const int32_t* __restrict__ rowsrc, int M, int C) {
  int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  if (row >= M) return;
  long s = rowsrc[row];
  if (s < 0) return;
  for (int c = lane; c < C; c += 32) y[s * C + c] = __ldg(x + s * C + c);
}

#define MIXAQ_NPL_CASE(n, KERNEL, ...) case n: KERNEL<n><<<grid, 256, 0, st>>>(__VA_ARGS__); break;
template <int NPL, int R>
void launch_ln_r(const LnBranch& hi, const LnBranch& lo, cudaStream_t st) {
  const int rows_per_block = 8 * R;
  const int bh = (hi.M + rows_per_block - 1) / rows_per_block, bl = (lo.M + rows_per_block - 1) / rows_per_block;
  k_ln_quant<NPL, R><<<bh + bl, 256, 0, st>>>(hi, lo, bh);
}
// rows per warp: more rows amortise the per-warp constants and the divisions, but small problems need the warps
template <int NPL, int RMAX>
void launch_ln_npl(const LnBranch& hi, const LnBranch& lo, cudaStream_t st) {
  const int rows = hi.M + lo.M;
  if (RMAX >= 8 && rows >= 8 * 8 * 148 * 4) launch_ln_r<NPL, (RMAX >= 8 ? 8 : RMAX)>(hi, lo, st);
  else if (RMAX >= 4 && rows >= 4 * 8 * 148 * 4) launch_ln_r<NPL, (RMAX >= 4 ? 4 : RMAX)>(hi, lo, st);
  else if (RMAX >= 2 && rows >= 2 * 8 * 148 * 4) launch_ln_r<NPL, (RMAX >= 2 ? 2 : RMAX)>(hi, lo, st);
  else launch_ln_r<NPL, 1>(hi, lo, st);
}
#define MIXAQ_LN_CASE(n, rmax) case n: launch_ln_npl<n, rmax>(hi, lo, st); break;

template <int NG, int G, bool MERGE = false>
void launch_ln_g(const LnBranch& hi, const LnBranch& lo, cudaStream_t st) {
  const int rpb = 8 * (32 / G);                              // rows per block: 8 warps x 32/G rows
  const int bh = (hi.M + rpb - 1) / rpb, bl = (lo.M + rpb - 1) / rpb;
  k_ln_quant_g<NG, G, MERGE><<<bh + bl, 256, 0, st>>>(hi, lo, bh);
}

void launch_ln_quant(const LnBranch& hi, const LnBranch& lo, int C, cudaStream_t st) {
  if (hi.M + lo.M == 0) return;
  // narrow rows in large batches: several lanes per row, provided every lane then stores whole bytes of codes
  const int rows = hi.M + lo.M;
  const int min_bits = hi.M > 0 && lo.M > 0 ? (hi.q.bits < lo.q.bits ? hi.q.bits : lo.q.bits) : (hi.M > 0 ? hi.q.bits : lo.q.bits);
  bool done = false;
  if (rows >= 8192) {
    done = true;
    if (C == 32) launch_ln_g<1, 4>(hi, lo, st);
    else if (C == 64) launch_ln_g<2, 4>(hi, lo, st);
    else if (C == 96) launch_ln_g<3, 4>(hi, lo, st);
    else if (C == 128) launch_ln_g<4, 4>(hi, lo, st);
    else if (C == 192 && min_bits * 4 >= 8) launch_ln_g<6, 8>(hi, lo, st);
    else if (C == 256 && min_bits * 4 >= 8) launch_ln_g<8, 8>(hi, lo, st);
    else done = false;
  }
  // wide rows: 8 lanes per row pay at any batch size (a third of the instructions of one warp per row)
  if (!done && C == 384) { launch_ln_g<12, 8>(hi, lo, st); done = true; }
  if (!done && C == 512) { launch_ln_g<16, 8>(hi, lo, st); done = true; }
  if (!done && C == 768 && min_bits * 2 >= 8) { launch_ln_g<24, 16>(hi, lo, st); done = true; }
  if (!done && C == 1024 && min_bits * 2 >= 8) { launch_ln_g<32, 16>(hi, lo, st); done = true; }
  if (done) { ++g_launches; return; }
  switch (C / 32) {
    MIXAQ_LN_CASE(1, 8) MIXAQ_LN_CASE(2, 8) MIXAQ_LN_CASE(3, 8) MIXAQ_LN_CASE(4, 8) MIXAQ_LN_CASE(6, 4)
    MIXAQ_LN_CASE(8, 4) MIXAQ_LN_CASE(12, 2) MIXAQ_LN_CASE(16, 2) MIXAQ_LN_CASE(24, 1) MIXAQ_LN_CASE(32, 1)
    default: return;   // rejected by the host API before any launch
  }
  ++g_launches;
}

void launch_merge_gather(const MergeGatherArgs& a, cudaStream_t st) {
  long toks = (long)a.B * ((a.H + 1) / 2) * ((a.W + 1) / 2);
  // 4C = 384 ... 1024: the multi-lane LayerNorm kernel with the rows gathered from the four input neighbours
  const int K4 = 4 * a.C;
  if ((K4 == 384 || K4 == 512 || ((K4 == 768 || K4 == 1024) && a.q.bits * 2 >= 8)) && toks < (1L << 31)) {
    LnBranch hi, lo;
    hi.src = a.x; hi.rowsrc = nullptr; hi.gamma = a.gamma; hi.beta = a.beta; hi.out = a.out; hi.q = a.q; hi.M = (int)toks;
    hi.mgH = a.H; hi.mgW = a.W;
    lo = hi; lo.M = 0;
    if (K4 == 384) launch_ln_g<12, 8, true>(hi, lo, st);
    else if (K4 == 512) launch_ln_g<16, 8, true>(hi, lo, st);
    else if (K4 == 768) launch_ln_g<24, 16, true>(hi, lo, st);
    else launch_ln_g<32, 16, true>(hi, lo, st);
    ++g_launches;
    return;
  }
  unsigned grid = (unsigned)((toks + 7) / 8);
  switch (4 * a.C / 32) {
    MIXAQ_NPL_CASE(4, k_merge_gather, a) MIXAQ_NPL_CASE(8, k_merge_gather, a) MIXAQ_NPL_CASE(12, k_merge_gather, a)
    MIXAQ_NPL_CASE(16, k_merge_gather, a) MIXAQ_NPL_CASE(24, k_merge_gather, a) MIXAQ_NPL_CASE(32, k_merge_gather, a)
    MIXAQ_NPL_CASE(48, k_merge_gather, a) MIXAQ_NPL_CASE(64, k_merge_gather, a)
    default: return;
  }
  ++g_launches;
}

void launch_copy_rows(const float* x, float* y, const int32_t* rowsrc, int M, int C, cudaStream_t st) {
  if (M == 0) return;
  k_copy_rows<<<(M + 7) / 8, 256, 0, st>>>(x, y, rowsrc, M, C);
  ++g_launches;
}

bool ln_dim_supported(int C) {
  switch (C / 32) { case 1: case 2: case 3: case 4: case 6: case 8: case 12: case 16: case 24: case 32: return C % 32 == 0; }
  return false;
}
bool merge_dim_supported(int C) {
  switch (4 * C / 32) { case 4: case 8: case 12: case 16: case 24: case 32: case 48: case 64: return C % 32 == 0; }
  return false;
}

}  // namespace mixaq
