// Memory-bound row kernels: gather + LayerNorm + quantize + bit-pack (both branches in one launch),
// the patch-merging gather, and the pass-through copy of pruned windows (MixA-Q Section 3.2 / 3.4).
// One warp owns one token row; lane l holds channels l, l+32, l+64, ... so every load is a full 128-byte line.
#include "kernels.h"

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
#define MIXAQ_NPL_CASE(n, KERNEL, ...) case n: KERNEL<n><<<grid, 256, 0, st>>>(__VA_ARGS__); break;
#define MIXAQ_LN_CASE(n, rmax) case n: launch_ln_npl<n, rmax>(hi, lo, st); break;

void launch_ln_quant(const LnBranch& hi, const LnBranch& lo, int C, cudaStream_t st) {
  if (hi.M + lo.M == 0) return;
  switch (C / 32) {
    MIXAQ_LN_CASE(1, 8) MIXAQ_LN_CASE(2, 8) MIXAQ_LN_CASE(3, 8) MIXAQ_LN_CASE(4, 8) MIXAQ_LN_CASE(6, 4)
    MIXAQ_LN_CASE(8, 4) MIXAQ_LN_CASE(12, 2) MIXAQ_LN_CASE(16, 2) MIXAQ_LN_CASE(24, 1) MIXAQ_LN_CASE(32, 1)
    default: return;   // rejected by the host API before any launch
  }
  ++g_launches;
}

void launch_merge_gather(const MergeGatherArgs& a, cudaStream_t st) {
  long toks = (long)a.B * ((a.H + 1) / 2) * ((a.W + 1) / 2);
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
