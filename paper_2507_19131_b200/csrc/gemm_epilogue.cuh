// Fused epilogues of the integer GEMMs (MixA-Q Section 3.2: shared integer weights, per-branch step sizes,
// zero points and biases).  One call handles 32 consecutive output columns of 32 consecutive rows: the shape a
// warp receives from a 32-lane x 32-column TMEM load (one row per thread).
//   acc_raw[n] = sum_k a[m][k] * w[n][k]   with UNSIGNED activation codes a;
//   acc[n]     = acc_raw[n] - z_a * sum_k w[n][k]                (zero-point correction, exact in int32)
//   v[n]       = fma((float)acc[n], s_a*s_w[n], bias[n])
// The per-column constants (zc, mult, bias) of the tile sit in shared memory; every lane of a warp reads the
// same column, so the reads are broadcasts.
#pragma once
#include "kernels.h"

namespace mixaq {

constexpr int EPI_STAGE_LD = 36;                       // floats per row of a warp's 32 x 32 staging tile (padded)
constexpr int EPI_STAGE_FLOATS = 32 * EPI_STAGE_LD;

struct ColConsts {                                     // shared-memory arrays indexed by the tile's local column
  const int32_t* zc; const float* mult; const float* bias;
};

// row0: first row of the warp's 32-row slab (global row index in the branch's matrix); lane owns row0 + lane.
// n0: global first column of the group; lc0: its column inside the tile (index into the shared constants).
template <int MODE>
__device__ __forceinline__ void epilogue_row32(const GemmBranch& br, int N, int C, long row0, int lane, int n0, int lc0,
                                               const ColConsts& cc, const int32_t (&acc_raw)[32], float* stage) {
  const long m = row0 + lane;
  const bool row_ok = m < br.M;
  float v[32];
#pragma unroll
  for (int i4 = 0; i4 < 8; ++i4) {
    const int4 z4 = *reinterpret_cast<const int4*>(cc.zc + lc0 + 4 * i4);
    const float4 m4 = *reinterpret_cast<const float4*>(cc.mult + lc0 + 4 * i4);
    const int zz[4] = {z4.x, z4.y, z4.z, z4.w};
    const float mm[4] = {m4.x, m4.y, m4.z, m4.w};
    float bb[4] = {0.f, 0.f, 0.f, 0.f};
    if (MODE != EPI_MERGE) {
      const float4 b4 = *reinterpret_cast<const float4*>(cc.bias + lc0 + 4 * i4);
      bb[0] = b4.x; bb[1] = b4.y; bb[2] = b4.z; bb[3] = b4.w;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = 4 * i4 + j;
      const int32_t acc = acc_raw[i] - zz[j];
      if (br.tap_acc && row_ok) br.tap_acc[m * N + n0 + i] = acc;
      const float f = __int2float_rn(acc);
      if (MODE == EPI_MERGE) v[i] = __fmul_rn(f, mm[j]);
      else                   v[i] = __fmaf_rn(f, mm[j], bb[j]);
    }
  }
  if (MODE == EPI_QKV || MODE == EPI_FC1) {
    AQ q = br.q0;
    if (MODE == EPI_QKV) { int sec = n0 / C; if (sec == 1) q = br.q1; else if (sec == 2) q = br.q2; }
    uint32_t c[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) c[i] = quant_magic(MODE == EPI_FC1 ? gelu_f(v[i]) : v[i], q);
    if (row_ok) {
      const int bits = br.out_bits;
      uint8_t* dst = br.out_codes + m * ((long)N * bits / 8) + (long)n0 * bits / 8;
      const uint32_t kp = pack_const(q.zp, bits);
      if (bits == 8) store_magic_32<8>(dst, c, kp);
      else if (bits == 4) store_magic_32<4>(dst, c, kp);
      else store_magic_32<2>(dst, c, kp);
    }
    return;
  }
  // binary32 outputs: transpose the warp's 32 x 32 block through shared memory so that every global access
  // is a run of full 128-byte lines (8 lanes per row) instead of 32 row-strided 16-byte pieces.
  __syncwarp();
#pragma unroll
  for (int j = 0; j < 8; ++j)
    *reinterpret_cast<float4*>(stage + lane * EPI_STAGE_LD + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
  long src_mine = -1;
  if (MODE != EPI_MERGE && row_ok) src_mine = br.rowsrc[m];
  __syncwarp();
  const int cj = lane & 7, rsub = lane >> 3;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = 4 * i + rsub;
    const long mr = row0 + r;
    const long s = __shfl_sync(0xffffffffu, src_mine, r);
    const float4 a = *reinterpret_cast<const float4*>(stage + r * EPI_STAGE_LD + 4 * cj);
    if (mr >= br.M) continue;
    const int col = n0 + 4 * cj;
    if (MODE == EPI_PROJ) {
      // x1 = x_window + out; a pad token's residual input is zero
      float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
      if (s >= 0) x = __ldg(reinterpret_cast<const float4*>(br.res + s * N + col));
      *reinterpret_cast<float4*>(br.out_f + mr * N + col) =
          make_float4(__fadd_rn(x.x, a.x), __fadd_rn(x.y, a.y), __fadd_rn(x.z, a.z), __fadd_rn(x.w, a.w));
    } else if (MODE == EPI_FC2) {
      // y = x1 + out, written at the token's own position of the un-shifted map; pad tokens are dropped
      if (s >= 0) {
        const float4 x = __ldg(reinterpret_cast<const float4*>(br.res + mr * N + col));
        *reinterpret_cast<float4*>(br.out_f + s * N + col) =
            make_float4(__fadd_rn(x.x, a.x), __fadd_rn(x.y, a.y), __fadd_rn(x.z, a.z), __fadd_rn(x.w, a.w));
      }
    } else {  // EPI_MERGE
      *reinterpret_cast<float4*>(br.out_f + mr * N + col) = a;
    }
  }
}

}  // namespace mixaq
