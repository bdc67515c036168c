// Fused epilogues of the integer GEMMs (MixA-Q Section 3.2: shared integer weights, per-branch step sizes,
// zero points and biases).  One call handles 32 consecutive output columns of one row, which is exactly the
// shape one thread receives from a 32-lane x 32-column TMEM load.
//   acc_raw[n] = sum_k a[m][k] * w[n][k]   with UNSIGNED activation codes a;
//   acc[n]     = acc_raw[n] - z_a * sum_k w[n][k]                (zero-point correction, exact in int32)
//   v[n]       = fma((float)acc[n], s_a*s_w[n], bias[n])
#pragma once
#include "kernels.h"

namespace mixaq {

template <int MODE>
__device__ __forceinline__ void epilogue_row32(const GemmBranch& br, int N, int C, long m, int n0,
                                               const int32_t (&acc_raw)[32]) {
  float v[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    int n = n0 + i;
    int32_t acc = acc_raw[i] - __ldg(br.zc + n);
    if (br.tap_acc) br.tap_acc[m * N + n] = acc;
    float f = __int2float_rn(acc);
    if (MODE == EPI_MERGE) v[i] = __fmul_rn(f, __ldg(br.mult + n));
    else                   v[i] = __fmaf_rn(f, __ldg(br.mult + n), __ldg(br.bias + n));
  }
  if (MODE == EPI_QKV || MODE == EPI_FC1) {
    AQ q = br.q0;
    if (MODE == EPI_QKV) { int sec = n0 / C; if (sec == 1) q = br.q1; else if (sec == 2) q = br.q2; }
    uint32_t c[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) c[i] = quant_code(MODE == EPI_FC1 ? gelu_f(v[i]) : v[i], q);
    int bits = br.out_bits;
    store_codes_32(br.out_codes + m * ((long)N * bits / 8) + (long)n0 * bits / 8, c, bits);
  } else if (MODE == EPI_PROJ) {
    long s = br.rowsrc[m];
    float* dst = br.out_f + m * N + n0;
    if (s >= 0) {
      const float4* r4 = reinterpret_cast<const float4*>(br.res + s * N + n0);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float4 r = __ldg(r4 + i);
        reinterpret_cast<float4*>(dst)[i] = make_float4(__fadd_rn(r.x, v[4 * i]), __fadd_rn(r.y, v[4 * i + 1]),
                                                        __fadd_rn(r.z, v[4 * i + 2]), __fadd_rn(r.w, v[4 * i + 3]));
      }
    } else {
      // pad token: its residual input is zero
#pragma unroll
      for (int i = 0; i < 8; ++i)
        reinterpret_cast<float4*>(dst)[i] = make_float4(__fadd_rn(0.0f, v[4 * i]), __fadd_rn(0.0f, v[4 * i + 1]),
                                                        __fadd_rn(0.0f, v[4 * i + 2]), __fadd_rn(0.0f, v[4 * i + 3]));
    }
  } else if (MODE == EPI_FC2) {
    long s = br.rowsrc[m];
    if (s >= 0) {
      const float4* r4 = reinterpret_cast<const float4*>(br.res + m * N + n0);
      float4* d4 = reinterpret_cast<float4*>(br.out_f + s * N + n0);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float4 r = __ldg(r4 + i);
        d4[i] = make_float4(__fadd_rn(r.x, v[4 * i]), __fadd_rn(r.y, v[4 * i + 1]),
                            __fadd_rn(r.z, v[4 * i + 2]), __fadd_rn(r.w, v[4 * i + 3]));
      }
    }
  } else {  // EPI_MERGE
    float4* d4 = reinterpret_cast<float4*>(br.out_f + m * N + n0);
#pragma unroll
    for (int i = 0; i < 8; ++i) d4[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
  }
}

}  // namespace mixaq
