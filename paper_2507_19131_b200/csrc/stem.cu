// The steps on either side of the Two-Branch blocks: patch embedding in front (4x4 patches -> quantize -> integer
// projection -> + bias -> LayerNorm) and the LayerNorm of a stage's output map behind.  The paper counts these among
// the layers whose cost the method does not reduce (Appendix 6.2); all tokens run at the high bit width.
#include "kernels.h"

namespace mixaq {

// One thread per (output token, patch row ky): 4 pixels x 3 channels = 12 consecutive floats of the image
// (zeros outside it), quantized and stored as 12 codes at patch index (ky*4 + kx)*3 + c.  Rows are padded from 48
// to 64 codes (the integer GEMM wants K a multiple of 32; the padded weight columns are zero): the ky == 0 thread
// clears them.
__global__ void __launch_bounds__(256) k_patch_gather(PatchGatherArgs a) {
  const int H = (a.Hi + 3) / 4, W = (a.Wi + 3) / 4;
  const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const long tok = idx >> 2;
  const int ky = (int)(idx & 3);
  if (tok >= (long)a.B * H * W) return;
  const int b = (int)(tok / ((long)H * W)), r = (int)(tok - (long)b * H * W);
  const int ty = r / W, tx = r - ty * W;
  const int yy = 4 * ty + ky;
  uint32_t w[3] = {0, 0, 0};
  const AQ q = a.q;
#pragma unroll
  for (int j = 0; j < 12; ++j) {
    const int xx = 4 * tx + j / 3;
    float v = 0.0f;
    if (yy < a.Hi && xx < a.Wi) v = __ldg(a.img + (((long)b * a.Hi + yy) * a.Wi + xx) * 3 + (j % 3));
    w[j >> 2] |= quant_code(v, q) << (8 * (j & 3));
  }
  uint32_t* dst = reinterpret_cast<uint32_t*>(a.out + tok * 64 + ky * 12);
  dst[0] = w[0]; dst[1] = w[1]; dst[2] = w[2];
  if (ky == 0) *reinterpret_cast<uint4*>(a.out + tok * 64 + 48) = make_uint4(0, 0, 0, 0);
}

// y[row] = LayerNorm(x[row] + bias) with binary32 output; bias may be NULL.  One warp per row, the statistics of the
// numeric contract (lane l holds channels l, l+32, ...).
template <int NPL>
__global__ void __launch_bounds__(256) k_bias_ln(const float* __restrict__ x, const float* __restrict__ bias,
                                                 const float* __restrict__ gamma, const float* __restrict__ beta,
                                                 float* __restrict__ y, long rows) {
  const int C = NPL * 32;
  const long row = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  float v[NPL];
#pragma unroll
  for (int i = 0; i < NPL; ++i) {
    const int c = lane + 32 * i;
    v[i] = __ldg(x + row * C + c);
    if (bias) v[i] = __fadd_rn(v[i], __ldg(bias + c));
  }
  float mean, rstd;
  ln_stats<NPL>(v, (float)C, mean, rstd);
#pragma unroll
  for (int i = 0; i < NPL; ++i) {
    const int c = lane + 32 * i;
    y[row * C + c] = ln_apply(v[i], mean, rstd, __ldg(gamma + c), __ldg(beta + c));
  }
}

// padded copy of the stem projection: [C0][48] -> [C0][64], columns 48..63 zero
__global__ void k_pad_weights(const int8_t* __restrict__ w, int N, int K, int Kp, int8_t* __restrict__ out) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= N * Kp) return;
  const int n = idx / Kp, k = idx - n * Kp;
  out[idx] = k < K ? w[n * K + k] : (int8_t)0;
}

void launch_patch_gather(const PatchGatherArgs& a, cudaStream_t st) {
  const long threads = (long)a.B * ((a.Hi + 3) / 4) * ((a.Wi + 3) / 4) * 4;
  k_patch_gather<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(a);
  ++g_launches;
}

#define MIXAQ_BLN_CASE(n) case n: k_bias_ln<n><<<grid, 256, 0, st>>>(x, bias, gamma, beta, y, rows); break;
bool launch_bias_ln(const float* x, const float* bias, const float* gamma, const float* beta, float* y, long rows,
                    int C, cudaStream_t st) {
  if (rows <= 0) return true;
  const unsigned grid = (unsigned)((rows + 7) / 8);
  switch (C / 32) {
    MIXAQ_BLN_CASE(1) MIXAQ_BLN_CASE(2) MIXAQ_BLN_CASE(3) MIXAQ_BLN_CASE(4) MIXAQ_BLN_CASE(6) MIXAQ_BLN_CASE(8)
    MIXAQ_BLN_CASE(12) MIXAQ_BLN_CASE(16) MIXAQ_BLN_CASE(24) MIXAQ_BLN_CASE(32)
    default: return false;
  }
  ++g_launches;
  return true;
}

void launch_pad_weights(const int8_t* w, int N, int K, int Kp, int8_t* out, cudaStream_t st) {
  k_pad_weights<<<(N * Kp + 255) / 256, 256, 0, st>>>(w, N, K, Kp, out);
  ++g_launches;
}

}  // namespace mixaq
