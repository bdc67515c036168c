// One-time derived tables of a block: per-output-channel step-size products and zero-point corrections of
// every (linear layer, branch) pair, and the relative-position bias expanded to the attention kernel's fragment order.
#include "kernels.h"

namespace mixaq {

// one warp per output channel: zc[n] = z_a * sum_k w[n][k];  mult[n] = s_a * s_w[n]
__global__ void __launch_bounds__(256) k_prepare_linear(const int8_t* __restrict__ w, const float* __restrict__ sw,
                                                        int N, int K, float sa, int za, float* mult, int32_t* zc) {
  int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  if (n >= N) return;
  int s = 0;
  for (int k = lane; k < K; k += 32) s += (int)w[(long)n * K + k];
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
  if (lane == 0) { zc[n] = za * s; mult[n] = __fmul_rn(sa, sw[n]); }
}

// Relative-position bias in the order the attention kernel's accumulator fragments want it:
// out[((h*4 + mt)*7 + nt)*32 + lane] = float4 of bias[h][i][j] at (i, j) = (16mt+g, 8nt+2t), (16mt+g, 8nt+2t+1),
// (16mt+g+8, 8nt+2t), (16mt+g+8, 8nt+2t+1) with g = lane/4, t = lane%4; 0 outside the 49 x 49 table, where
// bias[h][i][j] = table[((yi - yj + 6) * 13 + (xi - xj + 6)) * heads + h].
__global__ void k_prepare_relbias(const float* __restrict__ table, int heads, float* out) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= heads * 4 * 7 * 32 * 4) return;
  const int comp = idx & 3, lane = (idx >> 2) & 31;
  const int tile = idx >> 7;                       // (h*4 + mt)*7 + nt
  const int nt = tile % 7, mt = (tile / 7) & 3, h = tile / 28;
  const int i = 16 * mt + (lane >> 2) + 8 * (comp >> 1);
  const int j = 8 * nt + 2 * (lane & 3) + (comp & 1);
  float v = 0.0f;
  if (i < WT && j < WT) {
    int dy = i / WS - j / WS + (WS - 1), dx = i % WS - j % WS + (WS - 1);
    v = table[(dy * (2 * WS - 1) + dx) * heads + h];
  }
  out[idx] = v;
}

void launch_prepare_linear(const int8_t* w, const float* sw, int N, int K, float sa, int za, float* mult,
                           int32_t* zc, cudaStream_t st) {
  k_prepare_linear<<<(N + 7) / 8, 256, 0, st>>>(w, sw, N, K, sa, za, mult, zc);
  ++g_launches;
}

void launch_prepare_relbias(const float* table, int heads, float* out, cudaStream_t st) {
  int n = heads * 4 * 7 * 32 * 4;
  k_prepare_relbias<<<(n + 255) / 256, 256, 0, st>>>(table, heads, out);
  ++g_launches;
}

}  // namespace mixaq
