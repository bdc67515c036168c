// One-time derived tables of a block: per-output-channel step-size products and zero-point corrections of
// every (linear layer, branch) pair, and the relative-position bias expanded to [heads][49][49].
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

// bias[h][i][j] = table[((yi - yj + 6) * 13 + (xi - xj + 6)) * heads + h]
__global__ void k_prepare_relbias(const float* __restrict__ table, int heads, float* out) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= heads * WT * WT) return;
  int h = idx / (WT * WT), r = idx - h * WT * WT;
  int i = r / WT, j = r - i * WT;
  int dy = i / WS - j / WS + (WS - 1), dx = i % WS - j % WS + (WS - 1);
  out[idx] = table[(dy * (2 * WS - 1) + dx) * heads + h];
}

void launch_prepare_linear(const int8_t* w, const float* sw, int N, int K, float sa, int za, float* mult,
                           int32_t* zc, cudaStream_t st) {
  k_prepare_linear<<<(N + 7) / 8, 256, 0, st>>>(w, sw, N, K, sa, za, mult, zc);
  ++g_launches;
}

void launch_prepare_relbias(const float* table, int heads, float* out, cudaStream_t st) {
  int n = heads * WT * WT;
  k_prepare_relbias<<<(n + 255) / 256, 256, 0, st>>>(table, heads, out);
  ++g_launches;
}

}  // namespace mixaq
