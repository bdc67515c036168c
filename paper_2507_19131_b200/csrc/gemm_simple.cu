// Plain integer GEMM (dp4a) with the fused epilogues: one thread per output row, 32 columns per CTA.
// Bring-up and cross-check path for the tensor-core kernel; same epilogue code, same results.
#include "gemm_epilogue.cuh"

namespace mixaq {

__device__ __forceinline__ int dp4a_us(uint32_t a, uint32_t b, int c) {
  int d;
  asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

template <int MODE>
__global__ void __launch_bounds__(128) k_gemm_simple(GemmArgs g, int tiles_hi) {
  __shared__ uint32_t s_w[32][8];              // 32 columns x 32 k-bytes
  const bool is_hi = (int)blockIdx.x < tiles_hi;
  const GemmBranch& br = is_hi ? g.br[0] : g.br[1];
  const int tile = is_hi ? blockIdx.x : blockIdx.x - tiles_hi;
  const long m = (long)tile * 128 + threadIdx.x;
  const int n0 = blockIdx.y * 32;
  const bool valid = m < br.M;
  const int abits = br.a_bits;
  const long a_stride = (long)g.K * abits / 8;
  int32_t acc[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) acc[i] = 0;
  for (int kg = 0; kg < g.K / 32; ++kg) {
    __syncthreads();
    for (int i = threadIdx.x; i < 256; i += 128) {
      int n = i >> 3, wq = i & 7;
      s_w[n][wq] = *reinterpret_cast<const uint32_t*>(g.w + (long)(n0 + n) * g.K + kg * 32 + wq * 4);
    }
    __syncthreads();
    uint32_t aw[8];
    if (valid) load_codes_32(br.a + m * a_stride + (long)kg * 32 * abits / 8, abits, aw);
    else {
#pragma unroll
      for (int i = 0; i < 8; ++i) aw[i] = 0;
    }
#pragma unroll
    for (int n = 0; n < 32; ++n)
#pragma unroll
      for (int q = 0; q < 8; ++q) acc[n] = dp4a_us(aw[q], s_w[n][q], acc[n]);
  }
  if (valid) epilogue_row32<MODE>(br, g.N, g.C, m, n0, acc);
}

void launch_gemm_simple(const GemmArgs& g, cudaStream_t st) {
  int tiles_hi = (g.br[0].M + 127) / 128, tiles_lo = (g.br[1].M + 127) / 128;
  if (tiles_hi + tiles_lo == 0) return;
  dim3 grid(tiles_hi + tiles_lo, g.N / 32);
  switch (g.mode) {
    case EPI_QKV:   k_gemm_simple<EPI_QKV><<<grid, 128, 0, st>>>(g, tiles_hi); break;
    case EPI_PROJ:  k_gemm_simple<EPI_PROJ><<<grid, 128, 0, st>>>(g, tiles_hi); break;
    case EPI_FC1:   k_gemm_simple<EPI_FC1><<<grid, 128, 0, st>>>(g, tiles_hi); break;
    case EPI_FC2:   k_gemm_simple<EPI_FC2><<<grid, 128, 0, st>>>(g, tiles_hi); break;
    case EPI_MERGE: k_gemm_simple<EPI_MERGE><<<grid, 128, 0, st>>>(g, tiles_hi); break;
  }
  ++g_launches;
}

void launch_gemm(const GemmArgs& g, cudaStream_t st) { launch_gemm_simple(g, st); }

}  // namespace mixaq
