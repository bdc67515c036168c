// Fused window attention of one branch batch (MixA-Q Section 3.1: multi-head self-attention inside each
// non-overlapping 7x7 window; Figure 2a "Attn High" / "Attn Low"):
//   S_int = (q - z_q)(k - z_k)^T  (int32)  ->  S = fma(S_int, s_q*s_k/sqrt(d), relpos_bias) [+ shift mask]
//   P = softmax_row(S) in binary32  ->  P codes (unsigned, step 1/(2^b-1))
//   O_int = P_codes (v - z_v) (int32)  ->  O = O_int * s_p*s_v  ->  codes of the proj input quantizer.
// One CTA per (window slot, head); thread i owns query row i.
#include "kernels.h"

namespace mixaq {

__device__ __forceinline__ int dp4a_uu(uint32_t a, uint32_t b, int c) {
  int d;
  asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

__device__ __forceinline__ int shift_region(int pos, int L, int shift) {
  return pos < L - WS ? 0 : (pos < L - shift ? 1 : 2);
}

__global__ void __launch_bounds__(64) k_attention(AttnArgs a) {
  __shared__ uint32_t s_q[WT][8], s_k[WT][8], s_v[WT][8];
  __shared__ int s_reg[WT], s_ksum[WT];
  const int slots_hi = a.br[0].slots;
  int slot = blockIdx.x / a.heads, h = blockIdx.x - slot * a.heads;
  const bool is_hi = slot < slots_hi;
  const AttnBranch& br = is_hi ? a.br[0] : a.br[1];
  if (!is_hi) slot -= slots_hi;
  const int bits = br.bits, C = a.C;
  const long row_bytes = (long)3 * C * bits / 8;
  const int tid = threadIdx.x;

  // stage q, k, v of this head (32 codes each per token), unpacked to bytes
  for (int i = tid; i < 3 * WT; i += blockDim.x) {
    int sec = i / WT, t = i - sec * WT;
    const uint8_t* src = br.qkv + ((long)slot * WT + t) * row_bytes + (long)(sec * C + h * HEAD_DIM) * bits / 8;
    uint32_t w[8];
    load_codes_32(src, bits, w);
    uint32_t (*dst)[8] = sec == 0 ? s_q : (sec == 1 ? s_k : s_v);
#pragma unroll
    for (int e = 0; e < 8; ++e) dst[t][e] = w[e];
  }
  if (tid < WT) {
    int reg = 0;
    if (a.shift > 0) {
      int w = br.win[slot];
      int wy = w / a.nwx, wx = w - wy * a.nwx;
      int i = tid / WS, j = tid - i * WS;
      reg = shift_region(wy * WS + i, a.Hp, a.shift) * 3 + shift_region(wx * WS + j, a.Wp, a.shift);
    }
    s_reg[tid] = reg;
  }
  __syncthreads();
  if (tid < WT) {
    int ks = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) ks = dp4a_uu(s_k[tid][e], 0x01010101u, ks);
    s_ksum[tid] = ks;
  }
  __syncthreads();
  if (tid >= WT) return;

  const int i = tid;
  const int zq = br.q.zp, zk = br.k.zp, zv = br.v.zp;
  uint32_t qw[8];
  int qsum = 0;
#pragma unroll
  for (int e = 0; e < 8; ++e) { qw[e] = s_q[i][e]; qsum = dp4a_uu(qw[e], 0x01010101u, qsum); }
  const float* relb = a.relbias + ((long)h * WT + i) * WT;
  const int my_reg = s_reg[i];
  float lg[WT];
  float mx = -3.0e38f;
#pragma unroll
  for (int j = 0; j < WT; ++j) {
    int dot = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) dot = dp4a_uu(qw[e], s_k[j][e], dot);
    int s_int = dot - zk * qsum - zq * s_ksum[j] + HEAD_DIM * zq * zk;
    float v = __fmaf_rn(__int2float_rn(s_int), br.alpha, __ldg(relb + j));
    if (a.shift > 0) v = __fadd_rn(v, s_reg[j] != my_reg ? -100.0f : 0.0f);
    lg[j] = v;
    mx = fmaxf(mx, v);
  }
  const float kLog2e = 1.44269504088896340736f;
#pragma unroll
  for (int j = 0; j < WT; ++j) lg[j] = exp2_core(fmaxf(__fmul_rn(__fsub_rn(lg[j], mx), kLog2e), -125.0f));
  // sum: four interleaved partials (columns 8g+2t, 8g+2t+1 -> partial t), then (p0+p1)+(p2+p3)
  float part[4];
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    float p = 0.0f;
#pragma unroll
    for (int g = 0; g < 7; ++g)
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        int j = 8 * g + 2 * t + u;
        if (j < WT) p = __fadd_rn(p, lg[j]);
      }
    part[t] = p;
  }
  float sum = __fadd_rn(__fadd_rn(part[0], part[1]), __fadd_rn(part[2], part[3]));
  float inv = __fdiv_rn(1.0f, sum);
  const int pmax = (1 << bits) - 1;
  AQ pq; pq.scale = 0.f; pq.inv_scale = (float)pmax; pq.zpf = 0.0f; pq.qmaxf = (float)pmax; pq.zp = 0; pq.bits = bits;
  uint32_t pc[WT];
  int psum = 0;
#pragma unroll
  for (int j = 0; j < WT; ++j) { pc[j] = quant_code(__fmul_rn(lg[j], inv), pq); psum += (int)pc[j]; }
  if (br.tap_p) {
    uint8_t* tp = br.tap_p + (((long)slot * a.heads + h) * WT + i) * WT;
#pragma unroll
    for (int j = 0; j < WT; ++j) tp[j] = (uint8_t)pc[j];
  }
  int o_int[HEAD_DIM];
#pragma unroll
  for (int e = 0; e < HEAD_DIM; ++e) o_int[e] = -zv * psum;
#pragma unroll
  for (int j = 0; j < WT; ++j) {
#pragma unroll
    for (int e8 = 0; e8 < 8; ++e8) {
      uint32_t vw = s_v[j][e8];
#pragma unroll
      for (int b = 0; b < 4; ++b) o_int[e8 * 4 + b] += (int)pc[j] * (int)((vw >> (8 * b)) & 0xFFu);
    }
  }
  const long m = (long)slot * WT + i;
  if (br.tap_pv) {
#pragma unroll
    for (int e = 0; e < HEAD_DIM; ++e) br.tap_pv[m * C + h * HEAD_DIM + e] = o_int[e];
  }
  uint32_t oc[32];
  AQ oq = br.o;
#pragma unroll
  for (int e = 0; e < HEAD_DIM; ++e) oc[e] = quant_code(__fmul_rn(__int2float_rn(o_int[e]), br.so), oq);
  store_codes_32(br.out + m * ((long)C * bits / 8) + (long)h * HEAD_DIM * bits / 8, oc, bits);
}

void launch_attention(const AttnArgs& a, cudaStream_t st) {
  int slots = a.br[0].slots + a.br[1].slots;
  if (slots == 0) return;
  k_attention<<<slots * a.heads, 64, 0, st>>>(a);
  ++g_launches;
}

}  // namespace mixaq
