// Calibration of the activation quantizers (MixA-Q Section 4.3, post-training flow: one calibration sample, and the
// FULL feature map -- every window, not the windows a branch will later see -- initialises the step sizes of both
// branches).  The kernels below run the floating-point Two-Branch block (all quantizers off, weights = code x step)
// through ONE branch's LayerNorm parameters and biases and record the minimum and maximum of what each of the seven
// quantizer sites would see.  Arithmetic: LayerNorm, softmax and GELU exactly as in the quantized path (the same
// device functions); matrix products accumulated in binary64 in index order.  Speed is irrelevant here (the pass
// runs once per model), so the products are plain SIMT loops: one thread per output element.
#include "kernels.h"

namespace mixaq {

namespace {

// order-preserving map float -> unsigned, so that integer atomics give the float minimum / maximum
__device__ __forceinline__ uint32_t ordered_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
// obs[2*site] holds the key of the minimum (starts at 0xFFFFFFFF), obs[2*site+1] that of the maximum (starts at 0)
__device__ __forceinline__ void observe_warp(uint32_t* obs, int site, float lo, float hi) {
  uint32_t klo = ordered_key(lo), khi = ordered_key(hi);
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    klo = min(klo, __shfl_xor_sync(0xffffffffu, klo, off));
    khi = max(khi, __shfl_xor_sync(0xffffffffu, khi, off));
  }
  if ((threadIdx.x & 31) == 0) { atomicMin(obs + 2 * site, klo); atomicMax(obs + 2 * site + 1, khi); }
}

__device__ __forceinline__ int cal_window_src(int b, int H, int W, int Hp, int Wp, int shift, int nwx, int w, int t) {
  const int wy = w / nwx, wx = w - wy * nwx;
  const int i = t / WS, j = t - i * WS;
  int y = wy * WS + i + shift; if (y >= Hp) y -= Hp;
  int x = wx * WS + j + shift; if (x >= Wp) x -= Wp;
  if (y >= H || x >= W) return -1;
  return (b * H + y) * W + x;
}

// Row m of the window batch (all windows of all images in natural order, 49 rows each): source token, LayerNorm of the
// real tokens, zeros for pad tokens.  rowsrc == NULL on input means "rows are already a [M][C] matrix" (LN2).
template <int NPL>
__global__ void __launch_bounds__(256) k_cal_ln(const float* __restrict__ src, int32_t* __restrict__ rowsrc_out,
                                                const float* __restrict__ gamma, const float* __restrict__ beta,
                                                float* __restrict__ out, long M, int gather, int H, int W, int shift,
                                                int nwx, int nW, uint32_t* obs, int site, int site_in) {
  constexpr int C = NPL * 32;
  const long m = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (m >= M) return;
  long s = m;
  if (gather) {
    const int Hp = (H + WS - 1) / WS * WS, Wp = (W + WS - 1) / WS * WS;
    const long slot = m / WT;
    const int t = (int)(m - slot * WT), b = (int)(slot / nW), w = (int)(slot - (long)b * nW);
    s = cal_window_src(b, H, W, Hp, Wp, shift, nwx, w, t);
    if (lane == 0) rowsrc_out[m] = (int32_t)s;
  }
  float v[NPL];
#pragma unroll
  for (int i = 0; i < NPL; ++i) v[i] = s < 0 ? 0.0f : __ldg(src + s * C + lane + 32 * i);
  if (site_in >= 0) {                      // the raw input values of the real tokens (each token sits in one window)
    float ilo = INFINITY, ihi = -INFINITY;
    if (s >= 0) {
#pragma unroll
      for (int i = 0; i < NPL; ++i) { ilo = fminf(ilo, v[i]); ihi = fmaxf(ihi, v[i]); }
    }
    observe_warp(obs, site_in, ilo, ihi);
  }
  float mean, rstd;
  ln_stats<NPL>(v, (float)C, mean, rstd);
  float lo = INFINITY, hi = -INFINITY;
#pragma unroll
  for (int i = 0; i < NPL; ++i) {
    const int c = lane + 32 * i;
    const float y = s < 0 ? 0.0f : ln_apply(v[i], mean, rstd, __ldg(gamma + c), __ldg(beta + c));
    out[m * C + c] = y;
    lo = fminf(lo, y); hi = fmaxf(hi, y);
  }
  observe_warp(obs, site, lo, hi);
}

// patch-merging rows: 2x2 neighbours concatenated (zeros outside the map), LayerNorm over 4C
template <int NPL>
__global__ void __launch_bounds__(256) k_cal_merge_ln(const float* __restrict__ x, const float* __restrict__ gamma,
                                                      const float* __restrict__ beta, float* __restrict__ out,
                                                      int B, int H, int W, uint32_t* obs) {
  constexpr int K = NPL * 32, C = K / 4;
  const int H2 = (H + 1) / 2, W2 = (W + 1) / 2;
  const long tok = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (tok >= (long)B * H2 * W2) return;
  const int b = (int)(tok / ((long)H2 * W2)), r = (int)(tok - (long)b * H2 * W2);
  const int y2 = r / W2, x2 = r - y2 * W2;
  float v[NPL];
#pragma unroll
  for (int i = 0; i < NPL; ++i) {
    const int c = lane + 32 * i, g = c / C, cc = c - g * C;
    const int yy = 2 * y2 + (g & 1), xx = 2 * x2 + (g >> 1);
    v[i] = (yy < H && xx < W) ? __ldg(x + (((long)b * H + yy) * W + xx) * C + cc) : 0.0f;
  }
  float mean, rstd;
  ln_stats<NPL>(v, (float)K, mean, rstd);
  float lo = INFINITY, hi = -INFINITY;
#pragma unroll
  for (int i = 0; i < NPL; ++i) {
    const int c = lane + 32 * i;
    const float y = ln_apply(v[i], mean, rstd, __ldg(gamma + c), __ldg(beta + c));
    out[tok * K + c] = y;
    lo = fminf(lo, y); hi = fmaxf(hi, y);
  }
  observe_warp(obs, 0, lo, hi);
}

// out[m][n] = (float)( sum_k a[m][k] * (w[n][k] * sw[n])  [binary64, k ascending]  + bias[n] ), then per mode:
enum CalMode { CAL_QKV = 0, CAL_PROJ = 1, CAL_FC1 = 2, CAL_FC2 = 3, CAL_PLAIN = 4 };
struct CalLinearArgs {
  const float* a; const int8_t* w; const float* sw; const float* bias;   // bias nullable
  float* out;                 // QKV, FC1, PLAIN: [M][N];  PROJ: x1 [M][N];  FC2: the output feature map
  const float* res;           // PROJ: input feature map (gathered through rowsrc);  FC2: x1 [M][N]
  const int32_t* rowsrc;      // PROJ, FC2
  long M; int N, K, C;        // C: width of one q/k/v section (QKV)
  uint32_t* obs;
};
template <int MODE>
__global__ void __launch_bounds__(256) k_cal_linear(CalLinearArgs p) {
  const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;       // consecutive threads: consecutive n of one row
  const long m = idx / p.N;
  const int n = (int)(idx - m * p.N);
  float lo = INFINITY, hi = -INFINITY;
  if (m < p.M) {
    const float* ar = p.a + m * p.K;
    const int8_t* wr = p.w + (long)n * p.K;
    const double sw = (double)__ldg(p.sw + n);
    double s = 0.0;
    for (int k0 = 0; k0 < p.K; k0 += 16) {                              // K is a multiple of 32
      const int4 wv = __ldg(reinterpret_cast<const int4*>(wr + k0));
      const int words[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int code = (int)(int8_t)(words[j >> 2] >> (8 * (j & 3)));
        s = __dadd_rn(s, __dmul_rn((double)__ldg(ar + k0 + j), __dmul_rn((double)code, sw)));
      }
    }
    float v = (float)__dadd_rn(s, p.bias ? (double)__ldg(p.bias + n) : 0.0);
    if (MODE == CAL_QKV) {
      p.out[m * p.N + n] = v;
      lo = hi = v;
    } else if (MODE == CAL_PROJ) {
      const long src = p.rowsrc[m];
      const float xin = src >= 0 ? __ldg(p.res + src * p.N + n) : 0.0f;
      p.out[m * p.N + n] = __fadd_rn(xin, v);
    } else if (MODE == CAL_FC1) {
      v = gelu_f2(make_float2(v, v)).x;
      p.out[m * p.N + n] = v;
      lo = hi = v;
    } else if (MODE == CAL_FC2) {
      const long src = p.rowsrc[m];
      if (src >= 0) p.out[src * p.N + n] = __fadd_rn(__ldg(p.res + m * p.N + n), v);
    } else {
      p.out[m * p.N + n] = v;
    }
  }
  if (MODE == CAL_QKV) {
    // a warp may straddle two sections (or two rows): every lane reports to its own section
    const int sec = m < p.M ? n / p.C : 0;
#pragma unroll
    for (int q = 0; q < 3; ++q) {
      const bool mine = m < p.M && sec == q;
      observe_warp(p.obs, 1 + q, mine ? lo : INFINITY, mine ? hi : -INFINITY);
    }
  } else if (MODE == CAL_FC1) {
    observe_warp(p.obs, 6, lo, hi);
  }
}

// softmax of the numeric contract over 49 logits: exact maximum, exponentials through 2^t, four interleaved partial
// sums (column j of the 8-wide group j/8 goes to partial (j mod 8)/2, in increasing j), (p0+p1)+(p2+p3), one division
__device__ __forceinline__ void softmax49(float (&s)[WT]) {
  float mx = s[0];
#pragma unroll
  for (int j = 1; j < WT; ++j) mx = fmaxf(mx, s[j]);
#pragma unroll
  for (int j = 0; j < WT; ++j) {
    const float t = fmaxf(__fmul_rn(__fsub_rn(s[j], mx), 1.44269504088896340736f), -125.0f);
    s[j] = exp2_core2(make_float2(t, t)).x;
  }
  float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int t = 0; t < 4; ++t)
#pragma unroll
    for (int grp = 0; grp * 8 < WT; ++grp)
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int j = grp * 8 + 2 * t + u;
        if (j < WT) part[t] = __fadd_rn(part[t], s[j]);
      }
  const float inv = __fdiv_rn(1.0f, __fadd_rn(__fadd_rn(part[0], part[1]), __fadd_rn(part[2], part[3])));
#pragma unroll
  for (int j = 0; j < WT; ++j) s[j] = __fmul_rn(s[j], inv);
}

// one thread per (window slot, head, query row): logits in binary64, softmax of the contract, P.V in binary64
struct CalAttnArgs {
  const float* qkv; const float* relpos; float* o;
  long slots; int C, heads, shift, Hp, Wp, nwx, nW;
  uint32_t* obs;
};
__global__ void __launch_bounds__(128) k_cal_attention(CalAttnArgs a) {
  const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const long total = a.slots * a.heads * WT;
  float lo = INFINITY, hi = -INFINITY;
  if (idx < total) {
    const int i = (int)(idx % WT);
    const int h = (int)((idx / WT) % a.heads);
    const long slot = idx / ((long)WT * a.heads);
    const int w = (int)(slot % a.nW), wy = w / a.nwx, wx = w - wy * a.nwx;
    const int C = a.C;
    const float* base = a.qkv + slot * WT * 3 * C;
    const float* q = base + (long)i * 3 * C + h * HEAD_DIM;
    auto region = [&](int pos, int L) { return pos < L - WS ? 0 : (pos < L - a.shift ? 1 : 2); };
    const int ri = region(wy * WS + i / WS, a.Hp) * 3 + region(wx * WS + i % WS, a.Wp);
    const double rs = 1.0 / sqrt((double)HEAD_DIM);
    float s[WT];
    for (int j = 0; j < WT; ++j) {
      const float* k = base + (long)j * 3 * C + C + h * HEAD_DIM;
      double d = 0.0;
      for (int e = 0; e < HEAD_DIM; ++e) d = __dadd_rn(d, __dmul_rn((double)__ldg(q + e), (double)__ldg(k + e)));
      const int ridx = (i / WS - j / WS + WS - 1) * (2 * WS - 1) + (i % WS - j % WS + WS - 1);
      double maskv = 0.0;
      if (a.shift > 0) {
        const int rj = region(wy * WS + j / WS, a.Hp) * 3 + region(wx * WS + j % WS, a.Wp);
        maskv = rj == ri ? 0.0 : -100.0;
      }
      s[j] = (float)__dadd_rn(__dadd_rn(__dmul_rn(d, rs), (double)__ldg(a.relpos + (long)ridx * a.heads + h)), maskv);
    }
    softmax49(s);
    float* orow = a.o + (slot * WT + i) * C + h * HEAD_DIM;
    for (int e = 0; e < HEAD_DIM; ++e) {
      double d = 0.0;
      for (int j = 0; j < WT; ++j)
        d = __dadd_rn(d, __dmul_rn((double)s[j], (double)__ldg(base + (long)j * 3 * C + 2 * C + h * HEAD_DIM + e)));
      const float v = (float)d;
      orow[e] = v;
      lo = fminf(lo, v); hi = fmaxf(hi, v);
    }
  }
  observe_warp(a.obs, 4, lo, hi);
}

__global__ void k_cal_obs_init(uint32_t* obs, int sites) {
  const int i = threadIdx.x;
  if (i < 2 * sites) obs[i] = (i & 1) ? 0u : 0xFFFFFFFFu;
}

template <int MODE>
void launch_cal_linear(const CalLinearArgs& p, cudaStream_t st) {
  const long total = p.M * p.N;
  if (total == 0) return;
  k_cal_linear<MODE><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(p);
  ++g_launches;
}

}  // namespace

// keys written by the observers -> floats (host side)
float cal_key_to_float(uint32_t key) {
  const uint32_t u = (key & 0x80000000u) ? (key & 0x7FFFFFFFu) : ~key;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

#define MIXAQ_CAL_LN_CASE(n) case n: k_cal_ln<n><<<grid, 256, 0, st>>>(src, rowsrc_out, gamma, beta, out, M, gather, H, W, shift, nwx, nW, obs, site, site_in); break;
static bool launch_cal_ln(const float* src, int32_t* rowsrc_out, const float* gamma, const float* beta, float* out, long M,
                          int C, int gather, int H, int W, int shift, int nwx, int nW, uint32_t* obs, int site, int site_in, cudaStream_t st) {
  const unsigned grid = (unsigned)((M + 7) / 8);
  switch (C / 32) {
    MIXAQ_CAL_LN_CASE(1) MIXAQ_CAL_LN_CASE(2) MIXAQ_CAL_LN_CASE(3) MIXAQ_CAL_LN_CASE(4) MIXAQ_CAL_LN_CASE(6) MIXAQ_CAL_LN_CASE(8)
    MIXAQ_CAL_LN_CASE(12) MIXAQ_CAL_LN_CASE(16) MIXAQ_CAL_LN_CASE(24) MIXAQ_CAL_LN_CASE(32)
    default: return false;
  }
  ++g_launches;
  return true;
}

// The floating-point block through one branch.  Workspace (floats unless noted): rowsrc int32[M], ln [M][C],
// qkv [M][3C], o [M][C], x1 [M][C], h [M][hidden]; obs: 16 keys (seven sites and the block's input map).
bool launch_calibrate_block(const CalBlockArgs& c, cudaStream_t st) {
  const int C = c.C, Hd = c.hidden;
  const int Hp = (c.H + WS - 1) / WS * WS, Wp = (c.W + WS - 1) / WS * WS, nwx = Wp / WS, nW = (Hp / WS) * nwx;
  const long slots = (long)c.B * nW, M = slots * WT;
  k_cal_obs_init<<<1, 32, 0, st>>>(c.obs, 8);
  ++g_launches;
  if (!launch_cal_ln(c.x, c.rowsrc, c.ln1_g, c.ln1_b, c.ln, M, C, 1, c.H, c.W, c.shift, nwx, nW, c.obs, 0, 7, st)) return false;
  CalLinearArgs l;
  l.obs = c.obs; l.M = M; l.C = C; l.rowsrc = c.rowsrc;
  l.a = c.ln; l.w = c.w_qkv; l.sw = c.s_qkv; l.bias = c.b_qkv; l.out = c.qkv; l.res = nullptr; l.N = 3 * C; l.K = C;
  launch_cal_linear<CAL_QKV>(l, st);
  CalAttnArgs a;
  a.qkv = c.qkv; a.relpos = c.relpos; a.o = c.o; a.slots = slots; a.C = C; a.heads = c.heads; a.shift = c.shift;
  a.Hp = Hp; a.Wp = Wp; a.nwx = nwx; a.nW = nW; a.obs = c.obs;
  const long athreads = slots * c.heads * WT;
  k_cal_attention<<<(unsigned)((athreads + 127) / 128), 128, 0, st>>>(a);
  ++g_launches;
  l.a = c.o; l.w = c.w_proj; l.sw = c.s_proj; l.bias = c.b_proj; l.out = c.x1; l.res = c.x; l.N = C; l.K = C;
  launch_cal_linear<CAL_PROJ>(l, st);
  if (!launch_cal_ln(c.x1, nullptr, c.ln2_g, c.ln2_b, c.ln, M, C, 0, c.H, c.W, c.shift, nwx, nW, c.obs, 5, -1, st)) return false;
  l.a = c.ln; l.w = c.w_fc1; l.sw = c.s_fc1; l.bias = c.b_fc1; l.out = c.h; l.res = nullptr; l.N = Hd; l.K = C;
  launch_cal_linear<CAL_FC1>(l, st);
  l.a = c.h; l.w = c.w_fc2; l.sw = c.s_fc2; l.bias = c.b_fc2; l.out = c.y; l.res = c.x1; l.N = C; l.K = Hd;
  launch_cal_linear<CAL_FC2>(l, st);
  return true;
}

#define MIXAQ_CAL_MERGE_CASE(n) case n: k_cal_merge_ln<n><<<grid, 256, 0, st>>>(c.x, c.ln_g, c.ln_b, c.ln, c.B, c.H, c.W, c.obs); break;
bool launch_calibrate_merge(const CalMergeArgs& c, cudaStream_t st) {
  const long M = (long)c.B * ((c.H + 1) / 2) * ((c.W + 1) / 2);
  k_cal_obs_init<<<1, 32, 0, st>>>(c.obs, 1);
  ++g_launches;
  const unsigned grid = (unsigned)((M + 7) / 8);
  switch (4 * c.C / 32) {
    MIXAQ_CAL_MERGE_CASE(4) MIXAQ_CAL_MERGE_CASE(8) MIXAQ_CAL_MERGE_CASE(12) MIXAQ_CAL_MERGE_CASE(16) MIXAQ_CAL_MERGE_CASE(24)
    MIXAQ_CAL_MERGE_CASE(32) MIXAQ_CAL_MERGE_CASE(48) MIXAQ_CAL_MERGE_CASE(64)
    default: return false;
  }
  ++g_launches;
  CalLinearArgs l;
  l.obs = c.obs; l.M = M; l.C = c.N; l.rowsrc = nullptr; l.res = nullptr;
  l.a = c.ln; l.w = c.w; l.sw = c.sw; l.bias = nullptr; l.out = c.y; l.N = c.N; l.K = 4 * c.C;
  launch_cal_linear<CAL_PLAIN>(l, st);
  return true;
}

}  // namespace mixaq
