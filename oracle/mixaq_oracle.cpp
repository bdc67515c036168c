// Oracle for the quantized Two-Branch Swin Block forward (MixA-Q, Sections 3.1, 3.2, 3.4).
// TEST INFRASTRUCTURE ONLY: a plain, slow, one-window-at-a-time CPU program.  See mixaq_oracle.h.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -mfma -fopenmp -shared -fPIC  (no fast-math: every binary32
// operation below must round exactly once, and only std::fmaf may fuse).
#include "mixaq_oracle.h"
#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline int   f2i(float f) { int i; std::memcpy(&i, &f, 4); return i; }
inline float i2f(int i)   { float f; std::memcpy(&f, &i, 4); return f; }
inline float bitsf(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

// ---------------------------------------------------------------------------------------------
// Numeric contract, scalar pieces.
// ---------------------------------------------------------------------------------------------

// 2^t for t in [-125, 0] (used for t <= 0): round-to-nearest split t = n + f, |f| <= 1/2, a degree-5
// polynomial for 2^f evaluated by Horner with fused multiply-adds, then n is added to the exponent field.
const float kExp2C[6] = { bitsf(0x3f800001u), bitsf(0x3f317219u), bitsf(0x3e75fc83u),
                          bitsf(0x3d635716u), bitsf(0x3c1e883du), bitsf(0x3aafc47du) };
const float kMagic = 12582912.0f;   // 1.5 * 2^23: adding it rounds a small float to the nearest integer

inline float exp2_core(float t) {
  float r  = t + kMagic;
  float nf = r - kMagic;
  float f  = t - nf;
  float p  = kExp2C[5];
  for (int k = 4; k >= 0; --k) p = std::fmaf(p, f, kExp2C[k]);
  uint32_t bits = (uint32_t)f2i(p) + ((uint32_t)f2i(r) << 23);
  return bitsf(bits);
}
inline float exp2_clamped(float t) { return exp2_core(std::fmax(t, -125.0f)); }

// GELU(v) = v * Phi(v) = max(v, 0) - a * Phi(-a), a = |v|.  log2 Phi(-a) is a degree-7 polynomial on
// [0, 5]; beyond 5 the correction a*Phi(-a) < 1.5e-6 is held at its value at 5.
const float kGeluQ[8] = { bitsf(0xbf7fffbeu), bitsf(0xbf935b8fu), bitsf(0xbeeac5d4u), bitsf(0xbd5c93e3u),
                          bitsf(0x3c0a3aedu), bitsf(0xba6dcc74u), bitsf(0x38729e20u), bitsf(0xb5d6f9e3u) };
inline float gelu1(float v) {
  float a = std::fmin(std::fabs(v), 5.0f);
  float q = kGeluQ[7];
  for (int k = 6; k >= 0; --k) q = std::fmaf(q, a, kGeluQ[k]);
  float h = a * exp2_core(q);
  return std::fmax(v, 0.0f) - h;
}

inline uint8_t quant1(float x, const orc_aq& q) {
  float t = x * q.inv_scale;
  float r = std::nearbyintf(t);                 // round half to even (default rounding mode)
  float c = r + (float)q.zp;
  float qmax = (float)((1 << q.bits) - 1);
  c = std::fmin(std::fmax(c, 0.0f), qmax);
  return (uint8_t)c;
}

// Sum of n floats as 32 interleaved partial sums (element c goes to partial c mod 32, in increasing c)
// followed by a 5-level butterfly (offsets 16, 8, 4, 2, 1).
template <class F> inline float sum32(int n, F term) {
  float p[32];
  for (int l = 0; l < 32; ++l) {
    float s = 0.0f;
    for (int c = l; c < n; c += 32) s = term(c, s);
    p[l] = s;
  }
  for (int off = 16; off >= 1; off >>= 1) {
    float t[32];
    for (int l = 0; l < 32; ++l) t[l] = p[l] + p[l ^ off];
    std::memcpy(p, t, sizeof(p));
  }
  return p[0];
}

void layernorm_row(const float* x, int C, const float* g, const float* b, float* y) {
  float fC = (float)C;
  float mean = sum32(C, [&](int c, float s) { return s + x[c]; }) / fC;
  float var  = sum32(C, [&](int c, float s) { float d = x[c] - mean; return std::fmaf(d, d, s); }) / fC;
  float rstd = 1.0f / std::sqrt(var + 1e-5f);
  for (int c = 0; c < C; ++c) {
    float d = x[c] - mean;
    y[c] = std::fmaf(d * rstd, g[c], b[c]);
  }
}

// softmax over T logits: exact max, exponentials through exp2_clamped, sum as 4 interleaved partials
// (column j of the 8-wide group j/8 goes to partial (j mod 8)/2) then (p0+p1)+(p2+p3), one division.
void softmax_row(const float* s, int T, float* p) {
  const float kLog2e = 1.44269504088896340736f;
  float m = s[0];
  for (int j = 1; j < T; ++j) m = std::fmax(m, s[j]);
  float part[4] = {0.f, 0.f, 0.f, 0.f};
  std::vector<float> e(T);
  for (int j = 0; j < T; ++j) e[j] = exp2_clamped((s[j] - m) * kLog2e);
  for (int t = 0; t < 4; ++t)
    for (int grp = 0; grp * 8 < T; ++grp)
      for (int u = 0; u < 2; ++u) {
        int j = grp * 8 + 2 * t + u;
        if (j < T) part[t] = part[t] + e[j];
      }
  float sum = (part[0] + part[1]) + (part[2] + part[3]);
  float inv = 1.0f / sum;
  for (int j = 0; j < T; ++j) p[j] = e[j] * inv;
}

// ---------------------------------------------------------------------------------------------
// Geometry: windows, cyclic shift, padding (Section 3.1: non-overlapping windows; shifted blocks).
// ---------------------------------------------------------------------------------------------
inline int round_up(int a, int m) { return (a + m - 1) / m * m; }

long window_token(int H, int W, int ws, int shift, int w, int t) {
  int Hp = round_up(H, ws), Wp = round_up(W, ws);
  int nwx = Wp / ws;
  int wy = w / nwx, wx = w % nwx;
  int i = t / ws, j = t % ws;
  int ys = wy * ws + i, xs = wx * ws + j;          // coordinates in the shifted frame
  int y = (ys + shift) % Hp, x = (xs + shift) % Wp; // source coordinates in the padded map
  if (y >= H || x >= W) return -1;
  return (long)y * W + x;
}

inline int region_of(int pos, int L, int ws, int shift) {   // position in the shifted frame
  if (pos < L - ws) return 0;
  if (pos < L - shift) return 1;
  return 2;
}

void shift_mask(int H, int W, int ws, int shift, int w, float* mask) {
  int T = ws * ws;
  if (shift == 0) { std::fill(mask, mask + T * T, 0.0f); return; }
  int Hp = round_up(H, ws), Wp = round_up(W, ws);
  int nwx = Wp / ws;
  int wy = w / nwx, wx = w % nwx;
  std::vector<int> reg(T);
  for (int t = 0; t < T; ++t) {
    int ys = wy * ws + t / ws, xs = wx * ws + t % ws;
    reg[t] = region_of(ys, Hp, ws, shift) * 3 + region_of(xs, Wp, ws, shift);
  }
  for (int i = 0; i < T; ++i)
    for (int j = 0; j < T; ++j) mask[i * T + j] = (reg[i] == reg[j]) ? 0.0f : -100.0f;
}

void relpos_bias(const float* table, int ws, int heads, float* bias) {
  int T = ws * ws;
  for (int h = 0; h < heads; ++h)
    for (int i = 0; i < T; ++i)
      for (int j = 0; j < T; ++j) {
        int dy = i / ws - j / ws + (ws - 1);
        int dx = i % ws - j % ws + (ws - 1);
        bias[((long)h * T + i) * T + j] = table[(long)(dy * (2 * ws - 1) + dx) * heads + h];
      }
}

// ---------------------------------------------------------------------------------------------
// One window through one branch.
// ---------------------------------------------------------------------------------------------
struct WinTaps {   // destination row/window offsets inside the tap buffers
  const orc_taps* t; long row0; long win;
};

// integer linear layer on unsigned codes: acc[m][n] = sum_k (a[m][k] - za) * w[n][k]
void int_linear(const uint8_t* a, int M, int K, int za, const orc_linear& L, int32_t* acc) {
  for (int m = 0; m < M; ++m)
    for (int n = 0; n < L.out_f; ++n) {
      int64_t s = 0;
      const int8_t* wr = L.codes + (long)n * K;
      const uint8_t* ar = a + (long)m * K;
      for (int k = 0; k < K; ++k) s += (int64_t)((int)ar[k] - za) * (int)wr[k];
      acc[(long)m * L.out_f + n] = (int32_t)s;
    }
}

inline float dequant_bias(int32_t acc, float sa, float sw, float bias) {
  return std::fmaf((float)acc, sa * sw, bias);
}

void window_forward_quant(const orc_block& P, const orc_branch& br, const float* relb, const float* mask,
                          const float* xin /*[T][C], pad rows = 0*/, const uint8_t* real /*[T]*/,
                          float* yout /*[T][C]*/, const WinTaps* wt) {
  const int C = P.dim, T = P.window * P.window, nh = P.heads, d = C / nh, Hd = P.hidden;
  std::vector<float> ln((long)T * C);
  std::vector<uint8_t> a((long)T * C);
  // LN1 on real tokens; pad tokens are zero after normalisation
  for (int t = 0; t < T; ++t) {
    if (real[t]) layernorm_row(xin + (long)t * C, C, br.ln1_g, br.ln1_b, &ln[(long)t * C]);
    else std::fill(&ln[(long)t * C], &ln[(long)(t + 1) * C], 0.0f);
  }
  orc_quantize(ln.data(), (long)T * C, br.qkv_in, a.data());
  // QKV
  std::vector<int32_t> acc((long)T * 3 * C);
  int_linear(a.data(), T, C, br.qkv_in.zp, P.qkv, acc.data());
  std::vector<uint8_t> qkv((long)T * 3 * C);
  for (int t = 0; t < T; ++t)
    for (int n = 0; n < 3 * C; ++n) {
      float v = dequant_bias(acc[(long)t * 3 * C + n], br.qkv_in.scale, P.qkv.scale[n], br.b_qkv[n]);
      const orc_aq& qz = (n < C) ? br.q : (n < 2 * C ? br.k : br.v);
      qkv[(long)t * 3 * C + n] = quant1(v, qz);
    }
  // attention per head
  const float rs = (float)(1.0 / std::sqrt((double)d));
  const float alpha = (br.q.scale * br.k.scale) * rs;
  const int   pmax = (1 << br.bits) - 1;
  const orc_aq pq = { br.bits, 1.0f / (float)pmax, (float)pmax, 0 };
  const float so = pq.scale * br.v.scale;
  std::vector<int32_t> pv((long)T * C);
  std::vector<float> logits(T), prob(T);
  std::vector<uint8_t> pc(T);
  for (int h = 0; h < nh; ++h)
    for (int i = 0; i < T; ++i) {
      for (int j = 0; j < T; ++j) {
        int32_t s = 0;
        for (int e = 0; e < d; ++e)
          s += ((int)qkv[(long)i * 3 * C + h * d + e] - br.q.zp) * ((int)qkv[(long)j * 3 * C + C + h * d + e] - br.k.zp);
        float lg = std::fmaf((float)s, alpha, relb[((long)h * T + i) * T + j]);
        if (mask) lg = lg + mask[i * T + j];
        logits[j] = lg;
      }
      softmax_row(logits.data(), T, prob.data());
      orc_quantize(prob.data(), T, pq, pc.data());
      for (int e = 0; e < d; ++e) {
        int32_t s = 0;
        for (int j = 0; j < T; ++j) s += (int)pc[j] * ((int)qkv[(long)j * 3 * C + 2 * C + h * d + e] - br.v.zp);
        pv[(long)i * C + h * d + e] = s;
      }
      if (wt && wt->t->probs)   std::memcpy(wt->t->probs + ((wt->win * nh + h) * T + i) * T, prob.data(), T * sizeof(float));
      if (wt && wt->t->p_codes) std::memcpy(wt->t->p_codes + ((wt->win * nh + h) * T + i) * T, pc.data(), T);
    }
  std::vector<uint8_t> o((long)T * C);
  for (long e = 0; e < (long)T * C; ++e) o[e] = quant1((float)pv[e] * so, br.proj_in);
  // proj + residual
  std::vector<int32_t> pacc((long)T * C);
  int_linear(o.data(), T, C, br.proj_in.zp, P.proj, pacc.data());
  std::vector<float> x1((long)T * C);
  for (int t = 0; t < T; ++t)
    for (int n = 0; n < C; ++n)
      x1[(long)t * C + n] = xin[(long)t * C + n] +
                            dequant_bias(pacc[(long)t * C + n], br.proj_in.scale, P.proj.scale[n], br.b_proj[n]);
  // LN2 -> fc1 -> GELU -> fc2 + residual
  std::vector<uint8_t> f1((long)T * C);
  for (int t = 0; t < T; ++t) layernorm_row(&x1[(long)t * C], C, br.ln2_g, br.ln2_b, &ln[(long)t * C]);
  orc_quantize(ln.data(), (long)T * C, br.fc1_in, f1.data());
  std::vector<int32_t> a1((long)T * Hd);
  int_linear(f1.data(), T, C, br.fc1_in.zp, P.fc1, a1.data());
  std::vector<uint8_t> f2((long)T * Hd);
  for (int t = 0; t < T; ++t)
    for (int n = 0; n < Hd; ++n) {
      float v = dequant_bias(a1[(long)t * Hd + n], br.fc1_in.scale, P.fc1.scale[n], br.b_fc1[n]);
      f2[(long)t * Hd + n] = quant1(gelu1(v), br.fc2_in);
    }
  std::vector<int32_t> a2((long)T * C);
  int_linear(f2.data(), T, Hd, br.fc2_in.zp, P.fc2, a2.data());
  for (int t = 0; t < T; ++t)
    for (int n = 0; n < C; ++n)
      yout[(long)t * C + n] = x1[(long)t * C + n] +
                              dequant_bias(a2[(long)t * C + n], br.fc2_in.scale, P.fc2.scale[n], br.b_fc2[n]);
  if (wt) {
    const orc_taps* tp = wt->t; long r0 = wt->row0;
    if (tp->a_codes)   std::memcpy(tp->a_codes + r0 * C, a.data(), (long)T * C);
    if (tp->qkv_acc)   std::memcpy(tp->qkv_acc + r0 * 3 * C, acc.data(), (long)T * 3 * C * 4);
    if (tp->qkv_codes) std::memcpy(tp->qkv_codes + r0 * 3 * C, qkv.data(), (long)T * 3 * C);
    if (tp->pv_acc)    std::memcpy(tp->pv_acc + r0 * C, pv.data(), (long)T * C * 4);
    if (tp->o_codes)   std::memcpy(tp->o_codes + r0 * C, o.data(), (long)T * C);
    if (tp->proj_acc)  std::memcpy(tp->proj_acc + r0 * C, pacc.data(), (long)T * C * 4);
    if (tp->x1)        std::memcpy(tp->x1 + r0 * C, x1.data(), (long)T * C * 4);
    if (tp->f1_codes)  std::memcpy(tp->f1_codes + r0 * C, f1.data(), (long)T * C);
    if (tp->fc1_acc)   std::memcpy(tp->fc1_acc + r0 * Hd, a1.data(), (long)T * Hd * 4);
    if (tp->f2_codes)  std::memcpy(tp->f2_codes + r0 * Hd, f2.data(), (long)T * Hd);
    if (tp->fc2_acc)   std::memcpy(tp->fc2_acc + r0 * C, a2.data(), (long)T * C * 4);
  }
}

// "fp mode": the same block with every quantizer replaced by the identity; weights are code*scale.
// Accumulation in binary64 (no integer decision depends on it).
void fp_linear(const float* a, int M, int K, const orc_linear& L, const float* bias, float* out) {
  for (int m = 0; m < M; ++m)
    for (int n = 0; n < L.out_f; ++n) {
      double s = 0.0;
      for (int k = 0; k < K; ++k) s += (double)a[(long)m * K + k] * ((double)L.codes[(long)n * K + k] * (double)L.scale[n]);
      out[(long)m * L.out_f + n] = (float)(s + (bias ? (double)bias[n] : 0.0));
    }
}

// ranges (optional): 7 x {min, max} of what the quantizers of the sites QKV input, q, k, v, proj input, fc1 input,
// fc2 input would see, over every row of the window (pad rows included: they pass through the layers like any row)
struct SiteRanges { float lo[7], hi[7]; };
inline void observe(SiteRanges* r, int site, const float* v, long n) {
  if (!r) return;
  for (long i = 0; i < n; ++i) { r->lo[site] = std::fmin(r->lo[site], v[i]); r->hi[site] = std::fmax(r->hi[site], v[i]); }
}

void window_forward_fp(const orc_block& P, const orc_branch& br, const float* relb, const float* mask,
                       const float* xin, const uint8_t* real, float* yout, SiteRanges* rng = nullptr) {
  const int C = P.dim, T = P.window * P.window, nh = P.heads, d = C / nh, Hd = P.hidden;
  std::vector<float> ln((long)T * C), qkv((long)T * 3 * C), o((long)T * C), po((long)T * C), x1((long)T * C);
  for (int t = 0; t < T; ++t) {
    if (real[t]) layernorm_row(xin + (long)t * C, C, br.ln1_g, br.ln1_b, &ln[(long)t * C]);
    else std::fill(&ln[(long)t * C], &ln[(long)(t + 1) * C], 0.0f);
  }
  observe(rng, 0, ln.data(), (long)T * C);
  fp_linear(ln.data(), T, C, P.qkv, br.b_qkv, qkv.data());
  for (int t = 0; t < T; ++t)
    for (int sec = 0; sec < 3; ++sec) observe(rng, 1 + sec, &qkv[(long)t * 3 * C + sec * C], C);
  std::vector<float> logits(T), prob(T);
  const double rs = 1.0 / std::sqrt((double)d);
  for (int h = 0; h < nh; ++h)
    for (int i = 0; i < T; ++i) {
      for (int j = 0; j < T; ++j) {
        double s = 0.0;
        for (int e = 0; e < d; ++e) s += (double)qkv[(long)i * 3 * C + h * d + e] * (double)qkv[(long)j * 3 * C + C + h * d + e];
        logits[j] = (float)(s * rs + (double)relb[((long)h * T + i) * T + j] + (mask ? (double)mask[i * T + j] : 0.0));
      }
      softmax_row(logits.data(), T, prob.data());
      for (int e = 0; e < d; ++e) {
        double s = 0.0;
        for (int j = 0; j < T; ++j) s += (double)prob[j] * (double)qkv[(long)j * 3 * C + 2 * C + h * d + e];
        o[(long)i * C + h * d + e] = (float)s;
      }
    }
  observe(rng, 4, o.data(), (long)T * C);
  fp_linear(o.data(), T, C, P.proj, br.b_proj, po.data());
  for (long e = 0; e < (long)T * C; ++e) x1[e] = xin[e] + po[e];
  for (int t = 0; t < T; ++t) layernorm_row(&x1[(long)t * C], C, br.ln2_g, br.ln2_b, &ln[(long)t * C]);
  observe(rng, 5, ln.data(), (long)T * C);
  std::vector<float> h1((long)T * Hd), h2((long)T * C);
  fp_linear(ln.data(), T, C, P.fc1, br.b_fc1, h1.data());
  for (auto& v : h1) v = gelu1(v);
  observe(rng, 6, h1.data(), (long)T * Hd);
  fp_linear(h1.data(), T, Hd, P.fc2, br.b_fc2, h2.data());
  for (long e = 0; e < (long)T * C; ++e) yout[e] = x1[e] + h2[e];
}

// gather one window's tokens (pad -> zeros), run it, scatter the real tokens back
void run_window(const orc_block& P, const orc_branch& br, const float* relb, const float* x, float* y,
                int img, int H, int W, int w, const WinTaps* wt, SiteRanges* rng = nullptr) {
  const int C = P.dim, ws = P.window, T = ws * ws;
  std::vector<float> xin((long)T * C, 0.0f), yout((long)T * C);
  std::vector<uint8_t> real(T);
  std::vector<long> src(T);
  for (int t = 0; t < T; ++t) {
    src[t] = window_token(H, W, ws, P.shift, w, t);
    real[t] = src[t] >= 0;
    if (real[t]) std::memcpy(&xin[(long)t * C], x + ((long)img * H * W + src[t]) * C, C * sizeof(float));
  }
  std::vector<float> mask;
  if (P.shift > 0) { mask.resize((long)T * T); shift_mask(H, W, ws, P.shift, w, mask.data()); }
  const float* mk = P.shift > 0 ? mask.data() : nullptr;
  if (P.quant) window_forward_quant(P, br, relb, mk, xin.data(), real.data(), yout.data(), wt);
  else         window_forward_fp(P, br, relb, mk, xin.data(), real.data(), yout.data(), rng);
  for (int t = 0; t < T; ++t)
    if (real[t]) std::memcpy(y + ((long)img * H * W + src[t]) * C, &yout[(long)t * C], C * sizeof(float));
}

}  // namespace

// =================================================================================================
extern "C" {

void orc_set_threads(int n) {
#ifdef _OPENMP
  omp_set_num_threads(n);
#else
  (void)n;
#endif
}
int orc_get_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// number of windows a ratio assigns out of n: floor(ratio*n + 1e-6)   (the paper gives no rounding rule)
int orc_low_count(double ratio, int n) { return (int)std::floor(ratio * (double)n + 1e-6); }

void orc_quantize(const float* x, long n, orc_aq q, uint8_t* codes) {
  for (long i = 0; i < n; ++i) codes[i] = quant1(x[i], q);
}
void orc_dequantize(const uint8_t* codes, long n, orc_aq q, float* x) {
  for (long i = 0; i < n; ++i) x[i] = (float)((int)codes[i] - q.zp) * q.scale;
}
// sub-byte codes, little end first: element e of a row sits in byte e*bits/8 at bit (e*bits) mod 8
void orc_pack(const uint8_t* codes, long rows, int cols, int bits, uint8_t* out) {
  int per = 8 / bits; long rb = (cols + per - 1) / per;
  std::memset(out, 0, rows * rb);
  for (long r = 0; r < rows; ++r)
    for (int c = 0; c < cols; ++c)
      out[r * rb + c / per] |= (uint8_t)((codes[r * cols + c] & ((1 << bits) - 1)) << ((c % per) * bits));
}
void orc_unpack(const uint8_t* packed, long rows, int cols, int bits, uint8_t* codes) {
  int per = 8 / bits; long rb = (cols + per - 1) / per;
  for (long r = 0; r < rows; ++r)
    for (int c = 0; c < cols; ++c)
      codes[r * cols + c] = (packed[r * rb + c / per] >> ((c % per) * bits)) & ((1 << bits) - 1);
}
void orc_layernorm(const float* x, long rows, int C, const float* g, const float* b, float* y) {
  for (long r = 0; r < rows; ++r) layernorm_row(x + r * C, C, g, b, y + r * C);
}
void orc_exp2(const float* t, long n, float* y) { for (long i = 0; i < n; ++i) y[i] = exp2_clamped(t[i]); }
void orc_gelu(const float* x, long n, float* y) { for (long i = 0; i < n; ++i) y[i] = gelu1(x[i]); }
void orc_softmax_rows(const float* s, long rows, int T, float* p) {
  for (long r = 0; r < rows; ++r) softmax_row(s + r * T, T, p + r * T);
}
void orc_int_gemm(const uint8_t* a, long M, int K, int za, const int8_t* w, int N, int32_t* acc) {
  orc_linear L = { w, nullptr, N, K };
  int_linear(a, (int)M, K, za, L, acc);
}
long orc_window_token(int H, int W, int ws, int shift, int w, int t) { return window_token(H, W, ws, shift, w, t); }
void orc_shift_mask(int H, int W, int ws, int shift, int w, float* mask) { shift_mask(H, W, ws, shift, w, mask); }
void orc_relpos_bias(const float* table, int ws, int heads, float* bias) { relpos_bias(table, ws, heads, bias); }

// token energy: sum over channels of the squared int8 score code (Section 3.2: importance = L2 norm)
void orc_energy(const float* x, int B, int H, int W, int C, float inv_scale, int32_t* energy) {
  long n = (long)B * H * W;
  for (long i = 0; i < n; ++i) {
    int32_t e = 0;
    for (int c = 0; c < C; ++c) {
      float r = std::nearbyintf(x[i * C + c] * inv_scale);
      r = std::fmin(std::fmax(r, -127.0f), 127.0f);
      int code = (int)r;
      e += code * code;
    }
    energy[i] = e;
  }
}

void orc_window_scores(const int32_t* energy, int B, int H, int W, int ws, int shift, int64_t* scores) {
  int Hp = round_up(H, ws), Wp = round_up(W, ws);
  int nW = (Hp / ws) * (Wp / ws), T = ws * ws;
  for (int b = 0; b < B; ++b)
    for (int w = 0; w < nW; ++w) {
      int64_t s = 0;
      for (int t = 0; t < T; ++t) {
        long src = window_token(H, W, ws, shift, w, t);
        if (src >= 0) s += energy[(long)b * H * W + src];
      }
      scores[(long)b * nW + w] = s;
    }
}

void orc_select(const int64_t* scores, int B, int nW, double low_ratio, double prune_ratio, int reverse,
                int32_t* order, uint8_t* cls, int* counts) {
  int n_pr = orc_low_count(prune_ratio, nW);
  int n_lo = orc_low_count(low_ratio, nW - n_pr);
  int n_hi = nW - n_pr - n_lo;
  if (counts) { counts[0] = n_hi; counts[1] = n_lo; counts[2] = n_pr; }
  for (int b = 0; b < B; ++b) {
    const int64_t* s = scores + (long)b * nW;
    std::vector<int32_t> idx(nW);
    for (int w = 0; w < nW; ++w) idx[w] = w;
    std::stable_sort(idx.begin(), idx.end(), [&](int32_t a, int32_t c) {
      if (s[a] != s[c]) return reverse ? s[a] < s[c] : s[a] > s[c];
      return a < c;
    });
    for (int j = 0; j < nW; ++j) {
      if (order) order[(long)b * nW + j] = idx[j];
      if (cls) cls[(long)b * nW + idx[j]] = j < n_hi ? 0 : (j < n_hi + n_lo ? 1 : 2);
    }
  }
}

void orc_block_forward(const orc_block* p, const float* x, float* y, int B, int H, int W,
                       double low_ratio, double prune_ratio, const int32_t* energy, int reverse,
                       int32_t* order_out, uint8_t* cls_out, int64_t* score_out,
                       const orc_taps* taps_hi, const orc_taps* taps_lo) {
  const orc_block& P = *p;
  const int ws = P.window, T = ws * ws, C = P.dim;
  const int Hp = round_up(H, ws), Wp = round_up(W, ws), nW = (Hp / ws) * (Wp / ws);
  std::vector<int32_t> en;
  if (!energy) { en.resize((long)B * H * W); orc_energy(x, B, H, W, C, P.score_inv_scale, en.data()); energy = en.data(); }
  std::vector<int64_t> scores((long)B * nW);
  orc_window_scores(energy, B, H, W, ws, P.shift, scores.data());
  std::vector<int32_t> order((long)B * nW);
  std::vector<uint8_t> cls((long)B * nW);
  int cnt[3];
  orc_select(scores.data(), B, nW, low_ratio, prune_ratio, reverse, order.data(), cls.data(), cnt);
  if (order_out) std::memcpy(order_out, order.data(), order.size() * 4);
  if (cls_out)   std::memcpy(cls_out, cls.data(), cls.size());
  if (score_out) std::memcpy(score_out, scores.data(), scores.size() * 8);
  const int n_hi = cnt[0], n_lo = cnt[1];
  std::vector<float> relb((long)P.heads * T * T);
  relpos_bias(P.relpos, ws, P.heads, relb.data());
  // pruned windows are forwarded unchanged (Section 3.4): start from a copy, then overwrite the others
  std::memcpy(y, x, (size_t)B * H * W * C * sizeof(float));
  const long jobs = (long)B * (n_hi + n_lo);
#pragma omp parallel for schedule(dynamic, 4)
  for (long job = 0; job < jobs; ++job) {
    int b = (int)(job / (n_hi + n_lo)), j = (int)(job % (n_hi + n_lo));
    int w = order[(long)b * nW + j];
    bool high = j < n_hi;
    const orc_branch& br = high ? P.hi : P.lo;
    const orc_taps* tp = high ? taps_hi : taps_lo;
    WinTaps wt; const WinTaps* wtp = nullptr;
    if (tp) {
      long slot = high ? ((long)b * n_hi + j) : ((long)b * n_lo + (j - n_hi));
      wt.t = tp; wt.win = slot; wt.row0 = slot * T; wtp = &wt;
    }
    run_window(P, br, relb.data(), x, y, b, H, W, w, wtp);
  }
}

// The uniform quantized Swin block, written on the WHOLE map in the published order of a Swin block (norm -> zero
// padding -> cyclic shift -> window partition -> attention -> reverse -> crop -> FFN) and token by token in global
// coordinates.  It shares only the scalar primitives above (quantizer, LayerNorm row, softmax row, GELU, dequantize)
// with the two-branch path: no window gathering, no per-window mask or bias table, no batch bookkeeping.  Ratio 0 and
// ratio 1 of orc_block_forward must reproduce it bit for bit (Section 3.3: the ratio is the share of low windows).
static void uniform_block_quant_whole_map(const orc_block& P, const orc_branch& br, const float* x, float* y,
                                          int B, int H, int W) {
  const int C = P.dim, ws = P.window, nh = P.heads, d = C / nh, Hd = P.hidden, s = P.shift;
  const int Hp = round_up(H, ws), Wp = round_up(W, ws);
  const long NP = (long)Hp * Wp;
  const int pmax = (1 << br.bits) - 1;
  const orc_aq pq = { br.bits, 1.0f / (float)pmax, (float)pmax, 0 };
  const float alpha = (br.q.scale * br.k.scale) * (float)(1.0 / std::sqrt((double)d));
  const float so = pq.scale * br.v.scale;
  auto region = [&](int pos, int L) { return pos < L - ws ? 0 : (pos < L - s ? 1 : 2); };
  for (int b = 0; b < B; ++b) {
    const float* xb = x + (long)b * H * W * C;
    float* yb = y + (long)b * H * W * C;
    // 1. LayerNorm of the real tokens, zero padding AFTER the norm, input quantizer, QKV projection, q/k/v quantizers
    std::vector<uint8_t> qkv(NP * 3 * C);
#pragma omp parallel for schedule(static)
    for (long tok = 0; tok < NP; ++tok) {
      const int ty = (int)(tok / Wp), tx = (int)(tok % Wp);
      std::vector<float> ln(C, 0.0f);
      if (ty < H && tx < W) layernorm_row(xb + ((long)ty * W + tx) * C, C, br.ln1_g, br.ln1_b, ln.data());
      std::vector<uint8_t> a(C);
      for (int c = 0; c < C; ++c) a[c] = quant1(ln[c], br.qkv_in);
      for (int n = 0; n < 3 * C; ++n) {
        int32_t acc = 0;
        for (int c = 0; c < C; ++c) acc += ((int)a[c] - br.qkv_in.zp) * (int)P.qkv.codes[(long)n * C + c];
        const float v = dequant_bias(acc, br.qkv_in.scale, P.qkv.scale[n], br.b_qkv[n]);
        qkv[tok * 3 * C + n] = quant1(v, n < C ? br.q : (n < 2 * C ? br.k : br.v));
      }
    }
    // 2. every real token attends the tokens of its window in the cyclically shifted frame (pad tokens are keys),
    //    then proj + residual, LN2, fc1, GELU, fc2 + residual
#pragma omp parallel for schedule(dynamic, 16)
    for (long tok = 0; tok < NP; ++tok) {
      const int ty = (int)(tok / Wp), tx = (int)(tok % Wp);
      if (ty >= H || tx >= W) continue;                       // cropped away at the end
      const int ys = (ty - s + Hp) % Hp, xs = (tx - s + Wp) % Wp;       // my position in the shifted frame
      const int wy0 = ys / ws * ws, wx0 = xs / ws * ws;                 // my window's corner in the shifted frame
      const int iy = ys - wy0, ix = xs - wx0;
      const int my_reg = region(ys, Hp) * 3 + region(xs, Wp);
      const int T = ws * ws;
      std::vector<long> key(T);
      std::vector<int> key_reg(T);
      for (int j = 0; j < T; ++j) {
        const int ky = wy0 + j / ws, kx = wx0 + j % ws;
        key[j] = (long)((ky + s) % Hp) * Wp + (kx + s) % Wp;
        key_reg[j] = region(ky, Hp) * 3 + region(kx, Wp);
      }
      std::vector<float> logits(T), prob(T);
      std::vector<uint8_t> pc(T), o(C);
      for (int h = 0; h < nh; ++h) {
        for (int j = 0; j < T; ++j) {
          int32_t sdot = 0;
          for (int e = 0; e < d; ++e)
            sdot += ((int)qkv[tok * 3 * C + h * d + e] - br.q.zp) * ((int)qkv[key[j] * 3 * C + C + h * d + e] - br.k.zp);
          const int ridx = (iy - j / ws + ws - 1) * (2 * ws - 1) + (ix - j % ws + ws - 1);
          float lg = std::fmaf((float)sdot, alpha, P.relpos[(long)ridx * nh + h]);
          if (s > 0) lg = lg + (key_reg[j] == my_reg ? 0.0f : -100.0f);
          logits[j] = lg;
        }
        softmax_row(logits.data(), T, prob.data());
        for (int j = 0; j < T; ++j) pc[j] = quant1(prob[j], pq);
        for (int e = 0; e < d; ++e) {
          int32_t pv = 0;
          for (int j = 0; j < T; ++j) pv += (int)pc[j] * ((int)qkv[key[j] * 3 * C + 2 * C + h * d + e] - br.v.zp);
          o[h * d + e] = quant1((float)pv * so, br.proj_in);
        }
      }
      const float* xr = xb + ((long)ty * W + tx) * C;
      std::vector<float> x1(C), ln(C);
      for (int n = 0; n < C; ++n) {
        int32_t acc = 0;
        for (int c = 0; c < C; ++c) acc += ((int)o[c] - br.proj_in.zp) * (int)P.proj.codes[(long)n * C + c];
        x1[n] = xr[n] + dequant_bias(acc, br.proj_in.scale, P.proj.scale[n], br.b_proj[n]);
      }
      layernorm_row(x1.data(), C, br.ln2_g, br.ln2_b, ln.data());
      std::vector<uint8_t> f1(C), f2(Hd);
      for (int c = 0; c < C; ++c) f1[c] = quant1(ln[c], br.fc1_in);
      for (int n = 0; n < Hd; ++n) {
        int32_t acc = 0;
        for (int c = 0; c < C; ++c) acc += ((int)f1[c] - br.fc1_in.zp) * (int)P.fc1.codes[(long)n * C + c];
        f2[n] = quant1(gelu1(dequant_bias(acc, br.fc1_in.scale, P.fc1.scale[n], br.b_fc1[n])), br.fc2_in);
      }
      float* yr = yb + ((long)ty * W + tx) * C;
      for (int n = 0; n < C; ++n) {
        int32_t acc = 0;
        for (int c = 0; c < Hd; ++c) acc += ((int)f2[c] - br.fc2_in.zp) * (int)P.fc2.codes[(long)n * Hd + c];
        yr[n] = x1[n] + dequant_bias(acc, br.fc2_in.scale, P.fc2.scale[n], br.b_fc2[n]);
      }
    }
  }
}

void orc_uniform_block_forward(const orc_block* p, const orc_branch* br, const float* x, float* y,
                               int B, int H, int W) {
  const orc_block& P = *p;
  if (P.quant) { uniform_block_quant_whole_map(P, *br, x, y, B, H, W); return; }
  // fp mode (all quantizers off; pinned to a textbook Swin block in binary64): window by window
  const int ws = P.window, T = ws * ws;
  const int Hp = round_up(H, ws), Wp = round_up(W, ws), nW = (Hp / ws) * (Wp / ws);
  std::vector<float> relb((long)P.heads * T * T);
  relpos_bias(P.relpos, ws, P.heads, relb.data());
#pragma omp parallel for schedule(dynamic, 4)
  for (long job = 0; job < (long)B * nW; ++job)
    run_window(P, *br, relb.data(), x, y, (int)(job / nW), H, W, (int)(job % nW), nullptr);
}

// Calibration observer (Section 4.3: the full feature map calibrates both branches): the floating-point block
// (quantizers off, whatever P.quant says) with every window through the LayerNorm parameters and biases of `br`;
// y = its output, ranges[2*site], ranges[2*site+1] = min, max seen at the seven quantizer sites (order: QKV input, q,
// k, v, proj input, fc1 input, fc2 input) over all rows of all windows.
void orc_block_observe_fp(const orc_block* p, const orc_branch* br, const float* x, float* y, int B, int H, int W,
                          float* ranges /* [14] */) {
  orc_block P = *p;
  P.quant = 0;
  const int ws = P.window, T = ws * ws;
  const int Hp = round_up(H, ws), Wp = round_up(W, ws), nW = (Hp / ws) * (Wp / ws);
  std::vector<float> relb((long)P.heads * T * T);
  relpos_bias(P.relpos, ws, P.heads, relb.data());
  SiteRanges all;
  for (int i = 0; i < 7; ++i) { all.lo[i] = INFINITY; all.hi[i] = -INFINITY; }
#pragma omp parallel
  {
    SiteRanges mine = all;
#pragma omp for schedule(dynamic, 4)
    for (long job = 0; job < (long)B * nW; ++job)
      run_window(P, *br, relb.data(), x, y, (int)(job / nW), H, W, (int)(job % nW), nullptr, &mine);
#pragma omp critical
    for (int i = 0; i < 7; ++i) { all.lo[i] = std::fmin(all.lo[i], mine.lo[i]); all.hi[i] = std::fmax(all.hi[i], mine.hi[i]); }
  }
  for (int i = 0; i < 7; ++i) { ranges[2 * i] = all.lo[i]; ranges[2 * i + 1] = all.hi[i]; }
}

// the same for patch merging: min, max of the LayerNorm output that the merge's input quantizer would see
void orc_merge_observe_fp(const orc_merge* m, const float* x, int B, int H, int W, int C, float* y, float* range /* [2] */) {
  const int H2 = (H + 1) / 2, W2 = (W + 1) / 2, K = 4 * C, N = m->red.out_f;
  float lo = INFINITY, hi = -INFINITY;
  for (long tok = 0; tok < (long)B * H2 * W2; ++tok) {
    int b = (int)(tok / ((long)H2 * W2)), r = (int)(tok % ((long)H2 * W2));
    int y2 = r / W2, x2 = r % W2;
    std::vector<float> cat(K, 0.0f), ln(K);
    const int dy[4] = {0, 1, 0, 1}, dx[4] = {0, 0, 1, 1};
    for (int g = 0; g < 4; ++g) {
      int yy = 2 * y2 + dy[g], xx = 2 * x2 + dx[g];
      if (yy < H && xx < W) std::memcpy(&cat[(long)g * C], x + (((long)b * H + yy) * W + xx) * C, C * sizeof(float));
    }
    layernorm_row(cat.data(), K, m->ln_g, m->ln_b, ln.data());
    for (int k = 0; k < K; ++k) { lo = std::fmin(lo, ln[k]); hi = std::fmax(hi, ln[k]); }
    fp_linear(ln.data(), 1, K, m->red, nullptr, y + tok * N);
  }
  range[0] = lo; range[1] = hi;
}

// patch merging: 2x2 neighbours concatenated (zero-padded when H or W is odd) -> LN(4C) -> quantize ->
// integer GEMM with the [2C][4C] reduction weight, no bias.
void orc_merge_forward(const orc_merge* m, const float* x, int B, int H, int W, int C, float* y) {
  const int H2 = (H + 1) / 2, W2 = (W + 1) / 2, K = 4 * C, N = m->red.out_f;
#pragma omp parallel for schedule(static)
  for (long tok = 0; tok < (long)B * H2 * W2; ++tok) {
    int b = (int)(tok / ((long)H2 * W2)), r = (int)(tok % ((long)H2 * W2));
    int y2 = r / W2, x2 = r % W2;
    std::vector<float> cat(K, 0.0f), ln(K);
    const int dy[4] = {0, 1, 0, 1}, dx[4] = {0, 0, 1, 1};
    for (int g = 0; g < 4; ++g) {
      int yy = 2 * y2 + dy[g], xx = 2 * x2 + dx[g];
      if (yy < H && xx < W) std::memcpy(&cat[(long)g * C], x + (((long)b * H + yy) * W + xx) * C, C * sizeof(float));
    }
    layernorm_row(cat.data(), K, m->ln_g, m->ln_b, ln.data());
    if (m->quant) {
      std::vector<uint8_t> a(K);
      orc_quantize(ln.data(), K, m->in, a.data());
      std::vector<int32_t> acc(N);
      int_linear(a.data(), 1, K, m->in.zp, m->red, acc.data());
      for (int n = 0; n < N; ++n) y[tok * N + n] = (float)acc[n] * (m->in.scale * m->red.scale[n]);
    } else {
      fp_linear(ln.data(), 1, K, m->red, nullptr, y + tok * N);
    }
  }
}

// patch embedding: 4x4 patches (zero padding to multiples of 4) -> quantize -> integer projection -> + bias -> LN
void orc_patch_embed(const orc_embed* e, const float* img, int B, int Hi, int Wi, float* x0) {
  const int H = (Hi + 3) / 4, W = (Wi + 3) / 4, K = 48, N = e->proj.out_f;
#pragma omp parallel for schedule(static)
  for (long tok = 0; tok < (long)B * H * W; ++tok) {
    const int b = (int)(tok / ((long)H * W)), r = (int)(tok % ((long)H * W));
    const int ty = r / W, tx = r % W;
    std::vector<float> v(K, 0.0f), t(N), y(N);
    for (int ky = 0; ky < 4; ++ky)
      for (int kx = 0; kx < 4; ++kx) {
        const int yy = 4 * ty + ky, xx = 4 * tx + kx;
        if (yy < Hi && xx < Wi)
          for (int c = 0; c < 3; ++c) v[(ky * 4 + kx) * 3 + c] = img[(((long)b * Hi + yy) * Wi + xx) * 3 + c];
      }
    if (e->quant) {
      std::vector<uint8_t> a(K);
      orc_quantize(v.data(), K, e->in, a.data());
      std::vector<int32_t> acc(N);
      int_linear(a.data(), 1, K, e->in.zp, e->proj, acc.data());
      for (int n = 0; n < N; ++n) {
        const float d = (float)acc[n] * (e->in.scale * e->proj.scale[n]);
        t[n] = d + e->bias[n];
      }
    } else {
      fp_linear(v.data(), 1, K, e->proj, e->bias, t.data());
    }
    layernorm_row(t.data(), N, e->ln_g, e->ln_b, y.data());
    std::memcpy(x0 + tok * N, y.data(), N * sizeof(float));
  }
}

void orc_backbone_forward(int num_stages, const int* depths, const orc_block* blocks, const orc_merge* merges,
                          const float* x0, float* const* stage_out, int B, int H0, int W0,
                          const double* low_ratio_per_pair, const double* prune_ratio_per_pair, int allow_elevation,
                          int reverse) {
  int H = H0, W = W0, blk = 0;
  std::vector<float> cur, nxt;
  for (int s = 0; s < num_stages; ++s) {
    const int C = blocks[blk].dim;
    if (s == 0) cur.assign(x0, x0 + (size_t)B * H * W * C);
    else {
      const int Cprev = blocks[blk - 1].dim;
      int H2 = (H + 1) / 2, W2 = (W + 1) / 2;
      nxt.resize((size_t)B * H2 * W2 * C);
      orc_merge_forward(&merges[s - 1], cur.data(), B, H, W, Cprev, nxt.data());
      cur.swap(nxt); H = H2; W = W2;
    }
    // importance is computed once per stage, before its first block, and shared (Section 3.2)
    std::vector<int32_t> energy((size_t)B * H * W);
    orc_energy(cur.data(), B, H, W, C, blocks[blk].score_inv_scale, energy.data());
    // Windows keep their precision class within a stage (Section 4.4, "Windows Elevation": letting compressed windows
    // return to high precision in later blocks is the ablation, not the default): a pair's effective ratios are the
    // largest ratios of the pairs of this stage so far, so the set of non-high windows never shrinks.
    double low_eff = 0.0, prune_eff = 0.0;
    for (int i = 0; i < depths[s]; ++i, ++blk) {
      int pair = blk / 2;
      double lr = low_ratio_per_pair[pair], pr = prune_ratio_per_pair ? prune_ratio_per_pair[pair] : 0.0;
      if (!allow_elevation) {
        low_eff = std::max(low_eff, lr); prune_eff = std::max(prune_eff, pr);
        lr = low_eff; pr = prune_eff;
      }
      nxt.resize(cur.size());
      orc_block_forward(&blocks[blk], cur.data(), nxt.data(), B, H, W, lr, pr, energy.data(), reverse,
                        nullptr, nullptr, nullptr, nullptr, nullptr);
      cur.swap(nxt);
    }
    std::memcpy(stage_out[s], cur.data(), cur.size() * sizeof(float));
  }
}

}  // extern "C"
