// Internal interface between the host API (mixaq.cu) and the kernel translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "common.cuh"

namespace mixaq {

// kernels launched since the API call started (host bookkeeping); per thread, so that calls made on different
// contexts from different threads do not disturb each other's counts
extern thread_local int g_launches;

// ---- selection ------------------------------------------------------------------------------
void launch_energy(const float* x, int32_t* energy, long ntok, int C, float inv_scale, cudaStream_t st);

struct SelectArgs {
  const int32_t* energy;     // [B][H][W]
  int64_t* score;            // [B][nW]
  int32_t* order;            // [B][nW]
  uint8_t* cls;              // [B][nW]
  int32_t* rowsrc_hi;        // [B*n_hi*49] source token (b*H*W + y*W + x) or -1 for a pad token
  int32_t* rowsrc_lo;        // [B*n_lo*49]
  int32_t* rowsrc_pr;        // [B*n_pr*49]
  int32_t* win_hi;           // [B*n_hi] window index of every batch slot
  int32_t* win_lo;           // [B*n_lo]
  int B, H, W, shift, nwx, nW, n_hi, n_lo, n_pr, reverse;
};
// selections of `count` blocks that share one energy map (all blocks of a stage): 2 launches per 24 blocks
void launch_select(const SelectArgs* a, int count, cudaStream_t st);
// ascending window indices of one class per image: out[b][0 .. n_c) from cls[b][0 .. nW); c = 0, 1, 2 in one launch
void launch_class_lists(const uint8_t* cls, int B, int nW, int32_t* const out[3], const int count[3], cudaStream_t st);

// ---- row-wise LayerNorm + quantize + pack -----------------------------------------------------
struct LnBranch {
  const float* src;          // feature map (gather) or window-batch matrix [M][C]
  const int32_t* rowsrc;     // nullable: row m reads src + rowsrc[m]*C (rowsrc < 0: pad token -> zero after LN)
  const float *gamma, *beta;
  uint8_t* out;              // [M][C*bits/8]
  AQ q;
  int M;
  int mgH, mgW;              // patch merging only: size of the input map (row m is an OUTPUT token, its C channels are
                             // those of the 2x2 input neighbours, C/4 each)
};
void launch_ln_quant(const LnBranch& hi, const LnBranch& lo, int C, cudaStream_t st);

struct MergeGatherArgs {
  const float* x; const float *gamma, *beta; uint8_t* out; AQ q; int B, H, W, C;
};
void launch_merge_gather(const MergeGatherArgs& a, cudaStream_t st);
// ---- guard zones of the workspaces (debug aid) -------------------------------------------------------
constexpr int GUARD_BYTES = 256;          // after every buffer of a workspace
// fill = true: writes the guard pattern into every zone; fill = false: compares, and on a difference sets bit 1 of *status
void launch_guards(void* const* zones, int count, bool fill, int* status, cudaStream_t st);

void launch_copy_rows(const float* x, float* y, const int32_t* rowsrc, int M, int C, cudaStream_t st);

// ---- stem and output norms ---------------------------------------------------------------------------
struct PatchGatherArgs { const float* img; uint8_t* out; AQ q; int B, Hi, Wi; };   // out: [tokens][64] codes
void launch_patch_gather(const PatchGatherArgs& a, cudaStream_t st);
// y = LayerNorm(x + bias), binary32 in and out, rows x C; bias nullable.  false: C not supported.
bool launch_bias_ln(const float* x, const float* bias, const float* gamma, const float* beta, float* y, long rows,
                    int C, cudaStream_t st);
void launch_pad_weights(const int8_t* w, int N, int K, int Kp, int8_t* out, cudaStream_t st);

// ---- integer GEMM with fused epilogues ----------------------------------------------------------
enum EpiMode { EPI_QKV = 0, EPI_PROJ = 1, EPI_FC1 = 2, EPI_FC2 = 3, EPI_MERGE = 4 };

struct GemmBranch {
  const uint8_t* a;          // [M][K*a_bits/8] packed unsigned codes
  int M, a_bits;
  const float* mult;         // [N]  s_a * s_w[n]
  const int32_t* zc;         // [N]  z_a * sum_k w[n][k]
  const float* bias;         // [N]  (nullable for EPI_MERGE)
  AQ q0, q1, q2;             // output quantizers (QKV: q,k,v; FC1: q0)
  int out_bits;
  uint8_t* out_codes;        // QKV, FC1: [M][N*out_bits/8]
  float* out_f;              // PROJ: x1 [M][N];  FC2: y feature map;  MERGE: [M][N]
  const float* res;          // PROJ: feature map x (gathered through rowsrc);  FC2: x1 [M][N]
  const int32_t* rowsrc;     // PROJ, FC2
  int32_t* tap_acc;          // nullable [M][N]
};
struct GemmArgs {
  const int8_t* w;           // [N][K]
  int N, K, C;               // C: channels per q/k/v section (EPI_QKV)
  int mode;
  int* status;           // device status word (raised when a bounded wait runs out)
  GemmBranch br[2];
};
bool launch_gemm(const GemmArgs& g, cudaStream_t st);
void launch_wait_probe(int* status, cudaStream_t st);   // self-test of the bounded wait (it must run out)
// tensor-core issue-rate microbenchmark (kind 0: i8, 1: f8f6f4/E4M3); ns per SM into ns_out; returns the grid size
int launch_mma_peak(int kind, int groups, unsigned long long* ns_out, int* status, cudaStream_t st);
bool gemm_init();   // once per device context, before the first launch

// ---- fused window attention ----------------------------------------------------------------------
struct AttnBranch {
  const uint8_t* qkv;        // [M][3C*cbits/8]
  uint8_t* out;              // [M][C*cbits/8]
  const int32_t* win;        // [slots] window index (for the shift mask)
  AQ q, k, v, o;
  int bits, slots;           // bits: width of the codes' range (and of the probability quantizer)
  int cbits;                 // bits a stored code occupies: `bits` (bit-packed) or 8 (one code per byte)
  float alpha;               // s_q*s_k/sqrt(d)
  float so;                  // s_p*s_v
  uint8_t* tap_p;            // nullable
  float* tap_probs;          // nullable: softmax output [slots][heads][49][49]
  int32_t* tap_pv;           // nullable
};
struct AttnArgs {
  const float* relbias;      // [heads][4][7][32][4], accumulator-fragment order
  int C, heads, shift, Hp, Wp, nwx, nW;
  AttnBranch br[2];
};
void launch_attention(const AttnArgs& a, cudaStream_t st);

// ---- calibration: floating-point block / merge with min-max observers at the quantizer sites -----------------------
struct CalBlockArgs {
  const float* x; float* y;                       // feature maps [B][H][W][C]
  int B, H, W, C, heads, hidden, shift;
  const float *ln1_g, *ln1_b, *ln2_g, *ln2_b, *b_qkv, *b_proj, *b_fc1, *b_fc2;   // of the branch being calibrated
  const int8_t *w_qkv, *w_proj, *w_fc1, *w_fc2;
  const float *s_qkv, *s_proj, *s_fc1, *s_fc2, *relpos;
  int32_t* rowsrc; float *ln, *qkv, *o, *x1, *h;  // workspace: [M], [M][C], [M][3C], [M][C], [M][C], [M][hidden]
  uint32_t* obs;                                  // 16 order-preserving keys: min, max of the seven sites and of x
};
bool launch_calibrate_block(const CalBlockArgs& c, cudaStream_t st);
struct CalMergeArgs {
  const float* x; float* y; int B, H, W, C, N;
  const float *ln_g, *ln_b; const int8_t* w; const float* sw;
  float* ln;                                      // workspace [M][4C]
  uint32_t* obs;                                  // 2 keys
};
bool launch_calibrate_merge(const CalMergeArgs& c, cudaStream_t st);
float cal_key_to_float(uint32_t key);

// ---- preparation -----------------------------------------------------------------------------------
void launch_prepare_linear(const int8_t* w, const float* sw, int N, int K, float sa, int za, float* mult,
                           int32_t* zc, cudaStream_t st);
void launch_prepare_relbias(const float* table, int heads, float* out, cudaStream_t st);

}  // namespace mixaq
