/* Reference ("oracle") implementation of the quantized Two-Branch Swin Block forward of MixA-Q
 * (Section 3.1 "Replace Pruning with MP Execution", Section 3.2 "Two-Branch Swin Block",
 * Section 3.4 "Activation Pruning Incorporation").
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow CPU program that follows the
 * method step by step, one window at a time, so that it can be checked against the paper by eye.
 * Only the test-suite, the smoke check and the CPU-baseline leg of the benchmark may call it.  It shares
 * no code, header, table or helper with the CUDA library; its structs are its own.
 *
 * Precision: every floating-point value that feeds a quantizer (and therefore decides an integer code)
 * is binary32, built from individually rounded IEEE-754 add / mul / fma / div / sqrt in a fixed order,
 * because the kernels take those decisions in binary32.  Integer work is exact (int32 / int64).
 *
 * Parity pins (tests/test_oracle_*.py): every function below is pinned to something other than itself
 * (closed forms, libm in binary64, brute force on tiny inputs, special cases) EXCEPT the choices the paper
 * leaves open (where exactly the quantizers sit, the rounding rule, the softmax/GELU evaluation scheme,
 * how pad tokens are treated, the mask value -100).  For those: "parity unpinned" by the paper; they are
 * fixed by this repository's written numeric contract only.
 */
#ifndef MIXAQ_ORACLE_H
#define MIXAQ_ORACLE_H
#include <stdint.h>
#ifdef __cplusplus
extern "C" {
#endif

/* per-tensor asymmetric activation quantizer: q = clamp(rne(x*inv_scale) + zp, 0, 2^bits-1) */
typedef struct { int bits; float scale; float inv_scale; int zp; } orc_aq;

/* per-output-channel symmetric weight matrix, one signed code per byte, row-major [out][in] */
typedef struct { const int8_t* codes; const float* scale; int out_f; int in_f; } orc_linear;

/* one branch (high or low) of a block: private LayerNorms, quantizers, biases (Section 3.2) */
typedef struct {
  const float *ln1_g, *ln1_b, *ln2_g, *ln2_b;
  const float *b_qkv, *b_proj, *b_fc1, *b_fc2;
  orc_aq qkv_in, q, k, v, proj_in, fc1_in, fc2_in;
  int bits;                 /* bit width of the attention-probability quantizer of this branch */
} orc_branch;

typedef struct {
  int dim, heads, window, shift, hidden;
  orc_linear qkv, proj, fc1, fc2;      /* shared "shadow layer" weights (Section 3.2) */
  const float* relpos;                 /* [(2ws-1)^2][heads] */
  orc_branch hi, lo;
  float score_inv_scale;               /* int8 score-code step (inverse) */
  int quant;                           /* 1: quantized block; 0: "fp mode" (all quantizers are the identity) */
} orc_block;

/* optional taps: every pointer may be NULL.  Rows are in window-batch order: all high windows of image 0
 * (in rank order), of image 1, ...; the low batch likewise.  Codes are one per byte (unpacked). */
typedef struct {
  uint8_t* a_codes;     /* [M][C]   input codes of the QKV layer            */
  int32_t* qkv_acc;     /* [M][3C]  zero-point-corrected accumulators        */
  uint8_t* qkv_codes;   /* [M][3C]  q | k | v codes                          */
  float*   probs;       /* [nwin][heads][T][T] softmax output (fp32)         */
  uint8_t* p_codes;     /* [nwin][heads][T][T]                               */
  int32_t* pv_acc;      /* [M][C]                                            */
  uint8_t* o_codes;     /* [M][C]   input codes of proj                      */
  int32_t* proj_acc;    /* [M][C]                                            */
  float*   x1;          /* [M][C]   after the attention residual             */
  uint8_t* f1_codes;    /* [M][C]   input codes of fc1 (after LN2)           */
  int32_t* fc1_acc;     /* [M][4C]                                           */
  uint8_t* f2_codes;    /* [M][4C]  input codes of fc2 (after GELU)          */
  int32_t* fc2_acc;     /* [M][C]                                            */
} orc_taps;

typedef struct { const float *ln_g, *ln_b; orc_aq in; orc_linear red; int quant; } orc_merge;

/* Patch embedding in front of the backbone (the stem of the Swin backbone the paper quantizes; its cost belongs to the
 * layers the method does not reduce, Appendix 6.2): 4x4 non-overlapping patches of an [B][Hi][Wi][3] image (zero
 * padded to multiples of 4), patch vector index (ky*4 + kx)*3 + c, quantized with `in`, integer projection
 * [C0][48], then t = (float)acc * (s_in*s_w[n]) + bias[n] (two rounded operations), then LayerNorm(C0).
 * quant = 0: the same in floating point (binary64 accumulation).  Paper silent on all numerics: parity unpinned by
 * the paper, pinned to numpy convolution + LayerNorm in tests. */
typedef struct { const float *ln_g, *ln_b, *bias; orc_aq in; orc_linear proj; int quant; } orc_embed;

/* ---- primitives (each pinned separately) ---- */
int   orc_low_count(double ratio, int n);
void  orc_quantize(const float* x, long n, orc_aq q, uint8_t* codes);
void  orc_dequantize(const uint8_t* codes, long n, orc_aq q, float* x);
void  orc_pack(const uint8_t* codes, long rows, int cols, int bits, uint8_t* out);
void  orc_unpack(const uint8_t* packed, long rows, int cols, int bits, uint8_t* codes);
void  orc_layernorm(const float* x, long rows, int C, const float* g, const float* b, float* y);
void  orc_exp2(const float* t, long n, float* y);
void  orc_gelu(const float* x, long n, float* y);
void  orc_softmax_rows(const float* s, long rows, int T, float* p);
void  orc_int_gemm(const uint8_t* a, long M, int K, int za, const int8_t* w, int N, int32_t* acc);
/* source token (y*W+x) of in-window position t of window w under a cyclic shift, or -1 for a pad token */
long  orc_window_token(int H, int W, int ws, int shift, int w, int t);
void  orc_shift_mask(int H, int W, int ws, int shift, int w, float* mask /* [T][T] */);
void  orc_relpos_bias(const float* table, int ws, int heads, float* bias /* [heads][T][T] */);

/* ---- selection (Section 3.2; Section 3.4 for the pruned class) ---- */
void  orc_energy(const float* x, int B, int H, int W, int C, float inv_scale, int32_t* energy);
void  orc_window_scores(const int32_t* energy, int B, int H, int W, int ws, int shift, int64_t* scores);
/* order[b][j]: window index with rank j (score descending, index ascending; reversed when reverse=1);
 * cls[b][w] in {0 high, 1 low, 2 pruned}; counts = {n_hi, n_lo, n_pr} per image */
void  orc_select(const int64_t* scores, int B, int nW, double low_ratio, double prune_ratio, int reverse,
                 int32_t* order, uint8_t* cls, int* counts);

/* ---- the block, the separately written uniform block, merging and the backbone ---- */
/* energy may be NULL (score this block's own input).  order_out/cls_out/score_out/taps_* may be NULL. */
void  orc_block_forward(const orc_block* p, const float* x, float* y, int B, int H, int W,
                        double low_ratio, double prune_ratio, const int32_t* energy, int reverse,
                        int32_t* order_out, uint8_t* cls_out, int64_t* score_out,
                        const orc_taps* taps_hi, const orc_taps* taps_lo);
/* a uniform quantized Swin block through ONE branch, written separately on the whole map, token by token in global
 * coordinates (norm -> pad -> shift -> partition); shares only the scalar primitives with orc_block_forward.
 * (With quant = 0 it runs the fp-mode windows in natural order.) */
void  orc_uniform_block_forward(const orc_block* p, const orc_branch* br, const float* x, float* y,
                                int B, int H, int W);
void  orc_merge_forward(const orc_merge* m, const float* x, int B, int H, int W, int C, float* y);
/* Calibration observers (Section 4.3: one sample, the FULL feature map calibrates both branches): the floating-point
 * block / merge (quantizers off) and the min, max each quantizer site would see.  ranges = 7 x {min, max} in the order
 * QKV input, q, k, v, proj input, fc1 input, fc2 input, over all rows of all windows (pad rows included).  Pinned in
 * the tests to a textbook block written on the un-windowed map in binary64. */
void  orc_block_observe_fp(const orc_block* p, const orc_branch* br, const float* x, float* y, int B, int H, int W,
                           float* ranges /* [14] */);
void  orc_merge_observe_fp(const orc_merge* m, const float* x, int B, int H, int W, int C, float* y, float* range /* [2] */);
/* blocks: sum(depths) entries; merges: num_stages-1; stage_out: num_stages buffers [B][Hs][Ws][Cs] */
void  orc_backbone_forward(int num_stages, const int* depths, const orc_block* blocks, const orc_merge* merges,
                           const float* x0, float* const* stage_out, int B, int H0, int W0,
                           const double* low_ratio_per_pair, const double* prune_ratio_per_pair,
                           int allow_elevation /* 0: classes are kept within a stage (the paper's default) */,
                           int reverse /* 1: worst-case selection order (Table 4) in every block */);
void  orc_patch_embed(const orc_embed* e, const float* img, int B, int Hi, int Wi, float* x0 /* [B][ceil(Hi/4)][ceil(Wi/4)][C0] */);
void  orc_set_threads(int n);
int   orc_get_threads(void);
#ifdef __cplusplus
}
#endif
#endif
