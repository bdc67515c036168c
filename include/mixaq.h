/* mixaq.h -- C ABI of the B200 (sm_100a) library for the quantized Two-Branch Swin Block forward of MixA-Q.
 *
 * What one block call computes (MixA-Q Section 3.1 "Replace Pruning with MP Execution", Section 3.2
 * "Two-Branch Swin Block", Section 3.4 "Activation Pruning Incorporation"):
 *   1. the feature map is cut into non-overlapping ws x ws windows, after an optional cyclic shift;
 *   2. every window gets an importance score (squared L2 norm of its int8 score codes); per image the
 *      windows are ranked by (score descending, window index ascending); the top ones go to the
 *      high-precision branch, the next ones to the low-precision branch, and (optionally) the lowest ones are
 *      pruned, i.e. forwarded unchanged;
 *   3. each branch runs LN -> window attention -> LN -> FFN on its windows with the SAME integer weights
 *      ("shadow layers") but its own LayerNorm parameters, step sizes, zero points and activation bit width;
 *      all matrix products are integer with int32 accumulation;
 *   4. results are dequantized and scattered back to the un-shifted, un-padded feature map.
 *
 * Conventions
 *   - Every pointer inside the *_params structs, x, y, stage outputs, selections, taps and workspaces is a
 *     DEVICE pointer owned by the caller.  The library never frees them and keeps none past the call, with
 *     one exception: `prepared` buffers are read by every later forward call that gets the same params.
 *   - Alignment: feature maps, weight codes and LayerNorm parameters 16 bytes; workspaces and `prepared` buffers
 *     256 bytes (what cudaMalloc and the usual framework allocators give).  Anything less is refused with
 *     MIXAQ_INVALID_ARG before a launch.
 *   - Feature maps are [B][H][W][C] binary32, channels contiguous.  C must be a multiple of 32, C/heads
 *     must be 32, window must be 7, hidden must be a multiple of 32.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*); they allocate no device memory and do
 *     not synchronise.  Errors found on the host are returned before anything is launched.
 *   - Activation codes are unsigned, `bits` in {8, 4, 2}.  Sub-byte codes are stored bit-packed, little end
 *     first: element e of a row lives in byte e*bits/8 at bit (e*bits) mod 8.
 *   - There is no CPU fallback: without a CUDA device every entry point returns MIXAQ_CUDA_ERROR.
 */
#ifndef MIXAQ_H
#define MIXAQ_H
#include <stddef.h>
#include <stdint.h>
#ifdef __cplusplus
extern "C" {
#endif

typedef int mixaq_status;
#define MIXAQ_OK                    0
#define MIXAQ_INVALID_ARG          (-1)  /* null pointer, ratio outside [0,1], bad bit width ...          */
#define MIXAQ_UNSUPPORTED_SHAPE    (-2)  /* window != 7, C % 32 != 0, C/heads != 32, shift >= window ...  */
#define MIXAQ_WORKSPACE_TOO_SMALL  (-3)
#define MIXAQ_CUDA_ERROR           (-4)  /* a CUDA runtime/driver call failed; see mixaq_last_error()     */
#define MIXAQ_DEVICE_TIMEOUT       (-5)  /* a bounded wait inside a kernel ran out (status word)          */
#define MIXAQ_INTERNAL             (-6)
#define MIXAQ_WORKSPACE_OVERRUN    (-7)  /* a guard zone between two workspace buffers was overwritten     */

typedef struct mixaq_ctx mixaq_ctx;

/* Per-tensor asymmetric activation quantizer (Section 3.2: "independent step sizes and zero points"):
 * q = clamp(rne(x * inv_scale) + zero_point, 0, 2^bits - 1);  x ~ (q - zero_point) * scale. */
typedef struct { int bits; float scale; float inv_scale; int zero_point; } mixaq_aq;

/* Integer weight matrix shared by both branches: signed codes, one per byte, row-major [out][in];
 * per-output-channel step size.  `bits` documents the code range (|code| <= 2^(bits-1)-1). */
typedef struct { const int8_t* codes; const float* scale; int out_features; int in_features; int bits; } mixaq_linear;

/* One branch of a block: private LayerNorms, biases (may alias the other branch's), quantizers.
 * The attention-probability quantizer is implied: `bits` bits, zero point 0, step 1/(2^bits - 1). */
typedef struct {
  const float *ln1_g, *ln1_b, *ln2_g, *ln2_b;
  const float *b_qkv, *b_proj, *b_fc1, *b_fc2;
  mixaq_aq qkv_in, q, k, v, proj_in, fc1_in, fc2_in;
  int bits;
} mixaq_branch;

typedef struct {
  int dim, heads, window, shift, hidden;
  mixaq_linear qkv, proj, fc1, fc2;       /* [3C][C], [C][C], [hidden][C], [C][hidden]                    */
  const float* relpos_table;              /* [(2*window-1)^2][heads] binary32                              */
  mixaq_branch hi, lo;
  float score_inv_scale;                  /* score code = clamp(rne(x * score_inv_scale), -127, 127)       */
  void* prepared;                         /* device buffer of mixaq_block_prepared_bytes(), filled once by */
                                          /* mixaq_block_prepare(); read by every forward call             */
  int byte_codes;                         /* storage of the block's intermediate activation codes in the workspace.
                                             0: bit-packed at the branch's bit width (the default; a 4-bit branch
                                             moves half the bytes of an 8-bit one).  1: one code per byte whatever
                                             the bit width -- the same code values in [0, 2^bits), no expansion in
                                             shared memory before the integer MMAs; for maps with many channels,
                                             where one row tile is read by many column tiles and the codes stay in
                                             L2, that expansion costs more than the bytes save.  Taps then hold one
                                             code per byte too.  Workspace sizes depend on this field. */
} mixaq_block_params;

/* Patch merging between stages: 2x2 neighbours concatenated (zero padding for odd sizes) -> LN(4C) ->
 * quantize (`in`) -> integer GEMM with `reduction` [2C][4C], no bias.  (The paper's "downsampling layers",
 * Appendix 6.2: their cost is not reduced by the method.) */
typedef struct { const float *ln_g, *ln_b; mixaq_aq in; mixaq_linear reduction; void* prepared; } mixaq_merge_params;

/* Patch embedding in front of the backbone: 4x4 patches of an [B][Hi][Wi][3] binary32 image (zero padded to
 * multiples of 4; patch vector index (ky*4 + kx)*3 + c) -> quantize (`in`, all tokens at the high bit width) ->
 * integer projection [C0][48] -> (float)acc * (s_in*s_w[n]) + bias[n] -> LayerNorm(C0).  Like patch merging it is one
 * of the layers whose cost the method does not reduce (Appendix 6.2).  C0 must be a multiple of 32. */
typedef struct { const float *ln_g, *ln_b, *bias; mixaq_aq in; mixaq_linear proj; void* prepared; } mixaq_embed_params;

typedef struct {
  const int32_t* energy;   /* optional [B][H][W] token energies computed at stage entry (Section 3.2: the score is
                              computed once per stage and shared); NULL: score this block's own input x      */
  int reverse;             /* 0: highest scores go high.  1: worst-case order (Table 4): lowest scores go high */
} mixaq_select_opts;

/* Optional selection outputs (each pointer may be NULL). */
typedef struct {
  uint8_t* cls;            /* [B][nW]  0 high, 1 low, 2 pruned                                              */
  int32_t* order;          /* [B][nW]  window index by rank: first n_hi high, next n_lo low, last n_pr pruned */
  int64_t* score;          /* [B][nW]  window scores                                                         */
  int32_t *idx_hi, *idx_lo, *idx_pr;   /* [B][n_hi], [B][n_lo], [B][n_pr]: the windows of each class per image, in
                                          ascending window index (the counts are those of mixaq_branch_counts)   */
} mixaq_selection;

/* Optional debug taps of one branch (each pointer may be NULL).  Rows are in window-batch order: window slot
 * s = image * n_branch + rank-within-branch, row = s*49 + in-window token.  Code tensors are bit-packed at the
 * branch's bit width (one code per byte when the block's byte_codes is set); accumulators are zero-point corrected int32. */
typedef struct {
  uint8_t* a_codes;   int32_t* qkv_acc;  uint8_t* qkv_codes;
  float*   probs;     /* [slots][heads][49][49], the binary32 softmax output before its quantizer */
  uint8_t* p_codes;   /* [slots][heads][49][49], one code per byte */
  int32_t* pv_acc;    uint8_t* o_codes;  int32_t* proj_acc;  float* x1;
  uint8_t* f1_codes;  int32_t* fc1_acc;  uint8_t* f2_codes;  int32_t* fc2_acc;
} mixaq_branch_taps;
typedef struct { mixaq_branch_taps hi, lo; } mixaq_taps;

typedef struct {
  int num_stages;
  const int* depths;                    /* HOST array [num_stages]; every depth is even or 1                */
  const mixaq_block_params* blocks;     /* HOST array, sum(depths) entries                                  */
  const mixaq_merge_params* merges;     /* HOST array, num_stages-1 entries                                 */
  /* Optional steps on either side of the path (Appendix 6.2 counts them among the layers whose cost is not reduced).
   * embed != NULL: the `x0` argument of mixaq_backbone_forward is the IMAGE [B][H0][W0][3] and the patch embedding
   * runs first (the token map is ceil(H0/4) x ceil(W0/4)).  out_norm_g / out_norm_b != NULL (HOST arrays of
   * num_stages device pointers, both or neither): stage_out[s] receives LayerNorm(stage map s) with these parameters,
   * while the un-normalised map (kept in the workspace) feeds the next stage. */
  const mixaq_embed_params* embed;
  const float* const* out_norm_g;
  const float* const* out_norm_b;
} mixaq_backbone_params;

/* ---- context ---- */
/* Creates a context on `device` (makes it current).  Holds the status word, the captured graphs of
 * mixaq_backbone_forward and the profiling events. */
mixaq_status mixaq_create(mixaq_ctx** ctx, int device);
mixaq_status mixaq_destroy(mixaq_ctx* ctx);
/* Text of the last host-side error of this context (static storage, valid until the next call). */
const char*  mixaq_last_error(const mixaq_ctx* ctx);
/* Reads the device status word (synchronises `cuda_stream`): MIXAQ_OK, MIXAQ_DEVICE_TIMEOUT, or
 * MIXAQ_WORKSPACE_OVERRUN (see mixaq_set_workspace_guards; reported in preference to a time-out). */
mixaq_status mixaq_last_device_status(mixaq_ctx* ctx, void* cuda_stream);

/* Clears the status word (asynchronous on the stream). */
mixaq_status mixaq_clear_device_status(mixaq_ctx* ctx, void* cuda_stream);
/* Self-test of the failure path: launches one tiny CTA that waits, with the kernels' bounded wait, on a barrier that
 * nothing signals.  The wait runs out after about a millisecond, the CTA raises the status word and returns normally;
 * mixaq_last_device_status then reports MIXAQ_DEVICE_TIMEOUT and the context stays usable (clear the word with
 * mixaq_clear_device_status).  No copy engine, tensor memory or invalid access is involved. */
mixaq_status mixaq_selftest_wait_timeout(mixaq_ctx* ctx, void* cuda_stream);

/* ---- the one definition of "how many windows does a ratio take out of n": floor(ratio*n + 1e-6) ---- */
int          mixaq_low_count(float ratio, int n);
/* counts[3] = {n_hi, n_lo, n_pr} per image for an H x W map: n_pr = cnt(prune, nW), n_lo = cnt(low, nW-n_pr). */
mixaq_status mixaq_branch_counts(int H, int W, int window, float low_ratio, float prune_ratio, int* counts);

/* ---- one-time preparation of derived tables (column sums for the zero-point correction, step-size
 *      products, expanded relative-position bias).  Asynchronous on the stream. ---- */
size_t       mixaq_block_prepared_bytes(const mixaq_block_params* p);
mixaq_status mixaq_block_prepare(mixaq_ctx* ctx, const mixaq_block_params* p, void* cuda_stream);
size_t       mixaq_merge_prepared_bytes(const mixaq_merge_params* p);
mixaq_status mixaq_merge_prepare(mixaq_ctx* ctx, const mixaq_merge_params* p, void* cuda_stream);

/* ---- stage-entry scoring (Section 3.2): energy[b][y][x] = sum_c code(x[b][y][x][c])^2 ---- */
mixaq_status mixaq_stage_energy(mixaq_ctx* ctx, const float* x, int32_t* energy, int B, int H, int W, int C,
                                float score_inv_scale, void* cuda_stream);

/* ---- one Two-Branch Swin Block (Section 3.2, Figure 3).  x and y must not overlap. ---- */
size_t       mixaq_block_workspace_bytes(const mixaq_block_params* p, int B, int H, int W);
mixaq_status mixaq_block_forward(mixaq_ctx* ctx, const mixaq_block_params* p,
                                 const float* x, float* y, int B, int H, int W,
                                 float low_ratio, float prune_ratio,
                                 const mixaq_select_opts* opts /* nullable */,
                                 const mixaq_selection* sel_out /* nullable */,
                                 void* workspace, size_t workspace_bytes,
                                 const mixaq_taps* taps /* nullable */, void* cuda_stream);

/* ---- patch merging alone: x [B][H][W][C] -> y [B][ceil(H/2)][ceil(W/2)][2C] ---- */
size_t       mixaq_merge_workspace_bytes(const mixaq_merge_params* p, int B, int H, int W);
mixaq_status mixaq_merge_forward(mixaq_ctx* ctx, const mixaq_merge_params* p, const float* x, float* y,
                                 int B, int H, int W, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---- patch merging without a workspace (the paper has no counterpart: this entry point exists for the way the
 *      library is deployed, not for the method).  Same result as mixaq_merge_forward, bit for bit, but the
 *      intermediate code matrix lives in an array built into the library, so the call asks the caller for no
 *      workspace and allocates nothing itself (no cudaMalloc / cudaFree, no allocating library routine).
 *      It is meant for callers that cannot obtain device memory where they run the network: a plug-in inside
 *      an application whose own pool holds the whole device, a frame loop that must not hit the device-wide
 *      synchronisation an allocation implies, a process whose policy forbids driver allocations after start-up.
 *      x, y, the parameters and `prepared` are still the caller's, as for mixaq_merge_forward.
 *      Limits and rules:
 *        - the code matrix, B*ceil(H/2)*ceil(W/2) rows of 4C*in.bits/8 bytes, must fit in
 *          MIXAQ_STATIC_SCRATCH_BYTES; larger problems are refused with MIXAQ_WORKSPACE_TOO_SMALL (the text
 *          of mixaq_last_error names both sizes) before anything is launched;
 *        - every GPU that loads the library holds MIXAQ_STATIC_SCRATCH_BYTES of device memory until the
 *          process exits, used or not;
 *        - the first call on each device looks up the array's device address (with that device current);
 *          make that first call outside any stream capture;
 *        - all calls on one device share the one array: two calls whose kernels can overlap on the GPU (different
 *          streams, no ordering between them) race on it.  Calls ordered on one stream are safe.  The array
 *          keeps the previous call's bytes; each call rewrites every byte it later reads, so nothing is cleared. ---- */
#define MIXAQ_STATIC_SCRATCH_BYTES (8u << 20)
mixaq_status mixaq_merge_forward_static(mixaq_ctx* ctx, const mixaq_merge_params* p, const float* x, float* y,
                                        int B, int H, int W, void* cuda_stream);

/* ---- patch embedding (the step in front of the path) and LayerNorm of a stage output (the step behind it).
 *      image [B][Hi][Wi][3] -> x0 [B][ceil(Hi/4)][ceil(Wi/4)][C0], the input of mixaq_backbone_forward.
 *      mixaq_norm_forward: y = LayerNorm(x) over the last axis of a [rows][C] binary32 matrix (x and y may alias). ---- */
size_t       mixaq_embed_prepared_bytes(const mixaq_embed_params* p);
mixaq_status mixaq_embed_prepare(mixaq_ctx* ctx, const mixaq_embed_params* p, void* cuda_stream);
size_t       mixaq_embed_workspace_bytes(const mixaq_embed_params* p, int B, int Hi, int Wi);
mixaq_status mixaq_embed_forward(mixaq_ctx* ctx, const mixaq_embed_params* p, const float* image, float* x0,
                                 int B, int Hi, int Wi, void* workspace, size_t workspace_bytes, void* cuda_stream);
mixaq_status mixaq_norm_forward(mixaq_ctx* ctx, const float* gamma, const float* beta, const float* x, float* y,
                                long rows, int C, void* cuda_stream);

/* ---- calibration of the activation quantizers (Section 4.3, post-training flow): one calibration sample, and the
 *      FULL feature map (every window, whatever branch it will later run in) sets the ranges of BOTH branches, which
 *      then differ only in bit width.  mixaq_calibrate_block runs the floating-point block (all quantizers off,
 *      weights = code x step size) with every window through the LayerNorm parameters and biases of one branch
 *      (branch 0: high, 1: low), writes its output map to y and the minimum / maximum each quantizer site saw to
 *      `ranges` (a HOST struct).  The quantizer fields of `p` are not read and `p->prepared` is not needed.
 *      mixaq_calibrate_merge does the same for a patch merging (one site: the LayerNorm output).
 *      Both synchronise the stream.  mixaq_aq_from_range is the one definition of the quantizer that covers a range:
 *      scale = (hi - lo) / (2^bits - 1), inv_scale = 1 / scale, zero_point = clamp(rne(-lo / scale), 0, 2^bits - 1). ---- */
typedef struct { float lo, hi; } mixaq_range;
typedef struct { mixaq_range qkv_in, q, k, v, proj_in, fc1_in, fc2_in;
                 mixaq_range x_in;   /* the block's input map itself (its largest magnitude sets the score-code step) */
               } mixaq_block_ranges;
size_t       mixaq_calibrate_block_workspace_bytes(const mixaq_block_params* p, int B, int H, int W);
mixaq_status mixaq_calibrate_block(mixaq_ctx* ctx, const mixaq_block_params* p, int branch, const float* x, float* y,
                                   int B, int H, int W, mixaq_block_ranges* ranges,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t       mixaq_calibrate_merge_workspace_bytes(const mixaq_merge_params* p, int B, int H, int W);
mixaq_status mixaq_calibrate_merge(mixaq_ctx* ctx, const mixaq_merge_params* p, const float* x, float* y,
                                   int B, int H, int W, mixaq_range* range,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);
mixaq_status mixaq_aq_from_range(float lo, float hi, int bits, mixaq_aq* out);

/* ---- the backbone: for every stage [merge] -> stage energy -> blocks; one ratio per pair of consecutive
 *      blocks (Section 3.3), optional prune ratio per pair (Section 3.4).  x0 is the [B][H0][W0][C0] map after the
 *      patch-embedding stem (or, when p->embed is set, the [B][H0][W0][3] image itself); stage_out is a HOST array of
 *      num_stages device pointers receiving each stage's final map [B][Hs][Ws][Cs] (normalised when p->out_norm_* are
 *      set).  Ratio arrays are HOST arrays with one entry per block pair. ---- */
size_t       mixaq_backbone_workspace_bytes(const mixaq_backbone_params* p, int B, int H0, int W0);
mixaq_status mixaq_backbone_forward(mixaq_ctx* ctx, const mixaq_backbone_params* p, const float* x0,
                                    float* const* stage_out, int B, int H0, int W0,
                                    const float* low_ratio_per_pair, const float* prune_ratio_per_pair /* nullable */,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* mixaq_backbone_forward replays a CUDA graph when it is called again with exactly the same arguments (same
 * parameter structs byte for byte, pointers, sizes, ratios, workspace and stream): the first such call captures the
 * launches on `cuda_stream`, later calls cost one graph launch on the host.  The data behind the pointers may
 * change freely between calls.  Captured graphs are kept per context (16 at most) until mixaq_destroy.  Caching
 * needs a stream that can be captured: calls on the legacy default stream (NULL), calls made while the caller is
 * capturing the stream itself launch their kernels directly.  A call between mixaq_profile_begin/end is captured
 * together with its event records, launched once and not cached.
 * enabled = 0 switches the cache off and drops the stored graphs; it is on by default. */
mixaq_status mixaq_set_graph_cache(mixaq_ctx* ctx, int enabled);

/* Within a stage windows keep their precision class (Section 4.4, "Windows Elevation": letting compressed windows
 * return to high precision in later blocks is the paper's ablation, not its default).  mixaq_backbone_forward
 * therefore uses, for every block pair, the largest low-bit ratio and the largest prune ratio of the stage's pairs so
 * far, so the set of non-high windows never shrinks inside a stage.  allow = 1 makes every pair use its own ratios. */
mixaq_status mixaq_set_window_elevation(mixaq_ctx* ctx, int allow);

/* Worst-case window selection for mixaq_backbone_forward (Table 4: "importance in reverse order"): the LOWEST
 * scores go to the high-precision branch in every block.  Off by default; the block call has the same switch in
 * mixaq_select_opts. */
mixaq_status mixaq_set_reverse_selection(mixaq_ctx* ctx, int reverse);

/* Debug aid against out-of-bounds writes.  Every buffer the library carves out of a caller's workspace is followed by
 * a 256-byte guard zone (always; the *_workspace_bytes figures include them).  enabled = 1: mixaq_block_forward (also
 * as part of mixaq_backbone_forward) writes a pattern into the zones of the block's workspace before its first kernel
 * and compares them after its last; a difference raises the status word (MIXAQ_WORKSPACE_OVERRUN from
 * mixaq_last_device_status).  Two small launches per block; off by default. */
mixaq_status mixaq_set_workspace_guards(mixaq_ctx* ctx, int enabled);
/* Self-test of that check on a caller's buffer (>= 2 KiB of device memory): two 256-byte buffers are carved out of
 * it, their guard zones filled, and, with overrun = 1, one byte just past the second buffer is written (inside the
 * caller's memory) before the zones are compared. */
mixaq_status mixaq_selftest_workspace_guards(mixaq_ctx* ctx, void* buffer, size_t bytes, int overrun, void* cuda_stream);

/* NVTX ranges for external tracers (off by default): every kernel family launched through this context is wrapped in
 * a host-side range named like its profiling category, and mixaq_backbone_forward adds one range per stage and per
 * block.  The ranges mark where the launches are ISSUED: a forward that replays a cached graph issues none, so trace
 * with the graph cache off (mixaq_set_graph_cache) to see them. */
mixaq_status mixaq_set_nvtx(mixaq_ctx* ctx, int enabled);

/* Number of kernel launches the last block / merge / backbone call of this context issued. */
int          mixaq_last_launch_count(const mixaq_ctx* ctx);

/* ---- tensor-core issue rate as this library reaches it (the denominator for the GEMMs' tensor-pipe fraction, and the
 *      measurement behind the choice of MMA kind for the low-bit branch):
 *      all SMs at once issue `groups` x 4 tcgen05.mma of 128 x 256 x K from shared-memory operands into TMEM.
 *      kind 0: kind::i8 (u8 x s8 -> s32, K = 32), the path the GEMMs use.
 *      kind 1: kind::f8f6f4 with E4M3 operands (K = 32), the path that also carries the 4-bit and 6-bit operand formats
 *              in 8-bit containers: its rate bounds what those formats could give.
 *      kind 2: kind::mxf4, block-scaled E2M1 operands packed two per byte (K = 64, one UE8M0 scale per 32 values; the
 *              scale factors are left uninitialised, so the products mean nothing -- only the rate is measured).
 *      `scratch`: >= 8 KiB of device memory.  Synchronises the stream; result in 10^12 operations (2 per
 *      multiply-accumulate) per second. ---- */
mixaq_status mixaq_measure_mma_peak(mixaq_ctx* ctx, int kind, int groups, void* scratch, size_t scratch_bytes,
                                    double* tera_ops_per_s, void* cuda_stream);

/* ---- per-kernel timing (the paper reports no time breakdown; this is the library's own tracing aid).
 *      Between begin and end every kernel family launched through this context is bracketed by CUDA events on
 *      the launching stream.  end() synchronises the stream and returns, per category (see
 *      mixaq_profile_category_name), the summed device milliseconds and the number of event pairs; both HOST
 *      arrays have mixaq_profile_categories() entries.  A backbone forward on a capturable stream is timed as it runs
 *      inside its graph (the event records are graph nodes); other calls are timed as stream launches, which adds the
 *      launch gap to every kernel.  Category "empty_event_bracket": four event pairs per backbone
 *      forward with nothing between them -- what a bracket by itself adds to a kernel's figure. ---- */
int          mixaq_profile_categories(void);
const char*  mixaq_profile_category_name(int category);
mixaq_status mixaq_profile_begin(mixaq_ctx* ctx);
mixaq_status mixaq_profile_end(mixaq_ctx* ctx, void* cuda_stream, float* ms_per_category, int* launches_per_category);
/* The same, launch by launch in issue order: fills category[i] and ms[i] for the first `capacity` bracketed launches
 * since mixaq_profile_begin and stores their total number in *count (which may exceed capacity).  Ends the profiling
 * like mixaq_profile_end. */
mixaq_status mixaq_profile_end_records(mixaq_ctx* ctx, void* cuda_stream, int* category, float* ms, int capacity, int* count);

#ifdef __cplusplus
}
#endif
#endif /* MIXAQ_H */
