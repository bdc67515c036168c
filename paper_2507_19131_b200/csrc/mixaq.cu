// Host side of the C ABI declared in include/mixaq.h: argument validation, workspace carving, the launch
// schedule of one Two-Branch Swin Block (MixA-Q Section 3.2, Figure 3) and of the backbone loop.
// Nothing here computes: every step of the path runs in the kernels.
#include <nvtx3/nvToolsExt.h>
#include "../../include/mixaq.h"
#include "kernels.h"
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

namespace mixaq {
bool ln_dim_supported(int C);
bool merge_dim_supported(int C);
thread_local int g_launches = 0;
}  // namespace mixaq

using namespace mixaq;

struct ProfRec { int cat; cudaEvent_t e0, e1; };
// One captured backbone forward: the exact bytes of every argument that shaped it, and the instantiated graph.
struct GraphEntry { std::string key; cudaGraphExec_t exec; int launches; };
struct mixaq_ctx {
  int device;
  int* d_status;
  int launches;
  char err[256];
  bool profiling;
  bool graph_cache;                    // replay backbone forwards as CUDA graphs (see mixaq_set_graph_cache)
  bool reverse_selection;              // backbone: worst-case selection order (Table 4) in every block
  bool prof_capture;                   // the profiled call is being captured: event records become graph nodes
  std::vector<cudaGraphExec_t> prof_execs;   // graphs of profiled forwards, destroyed when the profiling ends
  bool guards;                         // fill the guard zones of the workspace before a forward, compare them after it
  bool nvtx;                           // name every kernel family, stage and block with an NVTX range (host side)
  bool allow_elevation;                // backbone: every pair uses its own ratios even if an earlier pair of the stage had larger ones
  std::vector<GraphEntry> graphs;
  std::vector<ProfRec> prof;          // event pairs recorded since mixaq_profile_begin
  std::vector<cudaEvent_t> pool;      // events ready for reuse
};

namespace mixaq {
// accessors for translation units that do not see the context's layout
int* ctx_status_word(mixaq_ctx* ctx) { return ctx->d_status; }
int ctx_device(const mixaq_ctx* ctx) { return ctx->device; }
void ctx_note(mixaq_ctx* ctx, const char* msg, int launches) {
  if (msg) snprintf(ctx->err, sizeof(ctx->err), "%s", msg);
  ctx->launches = launches;
}
}  // namespace mixaq

enum ProfCat { PC_ENERGY = 0, PC_SELECT, PC_LN1, PC_QKV, PC_ATTN, PC_PROJ, PC_LN2, PC_FC1, PC_FC2, PC_COPY,
               PC_MERGE_GATHER, PC_MERGE_GEMM, PC_STEM, PC_OUT_NORM, PC_BRACKET, PC_COUNT };
static const char* kProfNames[PC_COUNT] = {"energy", "select", "gather_ln1_quant", "gemm_qkv", "attention",
                                           "gemm_proj", "ln2_quant", "gemm_fc1_gelu", "gemm_fc2_scatter",
                                           "copy_pruned", "merge_gather_ln_quant", "gemm_merge", "patch_embed",
                                           "stage_output_norm", "empty_event_bracket"};

namespace {

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }
// The kernels read and write feature maps, parameters and codes with 16-byte accesses and describe operand matrices
// to the TMA unit (16-byte aligned base); workspaces and prepared buffers are carved in 256-byte steps.  A pointer
// that breaks this would fault on the device, so it is refused on the host.
inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Every buffer carved out of a workspace is followed by a guard zone of GUARD_BYTES that no kernel has a reason to
// touch.  With mixaq_set_workspace_guards the zones are filled with a pattern before a forward and compared after it.
thread_local std::vector<void*>* t_guard_log = nullptr;     // where the carver notes its guard zones (NULL: nowhere)
struct Carver {
  char* base; size_t off; bool guarded;
  // guarded = false: the `prepared` parameter tables, written once by the prepare calls (their layout is also read by
  // code that does not carve)
  explicit Carver(void* p, bool with_guards = true) : base((char*)p), off(0), guarded(with_guards) {}
  template <class T> T* take(size_t n) {
    T* p = base ? (T*)(base + off) : nullptr;
    off += align_up(n * sizeof(T));
    if (guarded) {
      if (base && t_guard_log) t_guard_log->push_back(base + off);
      off += GUARD_BYTES;
    }
    return p;
  }
};
// bytes a guarded carver needs for one buffer of n bytes
inline size_t carved_bytes(size_t n) { return align_up(n) + GUARD_BYTES; }
// scope in which carvers log their guard zones into `list` (when the context asks for guards)
struct GuardScope {
  std::vector<void*>* prev;
  GuardScope(const mixaq_ctx* ctx, std::vector<void*>* list) : prev(t_guard_log) { t_guard_log = (ctx && ctx->guards) ? list : nullptr; }
  ~GuardScope() { t_guard_log = prev; }
};

AQ to_aq(const mixaq_aq& q) {
  AQ a; a.scale = q.scale; a.inv_scale = q.inv_scale; a.zp = q.zero_point; a.bits = q.bits;
  a.zpf = (float)q.zero_point; a.qmaxf = (float)((1 << q.bits) - 1);
  return a;
}

mixaq_status fail(mixaq_ctx* ctx, mixaq_status s, const char* msg) {
  if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%s", msg);
  return s;
}

mixaq_status check_cuda(mixaq_ctx* ctx, const char* where) {
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) return MIXAQ_OK;
  if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%s: %s", where, cudaGetErrorString(e));
  return MIXAQ_CUDA_ERROR;
}

// Per-kernel CUDA-event timing (only while profiling is on; the events sit on the launching stream).
struct ProfScope {
  mixaq_ctx* ctx; cudaStream_t st; cudaEvent_t e1; bool on, range;
  ProfScope(mixaq_ctx* c, int cat, cudaStream_t s) : ctx(c), st(s), e1(nullptr), on(c && c->profiling), range(c && c->nvtx) {
    if (range) nvtxRangePushA(kProfNames[cat]);
    if (!on) return;
    cudaEvent_t ev[2];
    for (int i = 0; i < 2; ++i) {
      if (!ctx->pool.empty()) { ev[i] = ctx->pool.back(); ctx->pool.pop_back(); }
      else if (cudaEventCreate(&ev[i]) != cudaSuccess) { on = false; return; }
    }
    record(ev[0]);
    e1 = ev[1];
    ctx->prof.push_back({cat, ev[0], ev[1]});
  }
  // inside a stream capture the record becomes a graph node of its own (an "external" event keeps its timestamp)
  void record(cudaEvent_t e) {
    if (ctx->prof_capture) cudaEventRecordWithFlags(e, st, cudaEventRecordExternal);
    else cudaEventRecord(e, st);
  }
  ~ProfScope() { if (on) record(e1); if (range) nvtxRangePop(); }
};
// NVTX range over a stage or a block of the backbone walk (only with mixaq_set_nvtx)
struct NvtxScope {
  bool on;
  NvtxScope(const mixaq_ctx* c, const char* what, int index) : on(c && c->nvtx) {
    if (!on) return;
    char name[48];
    snprintf(name, sizeof(name), "%s %d", what, index);
    nvtxRangePushA(name);
  }
  ~NvtxScope() { if (on) nvtxRangePop(); }
};
#define PROF(cat) ProfScope prof_scope_##cat(ctx, cat, st)

bool bits_ok(int b) { return b == 8 || b == 4 || b == 2; }
bool aq_ok(const mixaq_aq& q, int bits) {
  return q.bits == bits && q.scale > 0.f && q.inv_scale > 0.f && q.zero_point >= 0 && q.zero_point < (1 << bits);
}
bool linear_ok(const mixaq_linear& l, int out_f, int in_f) {
  return l.codes && l.scale && l.out_features == out_f && l.in_features == in_f;
}
bool branch_ok(const mixaq_branch& b) {
  if (!bits_ok(b.bits)) return false;
  if (!b.ln1_g || !b.ln1_b || !b.ln2_g || !b.ln2_b || !b.b_qkv || !b.b_proj || !b.b_fc1 || !b.b_fc2) return false;
  return aq_ok(b.qkv_in, b.bits) && aq_ok(b.q, b.bits) && aq_ok(b.k, b.bits) && aq_ok(b.v, b.bits) &&
         aq_ok(b.proj_in, b.bits) && aq_ok(b.fc1_in, b.bits) && aq_ok(b.fc2_in, b.bits);
}

bool branch_ptrs_ok(const mixaq_branch& b) {
  return b.ln1_g && b.ln1_b && b.ln2_g && b.ln2_b && b.b_qkv && b.b_proj && b.b_fc1 && b.b_fc2;
}

// need_quantizers = false: the calibration pass, which runs before any quantizer exists
mixaq_status validate_block(mixaq_ctx* ctx, const mixaq_block_params* p, bool need_quantizers = true) {
  if (!p) return fail(ctx, MIXAQ_INVALID_ARG, "block params are NULL");
  if (p->window != WS) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "window must be 7");
  if (p->dim <= 0 || p->dim % 32 || !ln_dim_supported(p->dim)) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "unsupported dim");
  if (p->heads <= 0 || p->dim != p->heads * HEAD_DIM) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "dim/heads must be 32");
  if (p->hidden <= 0 || p->hidden % 32) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "hidden must be a multiple of 32");
  if (p->shift < 0 || p->shift >= WS) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "shift must be in [0, window)");
  if (!linear_ok(p->qkv, 3 * p->dim, p->dim) || !linear_ok(p->proj, p->dim, p->dim) ||
      !linear_ok(p->fc1, p->hidden, p->dim) || !linear_ok(p->fc2, p->dim, p->hidden))
    return fail(ctx, MIXAQ_INVALID_ARG, "weight matrix missing or of the wrong shape");
  if (!p->relpos_table) return fail(ctx, MIXAQ_INVALID_ARG, "relpos_table is NULL");
  {
    const void* q16[] = {p->qkv.codes, p->proj.codes, p->fc1.codes, p->fc2.codes,
                         p->hi.ln1_g, p->hi.ln1_b, p->hi.ln2_g, p->hi.ln2_b, p->lo.ln1_g, p->lo.ln1_b, p->lo.ln2_g, p->lo.ln2_b};
    for (const void* q : q16)
      if (!aligned_to(q, 16)) return fail(ctx, MIXAQ_INVALID_ARG, "weight codes and LayerNorm parameters must be 16-byte aligned");
    if (p->prepared && !aligned_to(p->prepared, 256)) return fail(ctx, MIXAQ_INVALID_ARG, "prepared buffer must be 256-byte aligned");
  }
  if (p->byte_codes != 0 && p->byte_codes != 1) return fail(ctx, MIXAQ_INVALID_ARG, "byte_codes must be 0 or 1");
  if (!need_quantizers) {
    if (!branch_ptrs_ok(p->hi) || !branch_ptrs_ok(p->lo)) return fail(ctx, MIXAQ_INVALID_ARG, "branch parameters invalid");
    return MIXAQ_OK;
  }
  if (!branch_ok(p->hi) || !branch_ok(p->lo)) return fail(ctx, MIXAQ_INVALID_ARG, "branch parameters invalid");
  if (!(p->score_inv_scale > 0.f)) return fail(ctx, MIXAQ_INVALID_ARG, "score_inv_scale must be positive");
  return MIXAQ_OK;
}

// layout of a block's prepared buffer
struct Prepared {
  float* mult[4][2]; int32_t* zc[4][2]; float* relbias; size_t bytes;
};
Prepared carve_prepared(const mixaq_block_params* p, void* base) {
  Prepared r; Carver c(base, false);
  const int N[4] = {3 * p->dim, p->dim, p->hidden, p->dim};
  for (int l = 0; l < 4; ++l)
    for (int b = 0; b < 2; ++b) { r.mult[l][b] = c.take<float>(N[l]); r.zc[l][b] = c.take<int32_t>(N[l]); }
  r.relbias = c.take<float>((size_t)p->heads * 4 * 7 * 32 * 4);   // fragment order, see k_prepare_relbias
  r.bytes = c.off;
  return r;
}

struct Geometry { int Hp, Wp, nwx, nW, n_hi, n_lo, n_pr; };
Geometry geometry(int H, int W, float low, float prune) {
  Geometry g;
  g.Hp = (H + WS - 1) / WS * WS; g.Wp = (W + WS - 1) / WS * WS;
  g.nwx = g.Wp / WS; g.nW = (g.Hp / WS) * g.nwx;
  g.n_pr = mixaq_low_count(prune, g.nW);
  g.n_lo = mixaq_low_count(low, g.nW - g.n_pr);
  g.n_hi = g.nW - g.n_pr - g.n_lo;
  return g;
}

// buffers the selection kernels fill for one block (all sized for the worst split)
struct SelWs {
  int64_t* score; int32_t* order; uint8_t* cls; int32_t *rowsrc[3], *win[2]; size_t bytes;
};
SelWs carve_sel(int B, int H, int W, void* base) {
  SelWs w; Carver c(base);
  Geometry g = geometry(H, W, 0.f, 0.f);
  const size_t slots = (size_t)B * g.nW, rows = slots * WT;
  w.score = c.take<int64_t>(slots); w.order = c.take<int32_t>(slots); w.cls = c.take<uint8_t>(slots);
  for (int i = 0; i < 3; ++i) w.rowsrc[i] = c.take<int32_t>(rows);
  for (int i = 0; i < 2; ++i) w.win[i] = c.take<int32_t>(slots);
  w.bytes = c.off;
  return w;
}

// workspace of one block call; sized for the worst split (all windows in the wider branch)
struct BlockWs {
  int32_t* energy; SelWs sel;
  uint8_t *a[2], *qkv[2], *o[2], *f1[2], *f2[2]; float* x1[2];
  size_t bytes;
};
BlockWs carve_block(const mixaq_block_params* p, int B, int H, int W, void* base) {
  BlockWs w; Carver c(base);
  Geometry g = geometry(H, W, 0.f, 0.f);
  const size_t slots = (size_t)B * g.nW, rows = slots * WT;
  const int C = p->dim, Hd = p->hidden;
  w.energy = c.take<int32_t>((size_t)B * H * W);
  w.sel = carve_sel(B, H, W, base ? (char*)base + c.off : nullptr);
  c.off += w.sel.bytes;
  for (int i = 0; i < 2; ++i) {
    const int bits = p->byte_codes ? 8 : (i == 0 ? p->hi.bits : p->lo.bits);     // container of a code
    w.a[i]   = c.take<uint8_t>(rows * C * bits / 8);
    w.qkv[i] = c.take<uint8_t>(rows * 3 * C * bits / 8);
    w.o[i]   = c.take<uint8_t>(rows * C * bits / 8);
    w.x1[i]  = c.take<float>(rows * C);
    w.f1[i]  = c.take<uint8_t>(rows * C * bits / 8);
    w.f2[i]  = c.take<uint8_t>(rows * Hd * bits / 8);
  }
  w.bytes = c.off;
  return w;
}

SelectArgs make_select_args(const SelWs& sel, const int32_t* energy, int B, int H, int W, int shift, const Geometry& g,
                            int reverse) {
  SelectArgs sa;
  sa.energy = energy; sa.score = sel.score; sa.order = sel.order; sa.cls = sel.cls;
  sa.rowsrc_hi = sel.rowsrc[0]; sa.rowsrc_lo = sel.rowsrc[1]; sa.rowsrc_pr = sel.rowsrc[2];
  sa.win_hi = sel.win[0]; sa.win_lo = sel.win[1];
  sa.B = B; sa.H = H; sa.W = W; sa.shift = shift; sa.nwx = g.nwx; sa.nW = g.nW;
  sa.n_hi = g.n_hi; sa.n_lo = g.n_lo; sa.n_pr = g.n_pr; sa.reverse = reverse;
  return sa;
}

void fill_gemm_branch(GemmBranch& g, const uint8_t* a, int M, int a_bits, const float* mult, const int32_t* zc,
                      const float* bias) {
  memset(&g, 0, sizeof(g));
  g.a = a; g.M = M; g.a_bits = a_bits; g.mult = mult; g.zc = zc; g.bias = bias;
}

}  // namespace

// =================================================================================================
extern "C" {

int mixaq_low_count(float ratio, int n) { return (int)std::floor((double)ratio * (double)n + 1e-6); }

mixaq_status mixaq_branch_counts(int H, int W, int window, float low_ratio, float prune_ratio, int* counts) {
  if (!counts || window != WS || H <= 0 || W <= 0) return MIXAQ_INVALID_ARG;
  if (!(low_ratio >= 0.f && low_ratio <= 1.f) || !(prune_ratio >= 0.f && prune_ratio <= 1.f)) return MIXAQ_INVALID_ARG;
  Geometry g = geometry(H, W, low_ratio, prune_ratio);
  counts[0] = g.n_hi; counts[1] = g.n_lo; counts[2] = g.n_pr;
  return MIXAQ_OK;
}

mixaq_status mixaq_create(mixaq_ctx** out, int device) {
  if (!out) return MIXAQ_INVALID_ARG;
  *out = nullptr;
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) { cudaGetLastError(); return MIXAQ_CUDA_ERROR; }
  if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return MIXAQ_CUDA_ERROR; }
  mixaq_ctx* c = new (std::nothrow) mixaq_ctx();
  if (!c) return MIXAQ_INTERNAL;
  c->device = device; c->launches = 0; c->err[0] = 0; c->d_status = nullptr; c->profiling = false; c->graph_cache = true; c->allow_elevation = false; c->reverse_selection = false; c->nvtx = false; c->prof_capture = false; c->guards = false;
  if (cudaMalloc(&c->d_status, sizeof(int)) != cudaSuccess || cudaMemset(c->d_status, 0, sizeof(int)) != cudaSuccess ||
      !gemm_init()) {
    cudaGetLastError(); if (c->d_status) cudaFree(c->d_status); delete c; return MIXAQ_CUDA_ERROR;
  }
  *out = c;
  return MIXAQ_OK;
}

mixaq_status mixaq_destroy(mixaq_ctx* ctx) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  if (ctx->d_status) cudaFree(ctx->d_status);
  for (auto& g : ctx->graphs) cudaGraphExecDestroy(g.exec);
  for (cudaGraphExec_t g : ctx->prof_execs) cudaGraphExecDestroy(g);
  for (auto& r : ctx->prof) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
  for (auto e : ctx->pool) cudaEventDestroy(e);
  delete ctx;
  return MIXAQ_OK;
}

const char* mixaq_last_error(const mixaq_ctx* ctx) { return ctx ? ctx->err : "no context"; }
int mixaq_last_launch_count(const mixaq_ctx* ctx) { return ctx ? ctx->launches : 0; }

mixaq_status mixaq_last_device_status(mixaq_ctx* ctx, void* cuda_stream) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  int h = 0;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaMemcpyAsync(&h, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
  { check_cuda(ctx, "status read"); return MIXAQ_CUDA_ERROR; }
  return h == 0 ? MIXAQ_OK : ((h & 2) ? MIXAQ_WORKSPACE_OVERRUN : MIXAQ_DEVICE_TIMEOUT);
}

mixaq_status mixaq_clear_device_status(mixaq_ctx* ctx, void* cuda_stream) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  if (cudaMemsetAsync(ctx->d_status, 0, sizeof(int), (cudaStream_t)cuda_stream) != cudaSuccess) return check_cuda(ctx, "clear status");
  return MIXAQ_OK;
}

mixaq_status mixaq_selftest_wait_timeout(mixaq_ctx* ctx, void* cuda_stream) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  launch_wait_probe(ctx->d_status, (cudaStream_t)cuda_stream);
  return check_cuda(ctx, "selftest_wait_timeout");
}

mixaq_status mixaq_measure_mma_peak(mixaq_ctx* ctx, int kind, int groups, void* scratch, size_t scratch_bytes,
                                    double* tera_ops_per_s, void* cuda_stream) {
  if (!ctx || !scratch || !tera_ops_per_s || groups <= 0 || kind < 0 || kind > 2) return MIXAQ_INVALID_ARG;
  if (scratch_bytes < 1024 * sizeof(unsigned long long)) return fail(ctx, MIXAQ_WORKSPACE_TOO_SMALL, "mma peak: scratch of 8 KiB needed");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  unsigned long long* d_ns = (unsigned long long*)scratch;
  const int sms = launch_mma_peak(kind, groups, d_ns, ctx->d_status, st);
  if (sms <= 0 || sms > 1024) return check_cuda(ctx, "mma peak") == MIXAQ_OK ? MIXAQ_INTERNAL : MIXAQ_CUDA_ERROR;
  std::vector<unsigned long long> ns(sms);
  if (cudaMemcpyAsync(ns.data(), d_ns, sizeof(unsigned long long) * sms, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) return check_cuda(ctx, "mma peak");
  unsigned long long worst = 1;
  for (auto v : ns) worst = v > worst ? v : worst;
  // every SM issued groups x 4 MMAs of 128 x 256 x 32 (kind 2: x 64) multiply-accumulates; all SMs ran at once: the
  // slowest one counts
  const double k_per_mma = kind == 2 ? 64.0 : 32.0;
  const double ops = 2.0 * 128.0 * 256.0 * k_per_mma * 4.0 * (double)groups * (double)sms;
  *tera_ops_per_s = ops / ((double)worst * 1e-9) / 1e12;
  return check_cuda(ctx, "mma peak");
}

int mixaq_profile_categories(void) { return PC_COUNT; }
const char* mixaq_profile_category_name(int cat) { return (cat >= 0 && cat < PC_COUNT) ? kProfNames[cat] : ""; }

mixaq_status mixaq_profile_begin(mixaq_ctx* ctx) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  for (auto& r : ctx->prof) { ctx->pool.push_back(r.e0); ctx->pool.push_back(r.e1); }
  ctx->prof.clear();
  ctx->profiling = true;
  return MIXAQ_OK;
}

mixaq_status mixaq_profile_end(mixaq_ctx* ctx, void* cuda_stream, float* ms_per_category, int* launches_per_category) {
  if (!ctx || !ms_per_category || !launches_per_category) return MIXAQ_INVALID_ARG;
  ctx->profiling = false;
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return check_cuda(ctx, "profile_end");
  for (cudaGraphExec_t g : ctx->prof_execs) cudaGraphExecDestroy(g);
  ctx->prof_execs.clear();
  for (int i = 0; i < PC_COUNT; ++i) { ms_per_category[i] = 0.f; launches_per_category[i] = 0; }
  for (auto& r : ctx->prof) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.e0, r.e1) == cudaSuccess) { ms_per_category[r.cat] += ms; launches_per_category[r.cat] += 1; }
    ctx->pool.push_back(r.e0); ctx->pool.push_back(r.e1);
  }
  ctx->prof.clear();
  return check_cuda(ctx, "profile_end");
}

mixaq_status mixaq_profile_end_records(mixaq_ctx* ctx, void* cuda_stream, int* category, float* ms, int capacity, int* count) {
  if (!ctx || !category || !ms || !count || capacity < 0) return MIXAQ_INVALID_ARG;
  ctx->profiling = false;
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return check_cuda(ctx, "profile_end_records");
  for (cudaGraphExec_t g : ctx->prof_execs) cudaGraphExecDestroy(g);
  ctx->prof_execs.clear();
  int n = 0;
  for (auto& r : ctx->prof) {
    float t = 0.f;
    if (n < capacity) {
      if (cudaEventElapsedTime(&t, r.e0, r.e1) != cudaSuccess) { cudaGetLastError(); t = 0.f; }
      category[n] = r.cat; ms[n] = t;
    }
    ++n;
    ctx->pool.push_back(r.e0); ctx->pool.push_back(r.e1);
  }
  ctx->prof.clear();
  *count = n;
  return check_cuda(ctx, "profile_end_records");
}

// -------------------------------------------------------------------------------------------------
size_t mixaq_block_prepared_bytes(const mixaq_block_params* p) {
  if (!p || p->dim <= 0 || p->hidden <= 0 || p->heads <= 0) return 0;
  return carve_prepared(p, nullptr).bytes;
}

mixaq_status mixaq_block_prepare(mixaq_ctx* ctx, const mixaq_block_params* p, void* cuda_stream) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  mixaq_status s = validate_block(ctx, p);
  if (s != MIXAQ_OK) return s;
  if (!p->prepared) return fail(ctx, MIXAQ_INVALID_ARG, "prepared buffer is NULL");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  Prepared pr = carve_prepared(p, p->prepared);
  const mixaq_linear* L[4] = {&p->qkv, &p->proj, &p->fc1, &p->fc2};
  for (int b = 0; b < 2; ++b) {
    const mixaq_branch& br = b == 0 ? p->hi : p->lo;
    const mixaq_aq* in[4] = {&br.qkv_in, &br.proj_in, &br.fc1_in, &br.fc2_in};
    for (int l = 0; l < 4; ++l)
      launch_prepare_linear(L[l]->codes, L[l]->scale, L[l]->out_features, L[l]->in_features, in[l]->scale,
                            in[l]->zero_point, pr.mult[l][b], pr.zc[l][b], st);
  }
  launch_prepare_relbias(p->relpos_table, p->heads, pr.relbias, st);
  return check_cuda(ctx, "block_prepare");
}

size_t mixaq_merge_prepared_bytes(const mixaq_merge_params* p) {
  if (!p || p->reduction.out_features <= 0) return 0;
  return align_up((size_t)p->reduction.out_features * 4) * 2;
}

mixaq_status mixaq_merge_prepare(mixaq_ctx* ctx, const mixaq_merge_params* p, void* cuda_stream) {
  if (!ctx || !p) return MIXAQ_INVALID_ARG;
  if (!p->prepared || !p->reduction.codes || !p->reduction.scale) return fail(ctx, MIXAQ_INVALID_ARG, "merge params incomplete");
  Carver c(p->prepared, false);
  float* mult = c.take<float>(p->reduction.out_features);
  int32_t* zc = c.take<int32_t>(p->reduction.out_features);
  launch_prepare_linear(p->reduction.codes, p->reduction.scale, p->reduction.out_features, p->reduction.in_features,
                        p->in.scale, p->in.zero_point, mult, zc, (cudaStream_t)cuda_stream);
  return check_cuda(ctx, "merge_prepare");
}

mixaq_status mixaq_stage_energy(mixaq_ctx* ctx, const float* x, int32_t* energy, int B, int H, int W, int C,
                                float score_inv_scale, void* cuda_stream) {
  if (!ctx || !x || !energy || B <= 0 || H <= 0 || W <= 0 || C <= 0 || !(score_inv_scale > 0.f)) return MIXAQ_INVALID_ARG;
  if (!aligned_to(x, 16) || !aligned_to(energy, 4)) return fail(ctx, MIXAQ_INVALID_ARG, "stage_energy: x must be 16-byte aligned");
  launch_energy(x, energy, (long)B * H * W, C, score_inv_scale, (cudaStream_t)cuda_stream);
  return check_cuda(ctx, "stage_energy");
}

// -------------------------------------------------------------------------------------------------
size_t mixaq_block_workspace_bytes(const mixaq_block_params* p, int B, int H, int W) {
  if (!p || B <= 0 || H <= 0 || W <= 0 || p->dim <= 0 || p->hidden <= 0) return 0;
  return carve_block(p, B, H, W, nullptr).bytes;
}

}  // extern "C"

// `presel`: selection buffers already filled for this block (the backbone selects once per stage); NULL: select here.
static mixaq_status block_forward_impl(mixaq_ctx* ctx, const mixaq_block_params* p, const float* x, float* y,
                                       int B, int H, int W, float low_ratio, float prune_ratio,
                                       const mixaq_select_opts* opts, const mixaq_selection* sel_out,
                                       void* workspace, size_t workspace_bytes, const mixaq_taps* taps,
                                       const SelWs* presel, void* cuda_stream) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  mixaq_status s = validate_block(ctx, p);
  if (s != MIXAQ_OK) return s;
  if (!x || !y || x == y) return fail(ctx, MIXAQ_INVALID_ARG, "x / y NULL or aliased");
  if (!aligned_to(x, 16) || !aligned_to(y, 16)) return fail(ctx, MIXAQ_INVALID_ARG, "x and y must be 16-byte aligned");
  if (B <= 0 || H <= 0 || W <= 0) return fail(ctx, MIXAQ_INVALID_ARG, "B, H, W must be positive");
  if (!(low_ratio >= 0.f && low_ratio <= 1.f) || !(prune_ratio >= 0.f && prune_ratio <= 1.f))
    return fail(ctx, MIXAQ_INVALID_ARG, "ratios must lie in [0, 1]");
  if (!p->prepared) return fail(ctx, MIXAQ_INVALID_ARG, "block was not prepared (prepared == NULL)");
  if ((long)B * H * W >= (1L << 31) / WT) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "too many tokens");
  Geometry g = geometry(H, W, low_ratio, prune_ratio);
  if ((size_t)g.nW * 8 > 48 * 1024) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "too many windows per image (max 6144)");
  if (!workspace) return fail(ctx, MIXAQ_INVALID_ARG, "workspace is NULL");
  if (!aligned_to(workspace, 256)) return fail(ctx, MIXAQ_INVALID_ARG, "workspace must be 256-byte aligned");
  std::vector<void*> guard_zones;
  BlockWs ws;
  { GuardScope gs(ctx, &guard_zones); ws = carve_block(p, B, H, W, workspace); }
  if (ws.bytes > workspace_bytes) return fail(ctx, MIXAQ_WORKSPACE_TOO_SMALL, "workspace too small");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int C = p->dim, Hd = p->hidden;
  Prepared pr = carve_prepared(p, p->prepared);
  if (!guard_zones.empty()) launch_guards(guard_zones.data(), (int)guard_zones.size(), true, ctx->d_status, st);
  g_launches = 0;

  // 1. scores and selection
  const SelWs& sel = presel ? *presel : ws.sel;
  if (!presel) {
    const int32_t* energy = opts ? opts->energy : nullptr;
    if (!energy) { PROF(PC_ENERGY); launch_energy(x, ws.energy, (long)B * H * W, C, p->score_inv_scale, st); energy = ws.energy; }
    SelectArgs sa = make_select_args(sel, energy, B, H, W, p->shift, g, opts ? opts->reverse : 0);
    { PROF(PC_SELECT); launch_select(&sa, 1, st); }
  }
  if (sel_out) {
    const size_t n = (size_t)B * g.nW;
    if (sel_out->cls)   cudaMemcpyAsync(sel_out->cls, sel.cls, n, cudaMemcpyDeviceToDevice, st);
    if (sel_out->order) cudaMemcpyAsync(sel_out->order, sel.order, n * 4, cudaMemcpyDeviceToDevice, st);
    if (sel_out->score) cudaMemcpyAsync(sel_out->score, sel.score, n * 8, cudaMemcpyDeviceToDevice, st);
    if (sel_out->idx_hi || sel_out->idx_lo || sel_out->idx_pr) {
      int32_t* const lists[3] = {sel_out->idx_hi, sel_out->idx_lo, sel_out->idx_pr};
      const int cnt[3] = {g.n_hi, g.n_lo, g.n_pr};
      launch_class_lists(sel.cls, B, g.nW, lists, cnt, st);
    }
  }

  const mixaq_branch* brp[2] = {&p->hi, &p->lo};
  const int M[2] = {B * g.n_hi * WT, B * g.n_lo * WT};
  const int slots[2] = {B * g.n_hi, B * g.n_lo};
  const mixaq_branch_taps* tp[2] = {taps ? &taps->hi : nullptr, taps ? &taps->lo : nullptr};
  // bits a stored code occupies: the branch's bit width (bit-packed) or a whole byte
  const int cb[2] = {p->byte_codes ? 8 : p->hi.bits, p->byte_codes ? 8 : p->lo.bits};

  // 2. gather + LN1 + quantize + pack
  LnBranch lb[2];
  for (int i = 0; i < 2; ++i) {
    lb[i].src = x; lb[i].rowsrc = sel.rowsrc[i]; lb[i].gamma = brp[i]->ln1_g; lb[i].beta = brp[i]->ln1_b;
    lb[i].out = ws.a[i]; lb[i].q = to_aq(brp[i]->qkv_in); lb[i].q.bits = cb[i]; lb[i].M = M[i];
  }
  { PROF(PC_LN1); launch_ln_quant(lb[0], lb[1], C, st); }

  // 3. QKV GEMM -> q, k, v codes
  GemmArgs ga;
  ga.status = ctx->d_status;
  ga.w = p->qkv.codes; ga.N = 3 * C; ga.K = C; ga.C = C; ga.mode = EPI_QKV;
  for (int i = 0; i < 2; ++i) {
    fill_gemm_branch(ga.br[i], ws.a[i], M[i], cb[i], pr.mult[0][i], pr.zc[0][i], brp[i]->b_qkv);
    ga.br[i].q0 = to_aq(brp[i]->q); ga.br[i].q1 = to_aq(brp[i]->k); ga.br[i].q2 = to_aq(brp[i]->v);
    ga.br[i].out_bits = cb[i]; ga.br[i].out_codes = ws.qkv[i];
    ga.br[i].tap_acc = tp[i] ? tp[i]->qkv_acc : nullptr;
  }
  { PROF(PC_QKV); if (!launch_gemm(ga, st)) return fail(ctx, MIXAQ_INTERNAL, "GEMM launch set-up failed (tensor map / tile shape)"); }

  // 4. window attention
  AttnArgs aa;
  aa.relbias = pr.relbias; aa.C = C; aa.heads = p->heads; aa.shift = p->shift; aa.Hp = g.Hp; aa.Wp = g.Wp;
  aa.nwx = g.nwx; aa.nW = g.nW;
  const float rs = (float)(1.0 / std::sqrt((double)HEAD_DIM));
  for (int i = 0; i < 2; ++i) {
    AttnBranch& ab = aa.br[i];
    ab.qkv = ws.qkv[i]; ab.out = ws.o[i]; ab.win = sel.win[i];
    ab.q = to_aq(brp[i]->q); ab.k = to_aq(brp[i]->k); ab.v = to_aq(brp[i]->v); ab.o = to_aq(brp[i]->proj_in);
    ab.bits = brp[i]->bits; ab.cbits = cb[i]; ab.slots = slots[i];
    ab.alpha = (brp[i]->q.scale * brp[i]->k.scale) * rs;
    ab.so = (1.0f / (float)((1 << brp[i]->bits) - 1)) * brp[i]->v.scale;
    ab.tap_p = tp[i] ? tp[i]->p_codes : nullptr; ab.tap_probs = tp[i] ? tp[i]->probs : nullptr; ab.tap_pv = tp[i] ? tp[i]->pv_acc : nullptr;
  }
  { PROF(PC_ATTN); launch_attention(aa, st); }

  // 5. proj GEMM + attention residual -> x1
  ga.w = p->proj.codes; ga.N = C; ga.K = C; ga.mode = EPI_PROJ;
  for (int i = 0; i < 2; ++i) {
    fill_gemm_branch(ga.br[i], ws.o[i], M[i], cb[i], pr.mult[1][i], pr.zc[1][i], brp[i]->b_proj);
    ga.br[i].out_f = ws.x1[i]; ga.br[i].res = x; ga.br[i].rowsrc = sel.rowsrc[i];
    ga.br[i].tap_acc = tp[i] ? tp[i]->proj_acc : nullptr;
  }
  { PROF(PC_PROJ); if (!launch_gemm(ga, st)) return fail(ctx, MIXAQ_INTERNAL, "GEMM launch set-up failed (tensor map / tile shape)"); }

  // 6. LN2 + quantize + pack
  for (int i = 0; i < 2; ++i) {
    lb[i].src = ws.x1[i]; lb[i].rowsrc = nullptr; lb[i].gamma = brp[i]->ln2_g; lb[i].beta = brp[i]->ln2_b;
    lb[i].out = ws.f1[i]; lb[i].q = to_aq(brp[i]->fc1_in); lb[i].q.bits = cb[i]; lb[i].M = M[i];
  }
  { PROF(PC_LN2); launch_ln_quant(lb[0], lb[1], C, st); }

  // 7. fc1 GEMM + GELU + requantize
  ga.w = p->fc1.codes; ga.N = Hd; ga.K = C; ga.mode = EPI_FC1;
  for (int i = 0; i < 2; ++i) {
    fill_gemm_branch(ga.br[i], ws.f1[i], M[i], cb[i], pr.mult[2][i], pr.zc[2][i], brp[i]->b_fc1);
    ga.br[i].q0 = to_aq(brp[i]->fc2_in); ga.br[i].out_bits = cb[i]; ga.br[i].out_codes = ws.f2[i];
    ga.br[i].tap_acc = tp[i] ? tp[i]->fc1_acc : nullptr;
  }
  { PROF(PC_FC1); if (!launch_gemm(ga, st)) return fail(ctx, MIXAQ_INTERNAL, "GEMM launch set-up failed (tensor map / tile shape)"); }

  // 8. fc2 GEMM + residual + scatter (reverse shift, crop)
  ga.w = p->fc2.codes; ga.N = C; ga.K = Hd; ga.mode = EPI_FC2;
  for (int i = 0; i < 2; ++i) {
    fill_gemm_branch(ga.br[i], ws.f2[i], M[i], cb[i], pr.mult[3][i], pr.zc[3][i], brp[i]->b_fc2);
    ga.br[i].out_f = y; ga.br[i].res = ws.x1[i]; ga.br[i].rowsrc = sel.rowsrc[i];
    ga.br[i].tap_acc = tp[i] ? tp[i]->fc2_acc : nullptr;
  }
  { PROF(PC_FC2); if (!launch_gemm(ga, st)) return fail(ctx, MIXAQ_INTERNAL, "GEMM launch set-up failed (tensor map / tile shape)"); }

  // 9. pruned windows are forwarded unchanged
  if (g.n_pr > 0) { PROF(PC_COPY); launch_copy_rows(x, y, sel.rowsrc[2], B * g.n_pr * WT, C, st); }

  if (taps) {
    for (int i = 0; i < 2; ++i) {
      const size_t rows = (size_t)M[i]; const int bits = cb[i];
      if (rows == 0) continue;
      if (tp[i]->a_codes)   cudaMemcpyAsync(tp[i]->a_codes, ws.a[i], rows * C * bits / 8, cudaMemcpyDeviceToDevice, st);
      if (tp[i]->qkv_codes) cudaMemcpyAsync(tp[i]->qkv_codes, ws.qkv[i], rows * 3 * C * bits / 8, cudaMemcpyDeviceToDevice, st);
      if (tp[i]->o_codes)   cudaMemcpyAsync(tp[i]->o_codes, ws.o[i], rows * C * bits / 8, cudaMemcpyDeviceToDevice, st);
      if (tp[i]->x1)        cudaMemcpyAsync(tp[i]->x1, ws.x1[i], rows * C * 4, cudaMemcpyDeviceToDevice, st);
      if (tp[i]->f1_codes)  cudaMemcpyAsync(tp[i]->f1_codes, ws.f1[i], rows * C * bits / 8, cudaMemcpyDeviceToDevice, st);
      if (tp[i]->f2_codes)  cudaMemcpyAsync(tp[i]->f2_codes, ws.f2[i], rows * Hd * bits / 8, cudaMemcpyDeviceToDevice, st);
    }
  }
  ctx->launches = g_launches;
  if (!guard_zones.empty()) launch_guards(guard_zones.data(), (int)guard_zones.size(), false, ctx->d_status, st);
  return check_cuda(ctx, "block_forward");
}

extern "C" {

mixaq_status mixaq_block_forward(mixaq_ctx* ctx, const mixaq_block_params* p, const float* x, float* y,
                                 int B, int H, int W, float low_ratio, float prune_ratio,
                                 const mixaq_select_opts* opts, const mixaq_selection* sel_out,
                                 void* workspace, size_t workspace_bytes, const mixaq_taps* taps,
                                 void* cuda_stream) {
  return block_forward_impl(ctx, p, x, y, B, H, W, low_ratio, prune_ratio, opts, sel_out, workspace, workspace_bytes,
                            taps, nullptr, cuda_stream);
}

// -------------------------------------------------------------------------------------------------
size_t mixaq_merge_workspace_bytes(const mixaq_merge_params* p, int B, int H, int W) {
  if (!p || B <= 0 || H <= 0 || W <= 0) return 0;
  const size_t toks = (size_t)B * ((H + 1) / 2) * ((W + 1) / 2);
  return align_up(toks * p->reduction.in_features * p->in.bits / 8);
}

mixaq_status mixaq_merge_forward(mixaq_ctx* ctx, const mixaq_merge_params* p, const float* x, float* y,
                                 int B, int H, int W, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!ctx || !p) return MIXAQ_INVALID_ARG;
  if (!x || !y || !workspace || B <= 0 || H <= 0 || W <= 0) return fail(ctx, MIXAQ_INVALID_ARG, "merge: bad argument");
  if (!aligned_to(x, 16) || !aligned_to(y, 16) || !aligned_to(workspace, 256) || !aligned_to(p->prepared, 256) ||
      !aligned_to(p->reduction.codes, 16) || !aligned_to(p->ln_g, 16) || !aligned_to(p->ln_b, 16))
    return fail(ctx, MIXAQ_INVALID_ARG, "merge: x, y, weights and LayerNorm parameters must be 16-byte aligned, workspace and prepared 256-byte");
  const int K = p->reduction.in_features, N = p->reduction.out_features, C = K / 4;
  if (K % 4 || N % 32 || !merge_dim_supported(C)) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "merge: unsupported dims");
  if (!p->ln_g || !p->ln_b || !p->reduction.codes || !p->reduction.scale || !p->prepared || !bits_ok(p->in.bits) ||
      !aq_ok(p->in, p->in.bits))
    return fail(ctx, MIXAQ_INVALID_ARG, "merge params incomplete");
  if (mixaq_merge_workspace_bytes(p, B, H, W) > workspace_bytes) return fail(ctx, MIXAQ_WORKSPACE_TOO_SMALL, "merge workspace");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  g_launches = 0;
  const int M = B * ((H + 1) / 2) * ((W + 1) / 2);
  MergeGatherArgs mg;
  mg.x = x; mg.gamma = p->ln_g; mg.beta = p->ln_b; mg.out = (uint8_t*)workspace; mg.q = to_aq(p->in);
  mg.B = B; mg.H = H; mg.W = W; mg.C = C;
  { PROF(PC_MERGE_GATHER); launch_merge_gather(mg, st); }
  Carver c(p->prepared, false);
  float* mult = c.take<float>(N);
  int32_t* zc = c.take<int32_t>(N);
  GemmArgs ga;
  ga.status = ctx->d_status;
  ga.w = p->reduction.codes; ga.N = N; ga.K = K; ga.C = N; ga.mode = EPI_MERGE;
  fill_gemm_branch(ga.br[0], (const uint8_t*)workspace, M, p->in.bits, mult, zc, nullptr);
  ga.br[0].out_f = y;
  fill_gemm_branch(ga.br[1], nullptr, 0, p->in.bits, mult, zc, nullptr);
  { PROF(PC_MERGE_GEMM); if (!launch_gemm(ga, st)) return fail(ctx, MIXAQ_INTERNAL, "GEMM launch set-up failed (tensor map / tile shape)"); }
  ctx->launches = g_launches;
  return check_cuda(ctx, "merge_forward");
}

// -------------------------------------------------------------------------------------------------
namespace {
struct BackboneWs {
  float* scratch; int32_t* energy; void* merge; void* block; char* sel;
  float* tokens;            // patch-embedding output (only with p->embed)
  void* embed;              // patch-embedding workspace
  float* raw[16];           // un-normalised stage maps (only with output norms)
  size_t merge_bytes, block_bytes, sel_bytes, embed_bytes, bytes;
};
// H0, W0: size of the token map entering stage 1
BackboneWs carve_backbone(const mixaq_backbone_params* p, int B, int H0, int W0, int Hi, int Wi, void* base) {
  BackboneWs w; Carver c(base);
  size_t max_map = 0, max_tok = 0, max_merge = 0, max_block = 0, max_sel = 0;
  int H = H0, W = W0, blk = 0;
  const bool norms = p->out_norm_g && p->out_norm_b;
  for (int s = 0; s < p->num_stages; ++s) {
    if (s > 0) {
      max_merge = std::max(max_merge, mixaq_merge_workspace_bytes(&p->merges[s - 1], B, H, W));
      H = (H + 1) / 2; W = (W + 1) / 2;
    }
    const mixaq_block_params* b0 = &p->blocks[blk];
    max_map = std::max(max_map, (size_t)B * H * W * b0->dim);
    max_tok = std::max(max_tok, (size_t)B * H * W);
    for (int i = 0; i < p->depths[s]; ++i, ++blk)
      max_block = std::max(max_block, mixaq_block_workspace_bytes(&p->blocks[blk], B, H, W));
    max_sel = std::max(max_sel, (size_t)p->depths[s] * carve_sel(B, H, W, nullptr).bytes);   // one set per block of the stage
    w.raw[s] = (norms && s < 16) ? c.take<float>((size_t)B * H * W * b0->dim) : nullptr;
  }
  w.scratch = c.take<float>(max_map);
  w.energy = c.take<int32_t>(max_tok);
  w.merge = c.take<uint8_t>(max_merge); w.merge_bytes = align_up(max_merge);
  w.block = c.take<uint8_t>(max_block); w.block_bytes = align_up(max_block);
  w.sel = (char*)c.take<uint8_t>(max_sel); w.sel_bytes = align_up(max_sel);
  w.tokens = nullptr; w.embed = nullptr; w.embed_bytes = 0;
  if (p->embed) {
    w.tokens = c.take<float>((size_t)B * H0 * W0 * p->blocks[0].dim);
    const size_t eb = mixaq_embed_workspace_bytes(p->embed, B, Hi, Wi);
    w.embed = c.take<uint8_t>(eb); w.embed_bytes = align_up(eb);
  }
  w.bytes = c.off;
  return w;
}
}  // namespace

size_t mixaq_backbone_workspace_bytes(const mixaq_backbone_params* p, int B, int H0, int W0) {
  if (!p || !p->depths || !p->blocks || p->num_stages <= 0 || p->num_stages > 16 || B <= 0 || H0 <= 0 || W0 <= 0) return 0;
  if (p->num_stages > 1 && !p->merges) return 0;
  const int Ht = p->embed ? (H0 + 3) / 4 : H0, Wt = p->embed ? (W0 + 3) / 4 : W0;
  return carve_backbone(p, B, Ht, Wt, H0, W0, nullptr).bytes;
}

mixaq_status mixaq_backbone_forward(mixaq_ctx* ctx, const mixaq_backbone_params* p, const float* x0,
                                    float* const* stage_out, int B, int H0, int W0,
                                    const float* low_ratio_per_pair, const float* prune_ratio_per_pair,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  if (!p || !p->depths || !p->blocks || p->num_stages <= 0 || (p->num_stages > 1 && !p->merges))
    return fail(ctx, MIXAQ_INVALID_ARG, "backbone params incomplete");
  if (!x0 || !stage_out || !low_ratio_per_pair || !workspace || B <= 0 || H0 <= 0 || W0 <= 0)
    return fail(ctx, MIXAQ_INVALID_ARG, "backbone: bad argument");
  if (!aligned_to(x0, 16) || !aligned_to(workspace, 256))
    return fail(ctx, MIXAQ_INVALID_ARG, "backbone: x0 must be 16-byte aligned, the workspace 256-byte");
  if (p->num_stages > 16) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "at most 16 stages");
  if ((p->out_norm_g != nullptr) != (p->out_norm_b != nullptr)) return fail(ctx, MIXAQ_INVALID_ARG, "output norms need gamma and beta");
  const bool norms = p->out_norm_g && p->out_norm_b;
  if (norms)
    for (int s = 0; s < p->num_stages; ++s)
      if (!p->out_norm_g[s] || !p->out_norm_b[s]) return fail(ctx, MIXAQ_INVALID_ARG, "output norm parameters of a stage are NULL");
  if (p->embed && (!p->embed->prepared || p->embed->proj.out_features != p->blocks[0].dim))
    return fail(ctx, MIXAQ_INVALID_ARG, "embed: not prepared, or its width differs from the first stage's");
  // with a patch embedding in front, H0 x W0 is the image; the token map of stage 1 is a quarter of it
  const int Hi = H0, Wi = W0;
  if (p->embed) { H0 = (Hi + 3) / 4; W0 = (Wi + 3) / 4; }
  int nblk = 0;
  for (int s = 0; s < p->num_stages; ++s) {
    if (p->depths[s] <= 0 || (p->depths[s] != 1 && p->depths[s] % 2)) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "depths must be even or 1");
    if (!stage_out[s]) return fail(ctx, MIXAQ_INVALID_ARG, "stage_out entry is NULL");
    if (!aligned_to(stage_out[s], 16)) return fail(ctx, MIXAQ_INVALID_ARG, "stage_out entries must be 16-byte aligned");
    nblk += p->depths[s];
  }
  for (int b = 0; b < nblk; ++b) {
    mixaq_status s = validate_block(ctx, &p->blocks[b]);
    if (s != MIXAQ_OK) return s;
    float r = low_ratio_per_pair[b / 2], q = prune_ratio_per_pair ? prune_ratio_per_pair[b / 2] : 0.f;
    if (!(r >= 0.f && r <= 1.f) || !(q >= 0.f && q <= 1.f)) return fail(ctx, MIXAQ_INVALID_ARG, "ratios must lie in [0, 1]");
  }
  BackboneWs ws = carve_backbone(p, B, H0, W0, Hi, Wi, workspace);
  if (ws.bytes > workspace_bytes) return fail(ctx, MIXAQ_WORKSPACE_TOO_SMALL, "backbone workspace too small");
  cudaStream_t st = (cudaStream_t)cuda_stream;

  // Replay as a CUDA graph when an identical call was captured before.  The key is made of every value that
  // shapes the launches: the fields of the HOST parameter structs, ratios, pointers, sizes and the stream.
  bool use_graph = ctx->graph_cache && st != nullptr && st != cudaStreamLegacy;
  if (use_graph) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) { cudaGetLastError(); use_graph = false; }
  }
  // A profiled forward is captured too, with the event records around its kernels as graph nodes, launched once and
  // not cached: the kernels are then timed as they run inside a graph, not with a stream launch between the events.
  const bool prof_graph = use_graph && ctx->profiling;
  std::string key;
  if (prof_graph) {
    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); use_graph = false; }
    else ctx->prof_capture = true;
  } else if (use_graph) {
    // field by field: the structs contain padding bytes whose content the caller does not control
    auto put = [&key](const void* ptr, size_t n) { key.append((const char*)ptr, n); };
    auto put_aq = [&](const mixaq_aq& q) { put(&q.bits, 4); put(&q.scale, 4); put(&q.inv_scale, 4); put(&q.zero_point, 4); };
    auto put_lin = [&](const mixaq_linear& l) {
      put(&l.codes, sizeof(l.codes)); put(&l.scale, sizeof(l.scale)); put(&l.out_features, 4); put(&l.in_features, 4); put(&l.bits, 4);
    };
    auto put_branch = [&](const mixaq_branch& b) {
      const float* ptrs[8] = {b.ln1_g, b.ln1_b, b.ln2_g, b.ln2_b, b.b_qkv, b.b_proj, b.b_fc1, b.b_fc2};
      put(ptrs, sizeof(ptrs));
      put_aq(b.qkv_in); put_aq(b.q); put_aq(b.k); put_aq(b.v); put_aq(b.proj_in); put_aq(b.fc1_in); put_aq(b.fc2_in);
      put(&b.bits, 4);
    };
    const int npairs = (nblk + 1) / 2;
    put(&p->num_stages, sizeof(int)); put(p->depths, sizeof(int) * p->num_stages);
    for (int b = 0; b < nblk; ++b) {
      const mixaq_block_params& q = p->blocks[b];
      const int dims[5] = {q.dim, q.heads, q.window, q.shift, q.hidden};
      put(dims, sizeof(dims));
      put_lin(q.qkv); put_lin(q.proj); put_lin(q.fc1); put_lin(q.fc2);
      put(&q.relpos_table, sizeof(q.relpos_table));
      put_branch(q.hi); put_branch(q.lo);
      put(&q.score_inv_scale, 4); put(&q.prepared, sizeof(q.prepared)); put(&q.byte_codes, 4);
    }
    for (int m = 0; m + 1 < p->num_stages; ++m) {
      const mixaq_merge_params& q = p->merges[m];
      put(&q.ln_g, sizeof(q.ln_g)); put(&q.ln_b, sizeof(q.ln_b)); put_aq(q.in); put_lin(q.reduction);
      put(&q.prepared, sizeof(q.prepared));
    }
    const char has_embed = p->embed ? 1 : 0, has_norms = norms ? 1 : 0;
    put(&has_embed, 1); put(&has_norms, 1);
    if (p->embed) {
      const mixaq_embed_params& q = *p->embed;
      put(&q.ln_g, sizeof(q.ln_g)); put(&q.ln_b, sizeof(q.ln_b)); put(&q.bias, sizeof(q.bias)); put_aq(q.in); put_lin(q.proj);
      put(&q.prepared, sizeof(q.prepared));
    }
    if (norms) { put(p->out_norm_g, sizeof(float*) * p->num_stages); put(p->out_norm_b, sizeof(float*) * p->num_stages); }
    put(&x0, sizeof(x0)); put(stage_out, sizeof(float*) * p->num_stages);
    const int dims[5] = {B, H0, W0, Hi, Wi}; put(dims, sizeof(dims));
    put(low_ratio_per_pair, sizeof(float) * npairs);
    const char has_prune = prune_ratio_per_pair ? 1 : 0; put(&has_prune, 1);
    if (prune_ratio_per_pair) put(prune_ratio_per_pair, sizeof(float) * npairs);
    put(&workspace, sizeof(workspace)); put(&workspace_bytes, sizeof(workspace_bytes)); put(&st, sizeof(st));
    const char elev = (ctx->allow_elevation ? 1 : 0) | (ctx->reverse_selection ? 2 : 0); put(&elev, 1);
    for (auto& g : ctx->graphs)
      if (g.key == key) {
        if (cudaGraphLaunch(g.exec, st) != cudaSuccess) return check_cuda(ctx, "backbone_forward (graph launch)");
        ctx->launches = g.launches;
        return MIXAQ_OK;
      }
    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); use_graph = false; }
  }

  mixaq_status result = MIXAQ_OK;
  int total = 0, H = H0, W = W0, blk = 0;
  const float* cur = x0;
  // while profiling: a few event pairs with nothing between them, so that what a bracket itself adds to every kernel's
  // time can be read off the same record
  if (ctx->profiling) for (int i = 0; i < 4; ++i) { PROF(PC_BRACKET); }
  if (p->embed) {
    // image -> token map of stage 1 (patch embedding), inside the same captured graph
    result = mixaq_embed_forward(ctx, p->embed, x0, ws.tokens, B, Hi, Wi, ws.embed, ws.embed_bytes, st);
    total += ctx->launches;
    cur = ws.tokens;
  }
  for (int s = 0; s < p->num_stages && result == MIXAQ_OK; ++s) {
    NvtxScope stage_range(ctx, "stage", s + 1);
    const int d = p->depths[s];
    // with output norms the un-normalised map stays in the workspace (the next stage reads it) and the caller's
    // buffer receives its LayerNorm
    float* out_s = norms ? ws.raw[s] : stage_out[s];
    if (s > 0) {
      // the merge writes where the first block of the stage does NOT write
      float* mdst = (d % 2 == 0) ? out_s : ws.scratch;
      result = mixaq_merge_forward(ctx, &p->merges[s - 1], cur, mdst, B, H, W, ws.merge, ws.merge_bytes, st);
      if (result != MIXAQ_OK) break;
      total += ctx->launches;
      cur = mdst; H = (H + 1) / 2; W = (W + 1) / 2;
    }
    // importance is scored once per stage, before its first block (Section 3.2): one energy map, and from it the
    // window classes and batch bookkeeping of EVERY block of the stage (own shift, own pair's ratios) in one go
    const mixaq_block_params* b0 = &p->blocks[blk];
    { PROF(PC_ENERGY); launch_energy(cur, ws.energy, (long)B * H * W, b0->dim, b0->score_inv_scale, st); }
    total += 1;
    const size_t sel_stride = carve_sel(B, H, W, nullptr).bytes;
    std::vector<SelWs> sels(d);
    std::vector<SelectArgs> sargs(d);
    // Windows keep their precision class within a stage (Section 4.4, "Windows Elevation"): unless elevation is
    // allowed, a pair's effective ratios are the largest ratios of the stage's pairs so far.
    std::vector<float> lr_eff(d), pr_eff(d);
    float lmax = 0.f, pmax = 0.f;
    for (int i = 0; i < d; ++i) {
      float lr = low_ratio_per_pair[(blk + i) / 2], pr = prune_ratio_per_pair ? prune_ratio_per_pair[(blk + i) / 2] : 0.f;
      if (!ctx->allow_elevation) { lmax = std::max(lmax, lr); pmax = std::max(pmax, pr); lr = lmax; pr = pmax; }
      lr_eff[i] = lr; pr_eff[i] = pr;
    }
    for (int i = 0; i < d; ++i) {
      const float lr = lr_eff[i], pr = pr_eff[i];
      Geometry g = geometry(H, W, lr, pr);
      if ((size_t)g.nW * 8 > 48 * 1024) { result = fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "too many windows per image (max 6144)"); break; }
      sels[i] = carve_sel(B, H, W, ws.sel + (size_t)i * sel_stride);
      sargs[i] = make_select_args(sels[i], ws.energy, B, H, W, p->blocks[blk + i].shift, g, ctx->reverse_selection ? 1 : 0);
    }
    if (result != MIXAQ_OK) break;
    g_launches = 0;
    { PROF(PC_SELECT); launch_select(sargs.data(), d, st); }
    total += g_launches;
    for (int i = 0; i < d; ++i, ++blk) {
      float* dst = ((d - 1 - i) % 2 == 0) ? out_s : ws.scratch;
      NvtxScope block_range(ctx, "block", blk);
      result = block_forward_impl(ctx, &p->blocks[blk], cur, dst, B, H, W, lr_eff[i], pr_eff[i], nullptr, nullptr,
                                  ws.block, ws.block_bytes, nullptr, &sels[i], st);
      if (result != MIXAQ_OK) break;
      total += ctx->launches;
      cur = dst;
    }
    if (result == MIXAQ_OK && norms) {
      PROF(PC_OUT_NORM);
      g_launches = 0;
      if (!launch_bias_ln(out_s, nullptr, p->out_norm_g[s], p->out_norm_b[s], stage_out[s], (long)B * H * W, b0->dim, st))
        result = fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "output norm: unsupported width");
      total += g_launches;
    }
  }
  if (use_graph) {
    cudaGraph_t graph = nullptr;
    cudaError_t e = cudaStreamEndCapture(st, &graph);
    ctx->prof_capture = false;
    if (result != MIXAQ_OK) { if (graph) cudaGraphDestroy(graph); cudaGetLastError(); return result; }
    cudaGraphExec_t exec = nullptr;
    if (e != cudaSuccess || !graph || cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) {
      if (graph) cudaGraphDestroy(graph);
      return check_cuda(ctx, "backbone_forward (graph capture)") == MIXAQ_OK
                 ? fail(ctx, MIXAQ_CUDA_ERROR, "backbone_forward: graph capture failed") : MIXAQ_CUDA_ERROR;
    }
    cudaGraphDestroy(graph);
    if (prof_graph && ctx->profiling) {
      ctx->prof_execs.push_back(exec);
    } else {
      if (ctx->graphs.size() >= 16) { cudaGraphExecDestroy(ctx->graphs.front().exec); ctx->graphs.erase(ctx->graphs.begin()); }
      ctx->graphs.push_back({key, exec, total});
    }
    if (cudaGraphLaunch(exec, st) != cudaSuccess) return check_cuda(ctx, "backbone_forward (graph launch)");
  }
  if (result != MIXAQ_OK) return result;
  ctx->launches = total;
  return check_cuda(ctx, "backbone_forward");
}

// -------------------------------------------------------------------------------------------------
// stem and output norms
namespace {
constexpr int EMBED_K = 48, EMBED_KP = 64;     // patch vector, padded to a multiple of 32 codes
struct EmbedPrepared { int8_t* w; float* mult; int32_t* zc; size_t bytes; };
EmbedPrepared carve_embed(const mixaq_embed_params* p, void* base) {
  EmbedPrepared r; Carver c(base, false);
  const int N = p->proj.out_features;
  r.w = c.take<int8_t>((size_t)N * EMBED_KP); r.mult = c.take<float>(N); r.zc = c.take<int32_t>(N);
  r.bytes = c.off;
  return r;
}
bool embed_ok(const mixaq_embed_params* p) {
  return p && p->ln_g && p->ln_b && p->bias && p->proj.codes && p->proj.scale && p->proj.in_features == EMBED_K &&
         p->proj.out_features > 0 && p->proj.out_features % 32 == 0 && ln_dim_supported(p->proj.out_features) &&
         bits_ok(p->in.bits) && aq_ok(p->in, p->in.bits) && p->in.bits == 8;
}
}  // namespace

size_t mixaq_embed_prepared_bytes(const mixaq_embed_params* p) {
  if (!p || p->proj.out_features <= 0) return 0;
  return carve_embed(p, nullptr).bytes;
}

mixaq_status mixaq_embed_prepare(mixaq_ctx* ctx, const mixaq_embed_params* p, void* cuda_stream) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  if (!embed_ok(p) || !p->prepared) return fail(ctx, MIXAQ_INVALID_ARG, "embed params incomplete (8-bit input, [C0][48] projection, C0 % 32 == 0)");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  EmbedPrepared pr = carve_embed(p, p->prepared);
  const int N = p->proj.out_features;
  launch_pad_weights(p->proj.codes, N, EMBED_K, EMBED_KP, pr.w, st);
  launch_prepare_linear(pr.w, p->proj.scale, N, EMBED_KP, p->in.scale, p->in.zero_point, pr.mult, pr.zc, st);
  return check_cuda(ctx, "embed_prepare");
}

size_t mixaq_embed_workspace_bytes(const mixaq_embed_params* p, int B, int Hi, int Wi) {
  if (!p || B <= 0 || Hi <= 0 || Wi <= 0 || p->proj.out_features <= 0) return 0;
  const size_t toks = (size_t)B * ((Hi + 3) / 4) * ((Wi + 3) / 4);
  return carved_bytes(toks * EMBED_KP) + carved_bytes(toks * p->proj.out_features * sizeof(float));
}

mixaq_status mixaq_embed_forward(mixaq_ctx* ctx, const mixaq_embed_params* p, const float* image, float* x0,
                                 int B, int Hi, int Wi, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  if (!embed_ok(p) || !p->prepared) return fail(ctx, MIXAQ_INVALID_ARG, "embed params incomplete");
  if (!image || !x0 || !workspace || B <= 0 || Hi <= 0 || Wi <= 0) return fail(ctx, MIXAQ_INVALID_ARG, "embed: bad argument");
  if (!aligned_to(image, 4) || !aligned_to(x0, 16) || !aligned_to(workspace, 256) || !aligned_to(p->prepared, 256) ||
      !aligned_to(p->ln_g, 16) || !aligned_to(p->ln_b, 16) || !aligned_to(p->bias, 16))
    return fail(ctx, MIXAQ_INVALID_ARG, "embed: x0 and parameters must be 16-byte aligned, workspace and prepared 256-byte");
  if (mixaq_embed_workspace_bytes(p, B, Hi, Wi) > workspace_bytes) return fail(ctx, MIXAQ_WORKSPACE_TOO_SMALL, "embed workspace");
  const size_t toks = (size_t)B * ((Hi + 3) / 4) * ((Wi + 3) / 4);
  if (toks >= (size_t)1 << 31) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "too many tokens");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int N = p->proj.out_features;
  Carver c(workspace);
  uint8_t* codes = c.take<uint8_t>(toks * EMBED_KP);
  float* t = c.take<float>(toks * N);
  EmbedPrepared pr = carve_embed(p, p->prepared);
  g_launches = 0;
  PatchGatherArgs pg; pg.img = image; pg.out = codes; pg.q = to_aq(p->in); pg.B = B; pg.Hi = Hi; pg.Wi = Wi;
  PROF(PC_STEM);
  launch_patch_gather(pg, st);
  GemmArgs ga;
  ga.status = ctx->d_status;
  ga.w = pr.w; ga.N = N; ga.K = EMBED_KP; ga.C = N; ga.mode = EPI_MERGE;      // dequantize only: acc * mult
  fill_gemm_branch(ga.br[0], codes, (int)toks, 8, pr.mult, pr.zc, nullptr);
  ga.br[0].out_f = t;
  fill_gemm_branch(ga.br[1], nullptr, 0, 8, pr.mult, pr.zc, nullptr);
  if (!launch_gemm(ga, st)) return fail(ctx, MIXAQ_INTERNAL, "GEMM launch set-up failed (tensor map / tile shape)");
  if (!launch_bias_ln(t, p->bias, p->ln_g, p->ln_b, x0, (long)toks, N, st)) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "embed: unsupported C0");
  ctx->launches = g_launches;
  return check_cuda(ctx, "embed_forward");
}

mixaq_status mixaq_norm_forward(mixaq_ctx* ctx, const float* gamma, const float* beta, const float* x, float* y,
                                long rows, int C, void* cuda_stream) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  if (!gamma || !beta || !x || !y || rows <= 0 || C <= 0) return fail(ctx, MIXAQ_INVALID_ARG, "norm: bad argument");
  if (!aligned_to(gamma, 16) || !aligned_to(beta, 16) || !aligned_to(x, 16) || !aligned_to(y, 16))
    return fail(ctx, MIXAQ_INVALID_ARG, "norm: pointers must be 16-byte aligned");
  g_launches = 0;
  if (!launch_bias_ln(x, nullptr, gamma, beta, y, rows, C, (cudaStream_t)cuda_stream))
    return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "norm: unsupported C");
  ctx->launches = g_launches;
  return check_cuda(ctx, "norm_forward");
}

mixaq_status mixaq_set_reverse_selection(mixaq_ctx* ctx, int reverse) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  ctx->reverse_selection = reverse != 0;
  return MIXAQ_OK;
}

mixaq_status mixaq_set_workspace_guards(mixaq_ctx* ctx, int enabled) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  ctx->guards = enabled != 0;
  return MIXAQ_OK;
}

mixaq_status mixaq_selftest_workspace_guards(mixaq_ctx* ctx, void* buffer, size_t bytes, int overrun, void* cuda_stream) {
  if (!ctx || !buffer || bytes < 4 * (size_t)(256 + GUARD_BYTES)) return MIXAQ_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  std::vector<void*> zones;
  uint8_t* second = nullptr;
  {
    const bool was = ctx->guards;
    ctx->guards = true;
    GuardScope gs(ctx, &zones);
    Carver c(buffer);
    c.take<uint8_t>(256);
    second = c.take<uint8_t>(256);
    ctx->guards = was;
  }
  launch_guards(zones.data(), (int)zones.size(), true, ctx->d_status, st);
  // a writer that runs one byte past the end of the second buffer (an ordinary write inside the caller's memory)
  if (overrun) cudaMemsetAsync(second + 256, 0, 1, st);
  launch_guards(zones.data(), (int)zones.size(), false, ctx->d_status, st);
  return check_cuda(ctx, "selftest_workspace_guards");
}

mixaq_status mixaq_set_nvtx(mixaq_ctx* ctx, int enabled) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  ctx->nvtx = enabled != 0;
  return MIXAQ_OK;
}

mixaq_status mixaq_set_window_elevation(mixaq_ctx* ctx, int allow) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  ctx->allow_elevation = allow != 0;
  return MIXAQ_OK;
}

mixaq_status mixaq_set_graph_cache(mixaq_ctx* ctx, int enabled) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  ctx->graph_cache = enabled != 0;
  if (!enabled) {
    for (auto& g : ctx->graphs) cudaGraphExecDestroy(g.exec);
    ctx->graphs.clear();
  }
  return MIXAQ_OK;
}

// -------------------------------------------------------------------------------------------------
// calibration (Section 4.3)
namespace {
struct CalWs { int32_t* rowsrc; float *ln, *qkv, *o, *x1, *h; uint32_t* obs; size_t bytes; };
CalWs carve_cal(const mixaq_block_params* p, int B, int H, int W, void* base) {
  CalWs w; Carver c(base);
  Geometry g = geometry(H, W, 0.f, 0.f);
  const size_t M = (size_t)B * g.nW * WT;
  w.obs = c.take<uint32_t>(16);
  w.rowsrc = c.take<int32_t>(M);
  w.ln = c.take<float>(M * p->dim); w.qkv = c.take<float>(M * 3 * p->dim); w.o = c.take<float>(M * p->dim);
  w.x1 = c.take<float>(M * p->dim); w.h = c.take<float>(M * p->hidden);
  w.bytes = c.off;
  return w;
}
// reads the observers' keys back (synchronises) and decodes them
mixaq_status read_ranges(mixaq_ctx* ctx, const uint32_t* d_obs, int sites, mixaq_range* out, cudaStream_t st) {
  uint32_t keys[16];
  if (cudaMemcpyAsync(keys, d_obs, sizeof(uint32_t) * 2 * sites, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) return check_cuda(ctx, "calibrate (read ranges)") == MIXAQ_OK ? MIXAQ_CUDA_ERROR : MIXAQ_CUDA_ERROR;
  for (int i = 0; i < sites; ++i) { out[i].lo = cal_key_to_float(keys[2 * i]); out[i].hi = cal_key_to_float(keys[2 * i + 1]); }
  return MIXAQ_OK;
}
}  // namespace

size_t mixaq_calibrate_block_workspace_bytes(const mixaq_block_params* p, int B, int H, int W) {
  if (!p || B <= 0 || H <= 0 || W <= 0 || p->dim <= 0 || p->hidden <= 0) return 0;
  return carve_cal(p, B, H, W, nullptr).bytes;
}

mixaq_status mixaq_calibrate_block(mixaq_ctx* ctx, const mixaq_block_params* p, int branch, const float* x, float* y,
                                   int B, int H, int W, mixaq_block_ranges* ranges,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!ctx) return MIXAQ_INVALID_ARG;
  mixaq_status s = validate_block(ctx, p, false);
  if (s != MIXAQ_OK) return s;
  if (!x || !y || x == y || !ranges || !workspace || B <= 0 || H <= 0 || W <= 0 || (branch != 0 && branch != 1))
    return fail(ctx, MIXAQ_INVALID_ARG, "calibrate_block: bad argument");
  if (!aligned_to(x, 16) || !aligned_to(y, 16) || !aligned_to(workspace, 256))
    return fail(ctx, MIXAQ_INVALID_ARG, "calibrate_block: x and y must be 16-byte aligned, the workspace 256-byte");
  if ((long)B * H * W >= (1L << 31) / WT) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "too many tokens");
  CalWs ws = carve_cal(p, B, H, W, workspace);
  if (ws.bytes > workspace_bytes) return fail(ctx, MIXAQ_WORKSPACE_TOO_SMALL, "calibrate_block workspace too small");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const mixaq_branch& br = branch == 0 ? p->hi : p->lo;
  CalBlockArgs c;
  c.x = x; c.y = y; c.B = B; c.H = H; c.W = W; c.C = p->dim; c.heads = p->heads; c.hidden = p->hidden; c.shift = p->shift;
  c.ln1_g = br.ln1_g; c.ln1_b = br.ln1_b; c.ln2_g = br.ln2_g; c.ln2_b = br.ln2_b;
  c.b_qkv = br.b_qkv; c.b_proj = br.b_proj; c.b_fc1 = br.b_fc1; c.b_fc2 = br.b_fc2;
  c.w_qkv = p->qkv.codes; c.w_proj = p->proj.codes; c.w_fc1 = p->fc1.codes; c.w_fc2 = p->fc2.codes;
  c.s_qkv = p->qkv.scale; c.s_proj = p->proj.scale; c.s_fc1 = p->fc1.scale; c.s_fc2 = p->fc2.scale; c.relpos = p->relpos_table;
  c.rowsrc = ws.rowsrc; c.ln = ws.ln; c.qkv = ws.qkv; c.o = ws.o; c.x1 = ws.x1; c.h = ws.h; c.obs = ws.obs;
  g_launches = 0;
  if (!launch_calibrate_block(c, st)) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "calibrate_block: unsupported dim");
  ctx->launches = g_launches;
  s = check_cuda(ctx, "calibrate_block");
  if (s != MIXAQ_OK) return s;
  return read_ranges(ctx, ws.obs, 8, &ranges->qkv_in, st);
}

size_t mixaq_calibrate_merge_workspace_bytes(const mixaq_merge_params* p, int B, int H, int W) {
  if (!p || B <= 0 || H <= 0 || W <= 0 || p->reduction.in_features <= 0) return 0;
  const size_t toks = (size_t)B * ((H + 1) / 2) * ((W + 1) / 2);
  return carved_bytes(16 * sizeof(uint32_t)) + carved_bytes(toks * p->reduction.in_features * sizeof(float));
}

mixaq_status mixaq_calibrate_merge(mixaq_ctx* ctx, const mixaq_merge_params* p, const float* x, float* y,
                                   int B, int H, int W, mixaq_range* range,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!ctx || !p) return MIXAQ_INVALID_ARG;
  if (!x || !y || !range || !workspace || B <= 0 || H <= 0 || W <= 0) return fail(ctx, MIXAQ_INVALID_ARG, "calibrate_merge: bad argument");
  if (!aligned_to(x, 16) || !aligned_to(y, 16) || !aligned_to(workspace, 256) || !aligned_to(p->reduction.codes, 16))
    return fail(ctx, MIXAQ_INVALID_ARG, "calibrate_merge: x, y and weights must be 16-byte aligned, the workspace 256-byte");
  const int K = p->reduction.in_features, N = p->reduction.out_features, C = K / 4;
  if (K % 4 || N <= 0 || !merge_dim_supported(C)) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "calibrate_merge: unsupported dims");
  if (!p->ln_g || !p->ln_b || !p->reduction.codes || !p->reduction.scale) return fail(ctx, MIXAQ_INVALID_ARG, "merge params incomplete");
  if (mixaq_calibrate_merge_workspace_bytes(p, B, H, W) > workspace_bytes) return fail(ctx, MIXAQ_WORKSPACE_TOO_SMALL, "calibrate_merge workspace");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  Carver cv(workspace);
  CalMergeArgs c;
  c.obs = cv.take<uint32_t>(16);
  c.ln = cv.take<float>((size_t)B * ((H + 1) / 2) * ((W + 1) / 2) * K);
  c.x = x; c.y = y; c.B = B; c.H = H; c.W = W; c.C = C; c.N = N;
  c.ln_g = p->ln_g; c.ln_b = p->ln_b; c.w = p->reduction.codes; c.sw = p->reduction.scale;
  g_launches = 0;
  if (!launch_calibrate_merge(c, st)) return fail(ctx, MIXAQ_UNSUPPORTED_SHAPE, "calibrate_merge: unsupported dim");
  ctx->launches = g_launches;
  mixaq_status s = check_cuda(ctx, "calibrate_merge");
  if (s != MIXAQ_OK) return s;
  return read_ranges(ctx, c.obs, 1, range, st);
}

mixaq_status mixaq_aq_from_range(float lo, float hi, int bits, mixaq_aq* out) {
  if (!out || !bits_ok(bits) || !(hi > lo)) return MIXAQ_INVALID_ARG;
  const int qmax = (1 << bits) - 1;
  out->bits = bits;
  out->scale = (float)(((double)hi - (double)lo) / (double)qmax);
  out->inv_scale = 1.0f / out->scale;
  double z = std::nearbyint(-(double)lo / (double)out->scale);
  out->zero_point = (int)std::fmin(std::fmax(z, 0.0), (double)qmax);
  return MIXAQ_OK;
}

}  // extern "C"
