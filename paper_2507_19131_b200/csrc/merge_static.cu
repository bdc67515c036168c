// mixaq_merge_forward_static: patch merging for callers that cannot allocate device memory.
//
// Some hosts of this library are not allowed to call cudaMalloc at the point where they run the network:
// an inference plug-in inside an application whose memory pool already owns the whole device, a real-time
// loop in which an allocation (which synchronises the device) would break the frame deadline, or code that
// runs after start-up in a process whose policy forbids further driver allocations.  mixaq_merge_forward
// asks such a caller for a workspace it cannot provide.  This variant needs none: the one intermediate of the
// merge (the quantized, bit-packed [tokens][4C] code matrix that the gather kernel writes and the integer GEMM
// reads) lives in a fixed array that is part of the library image.  Every GPU that loads the library holds
// these MIXAQ_STATIC_SCRATCH_BYTES until the process exits.
#include "../../include/mixaq.h"
#include "kernels.h"
#include <cstdio>
#include <mutex>

namespace mixaq {
bool merge_dim_supported(int C);
int* ctx_status_word(mixaq_ctx* ctx);
void ctx_note(mixaq_ctx* ctx, const char* msg, int launches);
int ctx_device(const mixaq_ctx* ctx);
}  // namespace mixaq

using namespace mixaq;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress, never an address.
static __device__ __align__(256) unsigned char g_merge_scratch[MIXAQ_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the array on the current device; looked up once per device.
cudaError_t scratch_address(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_merge_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

AQ make_aq(const mixaq_aq& q) {
  AQ a; a.scale = q.scale; a.inv_scale = q.inv_scale; a.zp = q.zero_point; a.bits = q.bits;
  a.zpf = (float)q.zero_point; a.qmaxf = (float)((1 << q.bits) - 1);
  return a;
}

size_t round256(size_t v) { return (v + 255) / 256 * 256; }

}  // namespace

extern "C" mixaq_status mixaq_merge_forward_static(mixaq_ctx* ctx, const mixaq_merge_params* p, const float* x,
                                                   float* y, int B, int H, int W, void* cuda_stream) {
  if (!ctx || !p) return MIXAQ_INVALID_ARG;
  char msg[200];
  if (!x || !y || B <= 0 || H <= 0 || W <= 0) { ctx_note(ctx, "merge_forward_static: bad argument", 0); return MIXAQ_INVALID_ARG; }
  const int K = p->reduction.in_features, N = p->reduction.out_features, C = K / 4;
  if (K <= 0 || K % 4 || N <= 0 || N % 32 || !merge_dim_supported(C)) {
    ctx_note(ctx, "merge_forward_static: unsupported dims", 0);
    return MIXAQ_UNSUPPORTED_SHAPE;
  }
  const int bits = p->in.bits;
  if (!p->ln_g || !p->ln_b || !p->reduction.codes || !p->reduction.scale || !p->prepared ||
      !(bits == 8 || bits == 4 || bits == 2) || !(p->in.scale > 0.f) || !(p->in.inv_scale > 0.f) ||
      p->in.zero_point < 0 || p->in.zero_point >= (1 << bits)) {
    ctx_note(ctx, "merge_forward_static: merge params incomplete", 0);
    return MIXAQ_INVALID_ARG;
  }
  const size_t toks = (size_t)B * ((H + 1) / 2) * ((W + 1) / 2);
  const size_t need = toks * (size_t)K * bits / 8;
  if (need > (size_t)MIXAQ_STATIC_SCRATCH_BYTES || toks > (size_t)0x7fffffff) {
    snprintf(msg, sizeof(msg), "merge_forward_static: the code matrix needs %zu bytes, the built-in scratch holds %zu; "
             "use mixaq_merge_forward with a workspace", need, (size_t)MIXAQ_STATIC_SCRATCH_BYTES);
    ctx_note(ctx, msg, 0);
    return MIXAQ_WORKSPACE_TOO_SMALL;
  }
  // the array's address is looked up for the CURRENT device: it has to be the one the context was created on
  int cur_dev = -1;
  if (cudaGetDevice(&cur_dev) != cudaSuccess || cur_dev != ctx_device(ctx)) {
    cudaGetLastError();
    ctx_note(ctx, "merge_forward_static: the current device is not the context's device", 0);
    return MIXAQ_INVALID_ARG;
  }
  unsigned char* scratch = nullptr;
  cudaError_t e = scratch_address(&scratch);
  if (e != cudaSuccess) {
    snprintf(msg, sizeof(msg), "merge_forward_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
    ctx_note(ctx, msg, 0);
    cudaGetLastError();
    return MIXAQ_CUDA_ERROR;
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  g_launches = 0;
  const int M = (int)toks;
  // every byte of the first `need` bytes is rewritten here and nothing beyond them is read below,
  // so whatever an earlier call left in the array does not matter and nothing has to be cleared
  MergeGatherArgs mg;
  mg.x = x; mg.gamma = p->ln_g; mg.beta = p->ln_b; mg.out = scratch; mg.q = make_aq(p->in);
  mg.B = B; mg.H = H; mg.W = W; mg.C = C;
  launch_merge_gather(mg, st);
  float* mult = reinterpret_cast<float*>(p->prepared);
  int32_t* zc = reinterpret_cast<int32_t*>(static_cast<char*>(p->prepared) + round256((size_t)N * 4));
  GemmArgs ga;
  ga.status = ctx_status_word(ctx);
  ga.w = p->reduction.codes; ga.N = N; ga.K = K; ga.C = N; ga.mode = EPI_MERGE;
  for (int i = 0; i < 2; ++i) {
    memset(&ga.br[i], 0, sizeof(GemmBranch));
    ga.br[i].a_bits = bits; ga.br[i].mult = mult; ga.br[i].zc = zc;
  }
  ga.br[0].a = scratch; ga.br[0].M = M; ga.br[0].out_f = y;
  if (!launch_gemm(ga, st)) {
    ctx_note(ctx, "merge_forward_static: GEMM launch set-up failed (tensor map / tile shape)", g_launches);
    return MIXAQ_INTERNAL;
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(msg, sizeof(msg), "merge_forward_static: %s", cudaGetErrorString(e));
    ctx_note(ctx, msg, g_launches);
    return MIXAQ_CUDA_ERROR;
  }
  ctx_note(ctx, nullptr, g_launches);
  return MIXAQ_OK;
}
